"""Full-depth parity at the sizes of the large workload configurations, through stored digests.

tests/golden/{bvn,mw}_full_depth_config*.txt hold, for a sample of matrices of configurations 3, 4
and 5, the sha256 of the COMPLETE schedule the CPU oracle produces (every permutation and every
coefficient of up to 24 thousand matchings per matrix; written by tests/golden/make_golden.py,
which calls the oracle only). Here the GPU result of the launch shape bench.py times is hashed the
same way: the late, sparse phase of a Birkhoff run, where the records of earlier searches live
longest, is compared with the oracle bit for bit and not only through invariants. The other
placements of the working copy (shared memory / 2-CTA cluster, one warp or one CTA per matrix) must
give the same bits as the benchmarked one on EVERY matrix at full depth.
"""
import hashlib
import os

import numpy as np
import pytest
import torch

import paper_2605_26845_b200 as ms
from paper_2605_26845_b200.workload import CONFIGS, bvn_capacity, make_demand

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(kind, cfg):
    rows = []
    with open(os.path.join(GOLDEN, f"{kind}_full_depth_config{cfg}.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            r, count, h = line.split()
            rows.append((int(r), int(count), h))
    return rows


def digest(count, perm, val):
    h = hashlib.sha256()
    h.update(np.int32(count).astype("<i4").tobytes())
    h.update(np.ascontiguousarray(perm[:count]).tobytes())
    h.update(np.ascontiguousarray(val[:count]).astype("<i4").tobytes())
    return h.hexdigest()


def check_against_golden(s, kind, cfg, min_rows):
    golden = read_golden(kind, cfg)
    assert len(golden) >= min_rows
    count = s.count.cpu().numpy()
    for r, want_count, want in golden:
        assert count[r] == want_count, (kind, cfg, r, int(count[r]), want_count)
        got = digest(int(count[r]), s.perm[r, :count[r]].cpu().numpy(), s.dur[r, :count[r]].cpu().numpy())
        assert got == want, (kind, cfg, r)


def same_schedules(a, b):
    assert (a.count == b.count).all() and (a.status == b.status).all()
    K = int(a.count.max())
    step = 4096                      # compared in slices of the matching axis: the masks stay small
    for k0 in range(0, K, step):
        k1 = min(K, k0 + step)
        kk = torch.arange(k0, k1, device="cuda")[None, :] < a.count[:, None]
        assert (a.perm[:, k0:k1][kk] == b.perm[:, k0:k1][kk]).all()
        assert (a.dur[:, k0:k1][kk] == b.dur[:, k0:k1][kk]).all()


@pytest.mark.parametrize("cfg,min_rows", [(3, 256), (4, 16), (5, 4)])
def test_bvn_complete_schedules_match_the_oracle_digests(cfg, min_rows):
    D = make_demand(cfg)
    d = torch.from_numpy(D).cuda()
    N = D.shape[1]
    s = ms.bvn_decompose(d, bvn_capacity(N))                 # the launch bench.py times for this shape
    assert (s.status == 0).all()
    check_against_golden(s, "bvn", cfg, min_rows)
    if cfg == 3:
        return                                              # placements at N = 64: test_gpu_configs.py
    # every other placement of the working copy, every matrix, full depth
    other = ms.bvn_decompose(d, bvn_capacity(N), scratch=False)   # shared memory (N = 128) / 2-CTA cluster (256)
    same_schedules(other, s)
    del other
    if cfg == 5:
        # 256 matrices go to the CTA-per-matrix kernel; a batch of at least eight matrices per SM takes
        # the one-warp kernel with the working copy in global memory and its search records in shared
        # memory: five copies of the batch make such a launch
        reps = -(-8 * torch.cuda.get_device_properties(0).multi_processor_count // D.shape[0])
        big = d.repeat(reps, 1, 1)
        wide = ms.bvn_decompose(big, bvn_capacity(N))
        for q in range(reps):
            part = ms.Schedule(*(getattr(wide, f)[q * D.shape[0]:(q + 1) * D.shape[0]]
                                 for f in ("perm", "dur", "count", "status")))
            same_schedules(part, s)


@pytest.mark.parametrize("cfg,min_rows", [(4, 1024), (5, 256)])
def test_greedy_largest_budget_matches_the_oracle_digests(cfg, min_rows):
    D = make_demand(cfg)
    d = torch.from_numpy(D).cuda()
    s = ms.mw_decompose(d, max(CONFIGS[cfg]["k_max"]))
    assert ((s.status == 0) | (s.status == 1)).all()
    check_against_golden(s, "mw", cfg, min_rows)
