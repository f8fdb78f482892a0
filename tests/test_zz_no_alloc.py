"""The allocation-free BvN entry point against the regular one.

moesched_bvn_decompose_static serves callers that are not allowed to allocate device
memory (the memory pool belongs to a host framework, or an allocation could stall a
latency-critical loop): its scratch is an array inside the library. It must return
exactly what moesched_bvn_decompose returns, call after call, although every call reuses
the same array with the previous call's leftovers in it.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_26845_b200 as ms
from paper_2605_26845_b200.workload import bvn_capacity, make_demand, random_matrices

pytestmark = pytest.mark.gpu


def _outputs(demand, k_max):
    B, N, _ = demand.shape
    return ms.Schedule(perm=torch.zeros((B, k_max, N), dtype=torch.uint8, device="cuda"),
                       dur=torch.zeros((B, k_max), dtype=torch.int32, device="cuda"),
                       count=torch.zeros(B, dtype=torch.int32, device="cuda"),
                       status=torch.zeros(B, dtype=torch.int32, device="cuda"),
                       extra=torch.zeros_like(demand))


def _same(a, b):
    assert (a.count == b.count).all() and (a.status == b.status).all()
    kk = torch.arange(a.perm.shape[1], device="cuda")[None, :] < a.count[:, None]
    assert (a.perm[kk] == b.perm[kk]).all() and (a.dur[kk] == b.dur[kk]).all()   # bit-exact, as elsewhere
    assert (a.extra == b.extra).all()


def test_static_entry_point_matches_regular_one_twice_in_a_row():
    # two different batches back to back: the second call finds the first one's data in the array
    batches = [make_demand(3, 48), random_matrices(7, 33, seed=5, kind="uniform", high=9, zero_frac=0.5),
               make_demand(3, 48, seed=99)]
    for D in batches:
        d = torch.from_numpy(np.ascontiguousarray(D)).cuda()
        cap = bvn_capacity(D.shape[1])
        ref = ms.bvn_decompose(d, cap, want_aug=True)
        got = ms.bvn_decompose_static(d, _outputs(d, cap))
        torch.cuda.synchronize()
        _same(got, ref)
        assert (got.status == 0).all()


def test_static_entry_point_against_the_oracle_without_touching_device_memory():
    """Checked against the CPU oracle here, not against the sibling entry point; and the call must leave the
    amount of free device memory exactly as it found it, which is the whole point for a caller
    that cannot allocate. Two shapes: small matrices (one warp per matrix, four matrices per
    CTA) and 200 ranks in a batch of two (one CTA of eight warps per matrix)."""
    cases = [(random_matrices(40, 24, seed=11, kind="uniform", high=50, zero_frac=0.4), bvn_capacity(24)),
             (random_matrices(2, 200, seed=12, kind="uniform", high=9, zero_frac=0.6), 300)]
    for D, k_max in cases:
        d = torch.from_numpy(np.ascontiguousarray(D)).cuda()
        out = _outputs(d, k_max)
        ms.bvn_decompose_static(d, out)                  # first call on the device: address look-up
        torch.cuda.synchronize()
        for t in (out.perm, out.dur, out.count, out.status, out.extra):
            t.zero_()
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        got = ms.bvn_decompose_static(d, out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before
        ref = oracle.bvn_decompose(D, k_max, threads=8)
        count = got.count.cpu().numpy()
        assert (count == ref["count"]).all() and (got.status.cpu().numpy() == ref["status"]).all()
        kk = np.arange(k_max)[None, :] < count[:, None]
        assert (got.perm.cpu().numpy()[kk] == ref["perm"][kk]).all()
        assert (got.dur.cpu().numpy()[kk] == ref["coef"][kk]).all()
        assert (got.extra.cpu().numpy() == ref["aug"]).all()


def test_static_entry_point_rejects_oversized_batches():
    # 300 matrices of 128 x 128 need 19.7 MB of working copy: beyond the 16 MiB array
    d = torch.zeros((300, 128, 128), dtype=torch.int32, device="cuda")
    with pytest.raises(ms.MoeschedError, match="too large"):
        ms.bvn_decompose_static(d, _outputs(d, 4))
    ok = torch.zeros((256, 128, 128), dtype=torch.int32, device="cuda")    # exactly 16 MiB: accepted
    out = ms.bvn_decompose_static(ok, _outputs(ok, 4))
    torch.cuda.synchronize()
    assert (out.count == 0).all() and (out.status == 0).all()
