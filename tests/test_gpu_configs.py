"""GPU parity at the full sizes of the five workload configurations.

The CPU oracle costs O(N^3) per matching, so at full size it is run on every matrix where
that takes seconds and on a stated sample (or a schedule prefix: a smaller budget yields a
prefix of the complete schedule) elsewhere; every remaining GPU output is checked through
properties that hold at any size: each matching is a permutation, durations / coefficients
follow from the replayed matrix, greedy weights never increase, the pieces add up to the
input exactly, the Birkhoff bound holds.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_26845_b200 as ms
from paper_2605_26845_b200.workload import CONFIGS, DEFAULT_MODEL, bvn_capacity, make_demand

pytestmark = pytest.mark.gpu
THREADS = oracle.hardware_threads()

_cache = {}


def demand(cfg):
    if cfg not in _cache:
        _cache.clear()                      # one configuration at a time keeps host memory small
        D = make_demand(cfg)
        _cache[cfg] = (D, torch.from_numpy(D).cuda())
    return _cache[cfg]


def used(s):
    return torch.arange(s.perm.shape[1], device="cuda")[None, :] < s.count[:, None]


def compare_prefix(s, ref, key, rows, kcap=None):
    """GPU schedule rows `rows` against oracle output computed for those rows (first kcap matchings)."""
    count = s.count[rows].cpu().numpy()
    rc = ref["count"]
    if kcap is not None:
        count = np.minimum(count, kcap)
    assert (count == rc).all(), (count[:8], rc[:8])
    K = ref["perm"].shape[1]
    perm = s.perm[rows, :K].cpu().numpy()
    dur = s.dur[rows, :K].cpu().numpy()
    kk = np.arange(K)[None, :] < rc[:, None]
    assert (perm[kk] == ref["perm"][kk]).all()
    assert (dur[kk] == ref[key][kk]).all()


def replay_greedy(d, s):
    """Properties of a greedy schedule, vectorised over the batch; returns the residual."""
    B, N, _ = d.shape
    R = d.to(torch.int64).clone()
    rows = torch.arange(N, device="cuda")[None, :].expand(B, N)
    bidx = torch.arange(B, device="cuda")[:, None].expand(B, N)
    prev = None
    for k in range(int(s.count.max())):
        live = s.count > k
        p = s.perm[:, k].to(torch.int64)
        p = torch.where(live[:, None], p, rows)                       # unused rows: harmless identity
        assert (torch.sort(p, dim=1).values == rows).all()            # a permutation
        vals = R[bidx, rows, p]
        w = vals.sum(1)
        assert (s.dur[:, k].to(torch.int64)[live] == vals.max(1).values[live]).all()
        assert (vals.max(1).values[live] > 0).all()
        if prev is not None:
            assert (w[live] <= prev[live]).all()                      # greedy weights never increase
        prev = w
        R[bidx, rows, p] = torch.where(live[:, None], torch.zeros_like(vals), vals)
    return R


def replay_bvn(aug, s):
    """sum_k c_k P_k must rebuild the balanced matrix exactly; coefficient = smallest matched entry."""
    B, N, _ = aug.shape
    A = aug.to(torch.int64).clone()
    rows = torch.arange(N, device="cuda")[None, :].expand(B, N)
    bidx = torch.arange(B, device="cuda")[:, None].expand(B, N)
    ok = torch.ones((), dtype=torch.bool, device="cuda")
    for k in range(int(s.count.max())):
        live = s.count > k
        p = torch.where(live[:, None], s.perm[:, k].to(torch.int64), rows)
        vals = A[bidx, rows, p]
        c = torch.where(live, s.dur[:, k].to(torch.int64), torch.zeros_like(s.count, dtype=torch.int64))
        ok &= (torch.sort(p, dim=1).values == rows).all()
        ok &= ((vals.min(1).values == c) | ~live).all() & ((c >= 1) | ~live).all()
        A[bidx, rows, p] = vals - c[:, None]
    assert bool(ok)
    return A


def eval_against_oracle(D, d, s, key, rows, model=DEFAULT_MODEL):
    got = ms.schedule_eval(d, s.perm, s.dur, s.count, model)
    assert (got["status"] == 0).all()
    assert (got["makespan_overlap_ns"] <= got["makespan_serial_ns"]).all()
    perm = s.perm[rows].cpu().numpy()
    dur = s.dur[rows].cpu().numpy()
    count = s.count[rows].cpu().numpy()
    kk = np.arange(perm.shape[1])[None, :] < count[:, None]
    perm = np.where(kk[:, :, None], perm, 0)                           # unused rows are never read
    ref = oracle.schedule_eval(D[rows.cpu().numpy()], perm, np.where(kk, dur, 0), count, model, threads=THREADS)
    for name in ms.SCORE_FIELDS:
        assert (got[name][rows].cpu().numpy() == ref[name]).all(), name
    return got


def sample_rows(B, n):
    return torch.arange(0, B, max(1, B // n), device="cuda")[:n]


# per configuration: greedy matrices checked against the oracle per budget, BvN matrices and prefix length
PLAN = {
    1: dict(mw_rows={8: 64}, bvn_rows=64, bvn_prefix=None),
    2: dict(mw_rows={4: 1024, 16: 1024}, bvn_rows=1024, bvn_prefix=None),
    3: dict(mw_rows={8: 128, 16: 128, 64: 4096}, bvn_rows=64, bvn_prefix=None),
    4: dict(mw_rows={16: 64, 32: 64, 128: 256}, bvn_rows=16, bvn_prefix=None),
    5: dict(mw_rows={4: 32, 8: 32, 16: 32, 32: 32, 256: 32}, bvn_rows=16, bvn_prefix=40),
}
# Complete schedules of many more matrices (configuration 3: 512, 4: 64 Birkhoff and 256 greedy,
# 5: 8 Birkhoff and 32 greedy, every matching of each) are compared through the oracle's stored
# digests in test_gpu_golden.py; here the oracle itself runs, element by element, on what it
# finishes in about a minute.


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_greedy_at_full_size(cfg):
    D, d = demand(cfg)
    B, N, _ = D.shape
    full = None
    for k_max, nrows in PLAN[cfg]["mw_rows"].items():
        s = ms.mw_decompose(d, k_max, want_residual=True)
        assert ((s.status == 0) | (s.status == 1)).all()
        R = replay_greedy(d, s)
        assert (R == s.extra.to(torch.int64)).all()                   # served + residual = demand
        assert ((s.status == 0) == (R.reshape(B, -1).sum(1) == 0)).all()
        assert ((s.status == 1) <= (s.count == k_max)).all()
        rows = sample_rows(B, nrows)
        ref = oracle.mw_decompose(D[rows.cpu().numpy()], k_max, threads=THREADS, want_residual=False)
        compare_prefix(s, ref, "dur", rows)
        assert (s.status[rows].cpu().numpy() == ref["status"]).all()
        eval_against_oracle(D, d, s, "dur", sample_rows(B, min(nrows, 64)))
        if full is not None:                                           # a smaller budget yields a prefix
            kk = used(full)
            kp = full.perm.shape[1]
            assert (s.perm[:, :kp][kk] == full.perm[kk]).all() and (s.dur[:, :kp][kk] == full.dur[kk]).all()
        full = s


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_bvn_at_full_size(cfg):
    D, d = demand(cfg)
    B, N, _ = D.shape
    cap = bvn_capacity(N)
    s = ms.bvn_decompose(d, cap, want_aug=True)                        # the launch shape bench.py times
    assert (s.status == 0).all() and (s.count <= cap).all()            # Birkhoff bound N^2 - 2N + 2
    aug = s.extra
    T = torch.maximum(d.sum(1).max(1).values, d.sum(2).max(1).values)
    assert (aug.sum(1) == T[:, None]).all() and (aug.sum(2) == T[:, None]).all() and (aug >= d).all()
    assert ((aug != d).reshape(B, -1).sum(1) <= 2 * N - 1).all()
    left = replay_bvn(aug, s)
    assert not left.any()
    plan = PLAN[cfg]
    rows = sample_rows(B, plan["bvn_rows"])
    k_ref = plan["bvn_prefix"] or cap
    ref = oracle.bvn_decompose(D[rows.cpu().numpy()], k_ref, threads=THREADS)
    compare_prefix(s, ref, "coef", rows, kcap=plan["bvn_prefix"])
    assert (aug[rows].cpu().numpy() == ref["aug"]).all()
    models = [DEFAULT_MODEL]
    if "expert_fixed_ns" in CONFIGS[cfg]:
        models = [dict(DEFAULT_MODEL, expert_fixed_ns=f) for f in CONFIGS[cfg]["expert_fixed_ns"]]
    overlap = []
    for m in models:
        got = eval_against_oracle(D, d, s, "coef", sample_rows(B, 8), m)
        assert (got["unserved_tokens"] == 0).all()
        overlap.append(got["makespan_overlap_ns"].double().mean().item())
    assert overlap == sorted(overlap)                                  # a larger fixed cost never helps
    if cfg == 3:
        # the shared-memory placement gives the same bits as the global working copy
        s2 = ms.bvn_decompose(d, cap, scratch=False)
        kk = used(s)
        assert (s2.count == s.count).all() and (s2.perm[kk] == s.perm[kk]).all() and (s2.dur[kk] == s.dur[kk]).all()


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_ideal_all_to_all_at_full_size(cfg):
    from paper_2605_26845_b200.workload import PROFILED_MODEL
    D, d = demand(cfg)
    for model in (DEFAULT_MODEL, PROFILED_MODEL):
        got = ms.ideal_a2a(d, model)
        ref = oracle.ideal_a2a(D, model)                               # cheap: every matrix
        for name in ("comm_ns", "makespan_ns", "status"):
            assert (got[name].cpu().numpy() == ref[name]).all(), name
    # no schedule of matchings can move the busiest port's tokens in less link time
    s = ms.mw_decompose(d, 4 * D.shape[1])
    complete = s.status == 0
    total = torch.where(used(s), s.dur, torch.zeros_like(s.dur)).sum(1).to(torch.int64)
    port = torch.maximum(d.sum(1).max(1).values, d.sum(2).max(1).values)
    assert (total[complete] >= port[complete]).all()


@pytest.mark.parametrize("cfg", [2, 3, 5])
def test_budget_sweep_from_one_decomposition(cfg):
    """The greedy schedule with the largest budget plus its prefix scores reproduce the scores of
    every smaller budget of the configuration."""
    D, d = demand(cfg)
    B = D.shape[0]
    budgets = CONFIGS[cfg]["k_max"]
    full = ms.mw_decompose(d, max(budgets))
    pre = ms.schedule_eval(d, full.perm, full.dur, full.count, DEFAULT_MODEL, prefix=True)
    rows = sample_rows(B, 16)
    rnp = rows.cpu().numpy()
    for k in budgets:
        part = ms.mw_decompose(d, k)
        sc = ms.schedule_eval(d, part.perm, part.dur, part.count, DEFAULT_MODEL)
        last = (part.count - 1).clamp(min=0).to(torch.int64)[:, None]
        some = part.count > 0
        assert (pre["prefix_overlap_ns"].gather(1, last)[:, 0][some] == sc["makespan_overlap_ns"][some]).all()
        assert (pre["prefix_unserved_tokens"].gather(1, last)[:, 0][some] == sc["unserved_tokens"][some]).all()
        ref = oracle.mw_decompose(D[rnp], k, threads=THREADS)
        osc = oracle.schedule_eval(D[rnp], ref["perm"], ref["dur"], ref["count"], DEFAULT_MODEL, threads=THREADS)
        assert (sc["makespan_overlap_ns"][rows].cpu().numpy() == osc["makespan_overlap_ns"]).all()
