"""Pins for the oracle's schedule scoring (dispatch -> compute -> combine), CPU only."""
import os

import numpy as np
import pytest

import oracle
from paper_2605_26845_b200.workload import DEFAULT_MODEL, bvn_capacity, make_demand, random_matrices

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def one_matching_schedule(N, tokens, k_stride=4):
    perm = np.zeros((1, k_stride, N), np.uint8)
    perm[0, :] = np.arange(N)
    dur = np.zeros((1, k_stride), np.int32)
    dur[0, 0] = tokens
    return perm, dur, np.array([1], np.int32)


def test_link_time_rounding_fixture():
    """One matching, no compute cost, no reconfiguration: overlap makespan = 2 * transfer time."""
    model = dict(DEFAULT_MODEL, reconfig_ns=0, expert_fixed_ns=0, expert_ps_per_token=0)
    for line in open(os.path.join(GOLDEN, "link_time_rounding.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        tokens, ns = map(int, line.split())
        D = np.zeros((1, 4, 4), np.int32)
        D[0, 0, 0] = tokens
        perm, dur, count = one_matching_schedule(4, tokens)
        out = oracle.schedule_eval(D, perm, dur, count, model)
        assert out["makespan_overlap_ns"][0] == 2 * ns
        assert out["makespan_serial_ns"][0] == 2 * ns


def test_single_matching_closed_form():
    # K = 1: nothing overlaps; makespan = 2 (delta + t) + comp in both modes.
    D = np.zeros((1, 4, 4), np.int32)
    D[0, 0, 0], D[0, 1, 1], D[0, 2, 2] = 1000, 400, 3
    perm, dur, count = one_matching_schedule(4, 1000)
    out = oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)
    t = -(-1000 * 14336 * 8 // 400)
    comp = 20_000 + 500                                           # 20 us + 1000 tokens * 0.5 ns
    assert out["makespan_overlap_ns"][0] == out["makespan_serial_ns"][0] == 2 * (10_000 + t) + comp
    assert out["compute_idle_ns"][0] == 0
    assert out["link_idle_tokens"][0] == 4 * 1000 - 1403          # three pairs finish early, one is empty
    assert out["unserved_tokens"][0] == 0 and out["status"][0] == 0


def test_hand_computed_three_matchings():
    # Model with round numbers: 1 token = 10 ns on the link (50 B * 8 / 40 Gb/s), delta = 5 ns,
    # compute = 100 ns + 1 ns/token.
    model = dict(bytes_per_token=50, link_gbps=40, reconfig_ns=5, expert_fixed_ns=100, expert_ps_per_token=1000)
    N = 2
    D = np.array([[[30, 4], [2, 10]]], np.int32)
    perm = np.array([[[0, 1], [1, 0], [0, 1]]], np.uint8)        # identity, swap, identity (nothing left)
    dur = np.array([[30, 4, 1]], np.int32)
    count = np.array([3], np.int32)
    out = oracle.schedule_eval(D, perm, dur, count, model)
    # k=1: served (30,10): g=30, s=40, t=300, comp=130.  k=2: served (4,2): g=4, s=6, t=40, comp=104.
    # k=3: served (0,0): g=0, t=10, comp=0 (no tokens, no kernel).
    # dispatch ends: 305, 350, 365.  compute ends: 435, 539, 539.  combine ends: 740, 785, 800.
    assert out["makespan_overlap_ns"][0] == 800
    assert out["makespan_serial_ns"][0] == (610 + 130) + (90 + 104) + (30 + 0)
    assert out["compute_idle_ns"][0] == (539 - 305) - 234
    assert out["link_idle_tokens"][0] == (60 - 40) + (8 - 6) + (2 - 0)
    assert out["unserved_tokens"][0] == 0
    # the same matchings in another order: the second dispatch now outlasts the first batch
    perm2 = np.array([[[1, 0], [0, 1], [0, 1]]], np.uint8)
    dur2 = np.array([[4, 30, 1]], np.int32)
    out = oracle.schedule_eval(D, perm2, dur2, count, model)
    # dispatch ends: 45, 350, 365.  compute ends: 149, 480, 480.  combine ends: 194, 785, 800.
    assert out["makespan_overlap_ns"][0] == 800
    assert out["compute_idle_ns"][0] == (480 - 45) - 234
    # compute-bound variant: a long fixed cost makes the second batch wait for the first
    model["expert_fixed_ns"] = 1000
    out = oracle.schedule_eval(D, perm, dur, count, model)
    # compute ends: 305+1030=1335, 1335+1004=2339, 2339.  combine: 1640, 2384, 2399.
    assert out["makespan_overlap_ns"][0] == 2399
    assert out["compute_idle_ns"][0] == 0


def critical_path(a, b, c):
    """Makespan of a 3-machine permutation flow shop by its critical-path formula."""
    K = len(a)
    best = 0
    for u in range(K):
        for v in range(u, K):
            best = max(best, sum(a[:u + 1]) + sum(b[u:v + 1]) + sum(c[v:]))
    return best


@pytest.mark.parametrize("cfg,B,kmax", [(1, 16, 8), (2, 6, 16)])
def test_overlap_recurrence_equals_critical_path(cfg, B, kmax):
    D = make_demand(cfg, B)
    N = D.shape[1]
    m = DEFAULT_MODEL
    for dec, key, cap in ((oracle.mw_decompose, "dur", kmax), (oracle.bvn_decompose, "coef", bvn_capacity(N))):
        s = dec(D, cap)
        out = oracle.schedule_eval(D, s["perm"], s[key], s["count"], m)
        for b in range(B):
            K = int(s["count"][b])
            R = D[b].astype(np.int64).copy()
            a, comp = [], []
            for k in range(K):
                d = int(s[key][b, k])
                vals = R[np.arange(N), s["perm"][b, k]]
                served = np.minimum(vals, d)
                R[np.arange(N), s["perm"][b, k]] -= served
                t = -(-d * m["bytes_per_token"] * 8 // m["link_gbps"])
                a.append(m["reconfig_ns"] + t)
                g = int(served.max())
                comp.append(m["expert_fixed_ns"] + -(-g * m["expert_ps_per_token"] // 1000) if g > 0 else 0)
            assert out["makespan_overlap_ns"][b] == critical_path(a, comp, a)
            assert out["makespan_serial_ns"][b] == 2 * sum(a) + sum(comp)
            assert out["makespan_overlap_ns"][b] <= out["makespan_serial_ns"][b]
            assert out["unserved_tokens"][b] == R.sum()
            assert out["compute_idle_ns"][b] >= 0 and out["link_idle_tokens"][b] >= 0


def test_truncated_schedule_leaves_unserved_tokens():
    D = make_demand(2, 4)
    s = oracle.mw_decompose(D, 4)
    out = oracle.schedule_eval(D, s["perm"], s["dur"], s["count"], DEFAULT_MODEL)
    assert (out["unserved_tokens"] == s["residual"].reshape(4, -1).sum(-1)).all()
    assert (out["unserved_tokens"] > 0).all()


def test_empty_schedule():
    D = make_demand(1, 2)
    perm = np.zeros((2, 3, 8), np.uint8)
    out = oracle.schedule_eval(D, perm, np.zeros((2, 3), np.int32), np.zeros(2, np.int32), DEFAULT_MODEL)
    for k in ("makespan_overlap_ns", "makespan_serial_ns", "compute_idle_ns", "link_idle_tokens"):
        assert (out[k] == 0).all()
    assert (out["unserved_tokens"] == D.reshape(2, -1).sum(-1)).all()


def test_bad_schedules_are_flagged():
    D = make_demand(1, 1)
    perm, dur, count = one_matching_schedule(8, 5)
    perm[0, 0, 3] = 2                                             # column 2 twice
    assert oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)["status"][0] == -1
    perm, dur, count = one_matching_schedule(8, 5)
    perm[0, 0, 3] = 9                                             # out of range
    assert oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)["status"][0] == -1
    perm, dur, count = one_matching_schedule(8, 5)
    dur[0, 0] = -5
    assert oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)["status"][0] == -1
    count[0] = 9                                                  # beyond the stride
    dur[0, 0] = 5
    assert oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)["status"][0] == -1


def test_fragmentation_penalty_trend():
    """Sec. 4.2: with a fixed per-batch compute cost the many small BvN matchings cost far more
    than the few large max-weight matchings; the gap closes when compute is purely linear."""
    D = make_demand(2, 8) // 16                                    # small-prompt regime: 512 tokens per rank
    N = D.shape[1]
    g = oracle.mw_decompose(D, 4 * N)
    v = oracle.bvn_decompose(D, bvn_capacity(N))
    ratios = []
    for fixed in (0, 20_000, 80_000):
        m = dict(DEFAULT_MODEL, expert_fixed_ns=fixed)
        mg = oracle.schedule_eval(D, g["perm"], g["dur"], g["count"], m)["makespan_overlap_ns"]
        mv = oracle.schedule_eval(D, v["perm"], v["coef"], v["count"], m)["makespan_overlap_ns"]
        ratios.append(float((mv / mg).mean()))
    assert ratios[0] < ratios[1] < ratios[2] and ratios[2] > 2.0


def test_knee_compute_model():
    """Fig. 1: flat up to the knee, linear beyond; no tokens, no kernel."""
    from paper_2605_26845_b200.workload import PROFILED_MODEL
    m = dict(PROFILED_MODEL, reconfig_ns=0, bytes_per_token=1, link_gbps=8)       # 1 token = 1 ns on the link
    assert m["expert_fixed_ns"] == 250_000 and m["expert_knee_tokens"] == 256
    for tokens, comp in ((1, 250_000), (256, 250_000), (257, 250_001), (1256, 250_500), (2256, 251_000)):
        D = np.zeros((1, 4, 4), np.int32)
        D[0, 1, 2] = tokens
        perm = np.zeros((1, 1, 4), np.uint8)
        perm[0, 0] = [0, 2, 1, 3]
        out = oracle.schedule_eval(D, perm, np.array([[tokens]], np.int32), np.array([1], np.int32), m)
        assert out["makespan_overlap_ns"][0] == 2 * tokens + comp
    # knee = 0 is the affine model
    a = dict(DEFAULT_MODEL)
    b = dict(DEFAULT_MODEL, expert_knee_tokens=0)
    D = make_demand(1, 4)
    s = oracle.mw_decompose(D, 8)
    ra = oracle.schedule_eval(D, s["perm"], s["dur"], s["count"], a)
    rb = oracle.schedule_eval(D, s["perm"], s["dur"], s["count"], b)
    assert (ra["makespan_overlap_ns"] == rb["makespan_overlap_ns"]).all()
    # with the profiled floor the fragmented BvN schedule pays 250 us per matching (Sec. 4.2)
    v = oracle.bvn_decompose(D, bvn_capacity(8))
    rk = oracle.schedule_eval(D, v["perm"], v["coef"], v["count"], PROFILED_MODEL)
    assert (rk["makespan_serial_ns"] >= 250_000 * v["count"]).all()


def test_ideal_all_to_all_bound():
    m = dict(DEFAULT_MODEL)
    # uniform matrix: every port carries N*m tokens
    D = np.full((1, 8, 8), 100, np.int32)
    out = oracle.ideal_a2a(D, m)
    t = -(-800 * 14336 * 8 // 400)
    assert out["comm_ns"][0] == t and out["makespan_ns"][0] == 2 * t + 20_000 + 400
    # incast: column 0 receives from everybody; the receiving port is the bottleneck
    D = np.zeros((1, 8, 8), np.int32)
    D[0, :, 0] = 50
    out = oracle.ideal_a2a(D, m)
    assert out["comm_ns"][0] == -(-400 * 14336 * 8 // 400)
    assert oracle.ideal_a2a(np.zeros((1, 4, 4), np.int32), m)["makespan_ns"][0] == 0
    neg = np.zeros((1, 4, 4), np.int32)
    neg[0, 1, 1] = -3
    assert oracle.ideal_a2a(neg, m)["status"][0] == -1
    # any complete schedule of matchings needs at least the busiest port's tokens of link time, and
    # the BvN schedule of the balanced matrix needs exactly that many (its coefficients sum to T)
    D = make_demand(2, 8)
    ideal = oracle.ideal_a2a(D, m)
    g = oracle.mw_decompose(D, 64)
    v = oracle.bvn_decompose(D, bvn_capacity(16))
    port = np.maximum(D.sum(1).max(1), D.sum(2).max(1))
    for b in range(8):
        assert v["coef"][b, :v["count"][b]].sum() == port[b]
        assert g["dur"][b, :g["count"][b]].sum() >= port[b]
        link = sum(-(-int(c) * 14336 * 8 // 400) for c in v["coef"][b, :v["count"][b]])
        assert ideal["comm_ns"][b] <= link <= ideal["comm_ns"][b] + v["count"][b]


def test_prefix_scores_are_the_scores_of_the_truncated_schedules():
    """A smaller greedy budget yields a prefix (Sec. 3.2), so entry k of the prefix scores must be
    the score of the decomposition run with budget k+1."""
    D = make_demand(2, 5)
    full = oracle.mw_decompose(D, 16)
    pre = oracle.schedule_prefix_eval(D, full["perm"], full["dur"], full["count"], DEFAULT_MODEL)
    for k in (1, 4, 9, 16):
        part = oracle.mw_decompose(D, k)
        sc = oracle.schedule_eval(D, part["perm"], part["dur"], part["count"], DEFAULT_MODEL)
        assert (pre["prefix_overlap_ns"][:, k - 1] == sc["makespan_overlap_ns"]).all()
        assert (pre["prefix_unserved_tokens"][:, k - 1] == sc["unserved_tokens"]).all()
        assert (pre["prefix_unserved_tokens"][:, k - 1] == part["residual"].reshape(5, -1).sum(1)).all()
    # makespan grows and unserved tokens shrink along the prefix
    K = full["count"][0]
    assert (np.diff(pre["prefix_overlap_ns"][0, :K]) > 0).all()
    assert (np.diff(pre["prefix_unserved_tokens"][0, :K]) <= 0).all()
    # hand case (same numbers as the three-matching example): combine ends 740, 785, 800
    model = dict(bytes_per_token=50, link_gbps=40, reconfig_ns=5, expert_fixed_ns=100, expert_ps_per_token=1000)
    D = np.array([[[30, 4], [2, 10]]], np.int32)
    perm = np.array([[[0, 1], [1, 0], [0, 1], [0, 1]]], np.uint8)
    dur = np.array([[30, 4, 1, 0]], np.int32)
    pre = oracle.schedule_prefix_eval(D, perm, dur, np.array([3], np.int32), model)
    assert list(pre["prefix_overlap_ns"][0]) == [740, 785, 800, -1]
    assert list(pre["prefix_unserved_tokens"][0]) == [6, 0, 0, -1]
    perm[0, 1] = [1, 1]
    bad = oracle.schedule_prefix_eval(D, perm, dur, np.array([3], np.int32), model)
    assert bad["status"][0] == -1 and (bad["prefix_overlap_ns"] == -1).all()


def test_stage_sums_beyond_2_to_60_ns_are_rejected_not_wrapped():
    """With the slowest link and the largest token the summed transfer times can pass 63 bits; the
    scoring rejects a schedule whose dispatch stage exceeds 2^60 ns instead of returning a wrapped sum."""
    N, K = 4, 600
    D = np.zeros((2, N, N), np.int32)
    perm = np.tile(np.arange(N, dtype=np.uint8), (2, K, 1))
    dur = np.zeros((2, K), np.int32)
    dur[0, :128] = 2**31 - 1            # sum 2^38: transfer times add up to about 2^61 ns at 2^23 ns per token
    dur[1, :32] = 2**31 - 1             # sum 2^36: about 2^59 ns, within range
    count = np.array([K, K], np.int32)
    model = dict(DEFAULT_MODEL, bytes_per_token=2**20, link_gbps=1)
    r = oracle.schedule_eval(D, perm, dur, count, model)
    assert list(r["status"]) == [-1, 0]
    assert r["makespan_overlap_ns"][0] == 0 and r["makespan_serial_ns"][0] == 0
    t = (2**31 - 1) * 2**23
    assert r["makespan_serial_ns"][1] == 2 * (32 * t + K * model["reconfig_ns"])
    assert r["makespan_overlap_ns"][1] > 2**59
