"""GPU parity of the Sinkhorn-Knopp route (paper Sec. 3.1): the CUDA entry points against the CPU oracle.

Both sides use IEEE double with the same order of operations, so every output is compared bit for bit
(floating-point values with ==), including the integers that floating point decides."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_26845_b200 as ms
from paper_2605_26845_b200.workload import CONFIGS, DEFAULT_MODEL, bvn_capacity, make_demand, random_matrices

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_scale_equal(D, iters, smooth, bits, threads=8):
    g = ms.sinkhorn_scale(dev(D), iters, smooth, bits)
    r = oracle.sinkhorn_scale(D, iters, smooth, bits, threads=threads)
    assert (g["status"].cpu().numpy() == r["status"]).all()
    for name in ("scaled", "fixed", "stretch", "row_err"):
        assert (g[name].cpu().numpy() == r[name]).all(), name
    return g, r


@pytest.mark.parametrize("N", [1, 2, 3, 8, 17, 31, 32, 33, 64, 65, 100, 128, 129, 200, 256])
def test_scaling_is_bit_identical_to_the_oracle(N):
    B = 5 if N <= 128 else 3
    D = random_matrices(B, N, seed=300 + N, kind="uniform", high=2000, zero_frac=0.5)
    assert_scale_equal(D, 1, 0.5, 20)
    assert_scale_equal(D, 7, 0.25, 16)
    D2 = random_matrices(B, N, seed=400 + N, kind="ties")
    assert_scale_equal(D2, 4, 1.0, 24)


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_scaling_of_the_workload_configurations(cfg):
    B = {1: 64, 2: 64, 3: 32, 4: 8, 5: 4}[cfg]
    D = make_demand(cfg, B)
    g, r = assert_scale_equal(D, 20, 0.5, 20)
    assert (r["status"] >= 0).all()


def test_rejected_and_degenerate_inputs():
    D = random_matrices(6, 12, seed=77, kind="uniform", high=10)
    D[0, 2, :] = 0                      # empty row
    D[1, :, 3] = 0                      # empty column
    D[2, 1, 1] = -1
    D[3] = 0                            # no demand at all
    D[4] = 0
    D[4, 0, 0] = 2**31 - 1              # one enormous pair: everything else rounds to zero
    assert_scale_equal(D, 3, 0.0, 20)
    g, r = assert_scale_equal(D, 3, 0.125, 8)
    assert r["status"][2] == -1 and (r["status"][[0, 1, 3]] >= 0).all()
    with pytest.raises(ms.MoeschedError):
        ms.sinkhorn_scale(dev(D), 0, 0.5, 20)
    with pytest.raises(ms.MoeschedError):
        ms.sinkhorn_scale(dev(D), 3, -1.0, 20)
    with pytest.raises(ms.MoeschedError):
        ms.sinkhorn_scale(dev(D), 3, 0.5, 25)
    empty = ms.sinkhorn_scale(torch.zeros((0, 4, 4), dtype=torch.int32, device="cuda"), 3, 0.5, 20)
    assert empty["fixed"].shape[0] == 0


@pytest.mark.parametrize("cfg,B", [(1, 16), (2, 8), (3, 3)])
def test_sinkhorn_birkhoff_pipeline_matches_the_oracle_end_to_end(cfg, B):
    """scale -> exact decomposition of the fixed-point matrix -> durations -> scoring against the
    original demand: every stage equals the oracle's, and the schedule serves every token."""
    D = make_demand(cfg, B)
    N = D.shape[1]
    bits, cap = 20, bvn_capacity(N)
    g, r = assert_scale_equal(D, 20, 0.5, bits)
    v = ms.bvn_decompose(g["fixed"], cap)
    rv = oracle.bvn_decompose(r["fixed"], cap, threads=8)
    count = v.count.cpu().numpy()
    assert (count == rv["count"]).all() and (v.status.cpu().numpy() == rv["status"]).all()
    kk = np.arange(cap)[None, :] < count[:, None]
    assert (v.perm.cpu().numpy()[kk] == rv["perm"][kk]).all()
    assert (v.dur.cpu().numpy()[kk] == rv["coef"][kk]).all()
    dur = ms.sinkhorn_durations(v.dur, v.count, g["stretch"], bits)
    rdur = oracle.sinkhorn_durations(rv["coef"], rv["count"], r["stretch"], bits)
    assert (dur.cpu().numpy()[kk] == rdur[kk]).all()
    s = ms.schedule_eval(dev(D), v.perm, dur, v.count, DEFAULT_MODEL)
    rs = oracle.schedule_eval(D, rv["perm"], rdur, rv["count"], DEFAULT_MODEL, threads=8)
    for name in ms.SCORE_FIELDS + ("status",):
        assert (s[name].cpu().numpy() == rs[name]).all(), name
    assert (rs["unserved_tokens"] == 0).all()


def test_durations_at_the_ends_of_the_range():
    coef = np.array([[1, 2, 1000, 2**20, 2**24, 2**31 - 1, 7, 7]], np.int32).repeat(5, axis=0)
    count = np.array([8, 6, 0, 3, 8], np.int32)
    stretch = np.array([1.0, 3.5, 9.0, 1e-3, 1e12])
    for bits in (1, 20, 24):
        got = ms.sinkhorn_durations(dev(coef), dev(count), dev(stretch), bits).cpu().numpy()
        want = oracle.sinkhorn_durations(coef, count, stretch, bits)
        kk = np.arange(8)[None, :] < count[:, None]
        assert (got[kk] == want[kk]).all()
        assert (got[~kk] == 0).all()           # untouched (the binding hands in zeros)


def test_full_size_headline_batch_properties():
    """At the benchmark's size the oracle checks a sample; the rest is checked by what must hold for any
    matrix: unit column sums, the reported row error, the rounding bound and the stretch."""
    cfg = 3
    D = make_demand(cfg, CONFIGS[cfg]["B"])
    g = ms.sinkhorn_scale(dev(D), 20, 0.5, 20)
    torch.cuda.synchronize()
    S = g["scaled"].cpu().numpy()
    Q = g["fixed"].cpu().numpy()
    assert (g["status"].cpu().numpy() == 0).all()
    assert np.abs(S.sum(1) - 1).max() < 1e-13
    assert np.allclose(np.abs(S.sum(2) - 1).max(1), g["row_err"].cpu().numpy(), rtol=0, atol=1e-13)
    assert (np.abs(Q - S * 2.0**20) <= 0.5).all()
    sample = np.arange(0, D.shape[0], 257)
    r = oracle.sinkhorn_scale(D[sample], 20, 0.5, 20, threads=8)
    assert (S[sample] == r["scaled"]).all() and (Q[sample] == r["fixed"]).all()
    assert (g["stretch"].cpu().numpy()[sample] == r["stretch"]).all()


# ---- real-valued Birkhoff-von Neumann decomposition of the scaled matrix (paper Sec. 3.1) ----

def assert_real_bvn_equal(A, k_max, tol, threads=8):
    g = ms.bvn_real_decompose(dev(A), k_max, tol)
    r = oracle.bvn_real_decompose(A, k_max, tol=tol, threads=threads)
    count = g["count"].cpu().numpy()
    assert (g["status"].cpu().numpy() == r["status"]).all() and (count == r["count"]).all()
    kk = np.arange(k_max)[None, :] < count[:, None]
    assert (g["perm"].cpu().numpy()[kk] == r["perm"][kk]).all()
    assert (g["lam"].cpu().numpy()[kk] == r["lam"][kk]).all()                  # doubles, bit for bit
    assert (g["sum_lambda"].cpu().numpy() == r["sum_lambda"]).all()
    assert (g["max_left"].cpu().numpy() == r["max_left"]).all()
    return g, r


@pytest.mark.parametrize("N", [1, 2, 5, 8, 17, 32, 33, 64, 100, 129, 200])
def test_real_bvn_of_scaled_matrices_is_bit_identical_to_the_oracle(N):
    B = 6 if N <= 64 else 2
    D = random_matrices(B, N, seed=500 + N, kind="uniform", high=300, zero_frac=0.4)
    sk = oracle.sinkhorn_scale(D, 60, 0.5, 20, threads=8)
    k_max = bvn_capacity(N) if N <= 64 else 150
    g, r = assert_real_bvn_equal(sk["scaled"], k_max, 1e-9)
    if N <= 64:
        assert (np.abs(r["sum_lambda"] - 1.0) < 1e-3).all()                    # the coefficients add up to one


def test_real_bvn_of_the_workload_and_special_inputs():
    D = make_demand(3, 24)
    sk = oracle.sinkhorn_scale(D, 20, 0.5, 20, threads=8)
    g, r = assert_real_bvn_equal(sk["scaled"], bvn_capacity(64), 1e-9)
    assert (r["count"] > 500).all()                                           # thousands of small matchings
    # exact inputs, early end without a perfect matching, rejected entries, a short budget
    N = 8
    A = np.zeros((7, N, N))
    A[0] = 1.0 / N
    A[1, np.arange(N), np.roll(np.arange(N), 3)] = 1.0
    A[2, :2, :2] = 0.5                                                         # no perfect matching at all
    A[3] = 1.0 / N
    A[3, 4, 4] = -0.25
    A[4] = 1.0 / N
    A[4, 1, 1] = np.nan
    A[5] = random_matrices(1, N, seed=9, kind="uniform", high=64)[0] / 64.0   # not balanced: stops early
    A[6] = 1e-13                                                               # everything below the tolerance
    g, r = assert_real_bvn_equal(A, 20, 1e-12)
    assert list(r["status"]) == [0, 0, 1, -1, -1, 1, 0] and r["count"][0] == N and r["count"][6] == 0
    assert_real_bvn_equal(A[:1], 3, 0.0)                                       # budget reached: TRUNCATED
    # dyadic matrices: the integer decomposition, scaled (see the oracle's pin), on the GPU as well
    D = random_matrices(4, 16, seed=3, kind="uniform", high=40, zero_frac=0.4)
    v = ms.bvn_decompose(dev(D), want_aug=True)
    g = ms.bvn_real_decompose(v.extra.double() / 4096.0, tol=0.0)
    assert (g["count"] == v.count).all() and (g["status"] == 0).all()
    kk = torch.arange(g["perm"].shape[1], device="cuda")[None, :] < v.count[:, None]
    assert (g["perm"][kk] == v.perm[kk]).all() and (g["lam"][kk] == v.dur[kk].double() / 4096.0).all()
