"""Pins of the oracle's Sinkhorn-Knopp scaling (paper Sec. 3.1, the preprocessing it names for the
Birkhoff-von Neumann decomposition) against what the mathematics fixes: the closed form of the 2 x 2
limit, the diagonal-scaling structure, invariances, an independent vectorised statement, and the
properties of the fixed-point matrix, the stretch and the durations derived from it."""
import numpy as np
import pytest

import oracle
from paper_2605_26845_b200.workload import DEFAULT_MODEL, bvn_capacity, make_demand, random_matrices


def test_two_by_two_limit_has_the_closed_form():
    """For [[a, b], [c, d]] the doubly stochastic scaling has S11 = S22 = sqrt(ad) / (sqrt(ad) + sqrt(bc))."""
    rng = np.random.default_rng(5)
    for _ in range(50):
        a, b, c, d = (int(v) for v in rng.integers(1, 1000, size=4))
        r = oracle.sinkhorn_scale(np.array([[[a, b], [c, d]]], np.int32), 2000, 0.0, 20)
        s11 = np.sqrt(a * d) / (np.sqrt(a * d) + np.sqrt(b * c))
        want = np.array([[s11, 1 - s11], [1 - s11, s11]])
        assert np.allclose(r["scaled"][0], want, rtol=0, atol=1e-12), (a, b, c, d)
        assert r["row_err"][0] < 1e-12 and r["status"][0] == 0


def test_transposed_operand_fails_the_closed_form():
    """A matrix and its transpose scale to transposed results: guards against swapped row/column passes
    being hidden by symmetric cases."""
    D = np.array([[[9, 1, 1], [1, 1, 9], [5, 1, 1]]], np.int32)
    a = oracle.sinkhorn_scale(D, 1, 0.5, 20)["scaled"][0]
    b = oracle.sinkhorn_scale(np.ascontiguousarray(D.transpose(0, 2, 1)), 1, 0.5, 20)["scaled"][0]
    # after ONE sweep columns sum to one exactly-ish, rows do not: the order of the two passes is visible
    assert np.allclose(a.sum(0), 1, atol=1e-15) and not np.allclose(a.sum(1), 1, atol=1e-3)
    assert not np.allclose(a, b.T, atol=1e-3)


@pytest.mark.parametrize("N", [3, 8, 17, 64])
def test_result_is_a_diagonal_scaling_of_the_smoothed_matrix_with_unit_sums(N):
    D = random_matrices(3, N, seed=40 + N, kind="uniform", high=50, zero_frac=0.5)
    smooth = 0.25
    r = oracle.sinkhorn_scale(D, 400, smooth, 20)
    X = D.astype(np.float64) + smooth
    for b in range(3):
        S = r["scaled"][b]
        assert np.allclose(S.sum(0), 1, rtol=0, atol=1e-13)
        assert np.allclose(S.sum(1), 1, rtol=0, atol=1e-9)
        ratio = S / X[b]                   # = u_i * v_j: every 2 x 2 minor of the ratio vanishes
        assert np.allclose(ratio[:-1, :-1] * ratio[1:, 1:], ratio[:-1, 1:] * ratio[1:, :-1], rtol=1e-10, atol=0)
        assert abs(r["row_err"][b] - np.abs(S.sum(1) - 1).max()) < 1e-13


def test_against_a_vectorised_statement_and_sweep_by_sweep_error():
    D = make_demand(1, 4)
    prev = None
    for iters in (1, 2, 5, 20):
        r = oracle.sinkhorn_scale(D, iters, 1.0, 20)
        X = D.astype(np.float64) + 1.0
        for _ in range(iters):
            X = X / X.sum(axis=2, keepdims=True)
            X = X / X.sum(axis=1, keepdims=True)
        assert np.allclose(r["scaled"], X, rtol=1e-12, atol=0)
        if prev is not None:
            assert (r["row_err"] <= prev + 1e-15).all()      # the row error never grows
        prev = r["row_err"]


def test_balanced_inputs_and_power_of_two_invariance():
    N = 8                                                # 1/8 is exact in binary floating point
    # a normalisation divides: m * J becomes exactly J / N for ANY m, not only for powers of two
    # (m / (m N) is correctly rounded to 1 / N; m times a rounded 1 / (m N) would not be)
    for m in (7, 8, 12, 1000, 4093):
        J = np.full((1, N, N), m, np.int32)
        r = oracle.sinkhorn_scale(J, 1, 0.0, 20)
        assert (r["scaled"] == 1.0 / N).all() and r["row_err"][0] == 0.0, m
        assert (r["fixed"] == 2**20 // N).all() and r["stretch"][0] == float(m * N)
    # an entry that is its whole row and column becomes exactly 1 whatever its value
    for m in (12, 16, 4093):
        P = np.zeros((1, N, N), np.int32)
        P[0, np.arange(N), np.roll(np.arange(N), 2)] = m
        r = oracle.sinkhorn_scale(P, 3, 0.0, 20)
        assert (r["scaled"][0] == (P[0] > 0)).all()
        assert (r["fixed"][0] == (P[0] > 0) * 2**20).all() and r["stretch"][0] == float(m)
    D = random_matrices(2, 9, seed=3, kind="uniform", high=100)
    a = oracle.sinkhorn_scale(D, 7, 0.5, 16)
    b = oracle.sinkhorn_scale(D * 4, 7, 2.0, 16)        # scaling by a power of two is exact in binary floating point
    assert (a["scaled"] == b["scaled"]).all() and (a["fixed"] == b["fixed"]).all()
    assert (b["stretch"] == 4 * a["stretch"]).all()


def test_rows_or_columns_without_mass_and_negative_entries_are_rejected():
    D = random_matrices(4, 5, seed=9, kind="uniform", high=10)
    D[0, 2, :] = 0
    D[1, :, 3] = 0
    D[2, 1, 1] = -1
    r = oracle.sinkhorn_scale(D, 3, 0.0, 20)
    assert list(r["status"]) == [-1, -1, -1, 0]
    assert (r["scaled"][:3] == 0).all() and (r["fixed"][:3] == 0).all() and (r["stretch"][:3] == 0).all()
    r = oracle.sinkhorn_scale(D, 3, 0.125, 20)           # smoothing gives the empty row and column mass
    assert list(r["status"][[0, 1, 3]]) == [0, 0, 0] and r["status"][2] == -1
    with pytest.raises(ValueError):
        oracle.sinkhorn_scale(D, 0, 0.0, 20)
    with pytest.raises(ValueError):
        oracle.sinkhorn_scale(D, 3, 0.0, 25)


def test_fixed_point_matrix_stretch_and_durations():
    D = make_demand(2, 6)
    bits = 20
    r = oracle.sinkhorn_scale(D, 30, 0.5, bits)
    scale = float(2**bits)
    assert (np.abs(r["fixed"] - r["scaled"] * scale) <= 0.5).all()
    for b in range(D.shape[0]):
        Q, st = r["fixed"][b].astype(np.float64), r["stretch"][b]
        pos = D[b] > 0
        assert (Q[pos] > 0).all() and r["status"][b] == 0
        cap = Q * st / scale                              # tokens each pair can send over the whole schedule
        assert (cap[pos] >= D[b][pos] * (1 - 1e-15)).all()
        assert np.isclose((D[b][pos] / cap[pos]).max(), 1.0, rtol=1e-15)   # the tightest pair sets the stretch
    coef = np.array([[1, 2, 1000, 2**20, 2**23, 0, 5]], np.int32)
    for st in (1.0, 3.5, 1e-3, 4096.0, 1e9):
        dur = oracle.sinkhorn_durations(coef, np.array([6], np.int32), np.array([st]), bits)[0]
        want = [int(np.ceil(int(c) * st / scale)) for c in coef[0, :6]]
        assert list(dur[:6]) == [min(w, 2**31 - 1) for w in want] and dur[6] == 0


def test_sinkhorn_then_birkhoff_serves_all_demand_with_many_small_matchings():
    """The paper's pipeline end to end on the oracle: the scaled schedule is far more fragmented than the
    greedy one (Sec. 3.1, Fig. 2) and, stretched by the tightest pair, it serves every token."""
    D = make_demand(1, 8)
    N = D.shape[1]
    bits = 20
    r = oracle.sinkhorn_scale(D, 50, 0.5, bits)
    assert (r["status"] == 0).all()
    v = oracle.bvn_decompose(r["fixed"], bvn_capacity(N))
    assert (v["status"] == 0).all()
    dur = oracle.sinkhorn_durations(v["coef"], v["count"], r["stretch"], bits)
    score = oracle.schedule_eval(D, v["perm"], dur, v["count"], DEFAULT_MODEL)
    assert (score["status"] == 0).all() and (score["unserved_tokens"] == 0).all()
    g = oracle.mw_decompose(D, N * N)
    assert (v["count"] > 3 * g["count"]).all()
    # the schedule is at least as long as the busiest port needs, and the balancing makes it longer
    port = np.maximum(D.sum(1).max(1), D.sum(2).max(1))
    total = np.array([dur[b, :v["count"][b]].sum() for b in range(D.shape[0])])
    assert (total >= port).all()


# ---- real-valued Birkhoff-von Neumann decomposition (paper Sec. 3.1: A = sum_k lambda_k P_k) ----

def test_real_bvn_on_dyadic_matrices_is_the_integer_decomposition_scaled():
    """For entries that are integers over a power of two every subtraction is exact, so the real-valued
    decomposition must reproduce the (separately pinned) integer one: same matchings, lambda = c / 2^s."""
    for N, seed in ((5, 1), (8, 2), (16, 3), (33, 4)):
        D = random_matrices(4, N, seed=seed, kind="uniform", high=40, zero_frac=0.4)
        v = oracle.bvn_decompose(D, bvn_capacity(N))
        assert (v["status"] == 0).all()
        T = v["aug"].sum(2)[:, 0]
        scale = 2.0 ** 12
        r = oracle.bvn_real_decompose(v["aug"] / scale, bvn_capacity(N), tol=0.0)
        assert (r["status"] == 0).all() and (r["count"] == v["count"]).all() and (r["max_left"] == 0).all()
        for b in range(4):
            K = v["count"][b]
            assert (r["perm"][b, :K] == v["perm"][b, :K]).all()
            assert (r["lam"][b, :K] == v["coef"][b, :K] / scale).all()
            assert r["sum_lambda"][b] == T[b] / scale                 # sum of the coefficients = the common line sum


def test_real_bvn_closed_forms_and_reconstruction():
    N = 8
    J = np.full((1, N, N), 1.0 / N)
    r = oracle.bvn_real_decompose(J, 100, tol=0.0)
    assert r["count"][0] == N and (r["lam"][0, :N] == 1.0 / N).all() and r["sum_lambda"][0] == 1.0
    assert (r["perm"][0, 0] == np.arange(N)).all() and r["status"][0] == 0
    P = np.zeros((1, N, N))
    P[0, np.arange(N), np.roll(np.arange(N), 3)] = 1.0
    r = oracle.bvn_real_decompose(P, 100)
    assert r["count"][0] == 1 and r["lam"][0, 0] == 1.0 and (r["perm"][0, 0] == np.roll(np.arange(N), 3)).all()
    # a scaled demand matrix: the pieces add up to the input, up to what is reported as left over
    D = make_demand(1, 6)
    sk = oracle.sinkhorn_scale(D, 200, 0.5, 20)
    tol = 1e-9
    r = oracle.bvn_real_decompose(sk["scaled"], bvn_capacity(N), tol=tol)
    for b in range(6):
        K = r["count"][b]
        rebuilt = np.zeros((N, N))
        for k in range(K):
            rebuilt[np.arange(N), r["perm"][b, k]] += r["lam"][b, k]
            assert sorted(r["perm"][b, k]) == list(range(N)) and r["lam"][b, k] > tol
        gap = sk["scaled"][b] - rebuilt
        assert gap.min() > -1e-12 and gap.max() <= max(r["max_left"][b], tol) + 1e-12
        assert K <= bvn_capacity(N)
        assert abs(r["sum_lambda"][b] - r["lam"][b, :K].sum()) < 1e-12
        assert 1 - N * (r["max_left"][b] + K * tol) - 1e-9 <= r["sum_lambda"][b] <= 1 + 1e-9
        # the paper reports up to 50 matchings and coefficients of a few hundredths for an 8 x 8 matrix
        # (Sec. 4.2): same order of magnitude here (mean coefficient = about 1 / K)
        assert 0.01 < r["sum_lambda"][b] / K < 0.1 and 3 * N < K <= 50


def test_real_bvn_stops_without_a_perfect_matching_and_rejects_bad_entries():
    A = np.array([[[0.5, 0.5, 0.0], [0.5, 0.5, 0.0], [0.0, 0.0, 0.0]]])
    r = oracle.bvn_real_decompose(A, 10)
    assert r["count"][0] == 0 and r["status"][0] == 1 and r["max_left"][0] == 0.5
    A = np.array([[[0.5, 0.5], [0.5, 0.25]]])                         # the second matching exhausts row 1 early
    r = oracle.bvn_real_decompose(A, 10, tol=0.0)
    assert r["count"][0] == 2 and list(r["lam"][0, :2]) == [0.25, 0.5] and r["status"][0] == 1
    assert r["max_left"][0] == 0.25 and r["sum_lambda"][0] == 0.75
    A = np.array([[[0.5, -0.1], [0.5, 0.5]], [[np.nan, 0.1], [0.5, 0.5]]])
    r = oracle.bvn_real_decompose(A, 10)
    assert list(r["status"]) == [-1, -1] and (r["count"] == 0).all()
    r = oracle.bvn_real_decompose(np.array([[[1.0, 1e-13], [1e-13, 1.0]]]), 10, tol=1e-12)
    assert r["count"][0] == 1 and r["status"][0] == 0               # entries at the tolerance count as zero
    r = oracle.bvn_real_decompose(np.full((1, 4, 4), 0.25), 2, tol=0.0)
    assert r["count"][0] == 2 and r["status"][0] == 1               # budget reached with entries left
