"""Pins for the oracle's greedy max-weight and Birkhoff-von Neumann decompositions (CPU only)."""
import os

import numpy as np
import pytest
from scipy.optimize import linear_sum_assignment

import oracle
from paper_2605_26845_b200.workload import (CONFIGS, bvn_capacity, make_demand, random_matrices,
                                            structured_cases)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_kv(name):
    out = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            out[k] = int(v)
    return out


def replay_greedy(D, perm, dur, count):
    """Check one greedy schedule step by step; returns the residual."""
    N = D.shape[0]
    R = D.astype(np.int64).copy()
    rows = np.arange(N)
    prev_w = None
    for k in range(count):
        p = perm[k].astype(int)
        assert sorted(p) == list(range(N))
        r, c = linear_sum_assignment(R, maximize=True)          # library optimum on the residual
        w = int(R[rows, p].sum())
        assert w == int(R[r, c].sum())
        assert prev_w is None or w <= prev_w                      # greedy weights never increase
        prev_w = w
        assert int(dur[k]) == int(R[rows, p].max()) and dur[k] > 0
        R[rows, p] = 0
    return R


@pytest.mark.parametrize("cfg,B", [(1, 64), (2, 24), (3, 4)])
def test_greedy_reconstruction_and_optimality(cfg, B):
    D = make_demand(cfg, B)
    N = D.shape[1]
    k_max = 4 * N
    out = oracle.mw_decompose(D, k_max)
    for b in range(B):
        assert out["status"][b] == 0
        R = replay_greedy(D[b], out["perm"][b], out["dur"][b], out["count"][b])
        assert not R.any()                                        # served + residual = D with residual 0
        assert (out["residual"][b] == 0).all()
        assert out["count"][b] <= np.count_nonzero(D[b])
        assert out["count"][b] >= N                               # a dense N x N matrix needs >= N matchings


@pytest.mark.parametrize("k_max", [1, 3, 8])
def test_greedy_budget_truncates(k_max):
    D = make_demand(2, 8)
    out = oracle.mw_decompose(D, k_max)
    full = oracle.mw_decompose(D, 64)
    for b in range(8):
        assert out["count"][b] == k_max and out["status"][b] == 1
        R = replay_greedy(D[b], out["perm"][b], out["dur"][b], k_max)
        assert (R == out["residual"][b]).all() and R.any()
        # a smaller budget yields a prefix of the complete schedule
        assert (out["perm"][b] == full["perm"][b][:k_max]).all()
        assert (out["dur"][b] == full["dur"][b][:k_max]).all()


@pytest.mark.parametrize("N", [1, 2, 5, 8, 17])
def test_closed_form_cases(N):
    cases = structured_cases(N, m=7)
    idx = np.arange(N)
    cap = max(bvn_capacity(N), N)

    z = cases["zero"][None]
    for out in (oracle.mw_decompose(z, 4), oracle.bvn_decompose(z, 4)):
        assert out["count"][0] == 0 and out["status"][0] == 0

    sp = cases["scaled_permutation"][None]                        # D = 7 P: one matching (P, 7) either way
    g, v = oracle.mw_decompose(sp, cap), oracle.bvn_decompose(sp, cap)
    assert g["count"][0] == 1 and v["count"][0] == 1
    assert (g["perm"][0, 0] == (idx + 1) % N).all() and g["dur"][0, 0] == 7
    assert (v["perm"][0, 0] == (idx + 1) % N).all() and v["coef"][0, 0] == 7
    assert (v["aug"][0] == sp[0]).all()                           # already balanced: nothing is added

    un = cases["uniform"][None]                                   # D = 7 J: N matchings of 7, identity first
    g, v = oracle.mw_decompose(un, cap), oracle.bvn_decompose(un, cap)
    assert g["count"][0] == N and v["count"][0] == N
    assert (g["dur"][0, :N] == 7).all() and (v["coef"][0, :N] == 7).all()
    assert (g["perm"][0, 0] == idx).all() and (v["perm"][0, 0] == idx).all()

    hc = cases["hot_column"][None]                                # incast: one sender per matching
    g = oracle.mw_decompose(hc, cap)
    assert g["count"][0] == N and (g["dur"][0, :N] == 7).all()
    assert sorted(np.argmax(g["perm"][0, :N] == 0, axis=1)) == list(range(N))

    dg = cases["diagonal"][None]
    g = oracle.mw_decompose(dg, cap)
    assert g["count"][0] == 1 and (g["perm"][0, 0] == idx).all() and g["dur"][0, 0] == N


def test_paper_counts_fixture():
    """Fig. 2: 50 BvN matchings and 7 max-weight matchings on an 8 x 8 matrix."""
    kv = read_kv("paper_fig2_matching_counts.txt")
    N = kv["N"]
    assert bvn_capacity(N) == kv["bvn_matchings"]
    # dense 8x8 with an empty diagonal: N-1 greedy matchings at least, N^2-2N+2 BvN matchings at most
    D = random_matrices(32, N, seed=3, kind="uniform", high=4000) + 1
    D[:, np.arange(N), np.arange(N)] = 0
    g = oracle.mw_decompose(D, 64)
    v = oracle.bvn_decompose(D, 64)
    assert (g["count"] >= kv["mw_matchings"]).all() and (g["count"] == kv["mw_matchings"]).any()
    assert (v["count"] <= kv["bvn_matchings"]).all() and (v["count"] > 4 * kv["mw_matchings"]).all()


@pytest.mark.parametrize("N", [2, 3, 8, 16, 33])
def test_augmentation_invariants(N):
    for kw in (dict(kind="uniform", high=100), dict(kind="uniform", high=9, zero_frac=0.6), dict(kind="ties")):
        for D in random_matrices(20, N, seed=31 * N, **kw):
            A = oracle.augment(D)
            E = A - D
            T = max(D.sum(0).max(), D.sum(1).max())
            assert (A.sum(0) == T).all() and (A.sum(1) == T).all()
            assert (E >= 0).all() and np.count_nonzero(E) <= 2 * N - 1
            assert E.sum() == N * T - D.sum()
            # north-west corner: the added cells form a monotone staircase
            cells = np.argwhere(E > 0)
            assert (np.diff(cells[:, 0]) >= 0).all() and (np.diff(cells[:, 1]) >= 0).all()
    D = np.array([[1, 0], [0, 0]], np.int32)                      # worked case: deficits (0,1) x (0,1)
    assert (oracle.augment(D) == np.array([[1, 0], [0, 1]])).all()
    D = np.array([[0, 3], [0, 0]], np.int32)                      # T=3; row 1 lacks 3, column 0 lacks 3
    assert (oracle.augment(D) == np.array([[0, 3], [3, 0]])).all()


def replay_bvn(A, perm, coef, count):
    N = A.shape[0]
    A = A.astype(np.int64).copy()
    rows = np.arange(N)
    for k in range(count):
        p = perm[k].astype(int)
        assert sorted(p) == list(range(N))
        vals = A[rows, p]
        assert vals.min() >= 1 and coef[k] == vals.min()          # coefficient = smallest matched entry
        A[rows, p] -= coef[k]
        assert (A.sum(0) == A.sum(1)[0]).all() and (A.sum(1) == A.sum(1)[0]).all()
    return A


@pytest.mark.parametrize("cfg,B", [(1, 64), (2, 16), (3, 2)])
def test_bvn_exact_reconstruction_and_bound(cfg, B):
    D = make_demand(cfg, B)
    N = D.shape[1]
    cap = bvn_capacity(N)
    out = oracle.bvn_decompose(D, cap)
    for b in range(B):
        assert out["status"][b] == 0 and out["count"][b] <= cap   # Birkhoff bound N^2 - 2N + 2
        assert (out["aug"][b] == oracle.augment(D[b])).all()
        left = replay_bvn(out["aug"][b], out["perm"][b], out["coef"][b], out["count"][b])
        assert not left.any()                                     # sum_k c_k P_k = A exactly
        assert out["count"][b] <= np.count_nonzero(out["aug"][b]) - 2 * N + 2 or N == 1


def test_bvn_takes_lexmin_support_matching_each_step():
    for D in random_matrices(30, 6, seed=77, kind="uniform", high=6, zero_frac=0.3):
        out = oracle.bvn_decompose(D[None], bvn_capacity(6), tier=1)
        A = out["aug"][0].astype(np.int64)
        for k in range(out["count"][0]):
            assert list(out["perm"][0, k]) == list(oracle.support_perm(A, 0))   # enumeration tier
            A[np.arange(6), out["perm"][0, k]] -= out["coef"][0, k]


@pytest.mark.parametrize("tier", [0, 2])
def test_decompositions_agree_across_tiers(tier):
    N = 8 if tier == 0 else 12
    for kw in (dict(kind="uniform", high=30), dict(kind="ties"), dict(kind="uniform", high=9, zero_frac=0.6)):
        D = random_matrices(6, N, seed=900 + tier, **kw)
        for fn, key in ((oracle.mw_decompose, "dur"), (oracle.bvn_decompose, "coef")):
            a = fn(D, bvn_capacity(N), tier=1)
            b = fn(D, bvn_capacity(N), tier=tier)
            assert (a["count"] == b["count"]).all() and (a["status"] == b["status"]).all()
            assert (a["perm"] == b["perm"]).all() and (a[key] == b[key]).all()


def test_bvn_budget_truncates():
    D = make_demand(1, 4)
    out = oracle.bvn_decompose(D, 5)
    assert (out["count"] == 5).all() and (out["status"] == 1).all()


def test_bad_input_status():
    D = make_demand(1, 3)
    D[1, 2, 3] = -1
    g, v = oracle.mw_decompose(D, 8), oracle.bvn_decompose(D, 50)
    for out in (g, v):
        assert list(out["status"]) == [0, -1, 0] and out["count"][1] == 0
    big = np.zeros((1, 8, 8), np.int32)
    big[0, 0, 0] = 2**31 - 1                                      # entries above 2^28 are out of range for the greedy path
    assert oracle.mw_decompose(big, 8)["status"][0] == -1
    assert oracle.bvn_decompose(big, 50)["status"][0] == 0
    big[0, 0, 1] = 1                                              # row sum overflows 31 bits (BvN)
    assert oracle.bvn_decompose(big, 50)["status"][0] == -1


def test_multithreaded_run_equals_serial():
    D = make_demand(2, 12)
    a = oracle.mw_decompose(D, 16, threads=1)
    b = oracle.mw_decompose(D, 16, threads=4)
    assert all((a[k] == b[k]).all() for k in a)


def test_workload_shapes():
    for cfg, c in CONFIGS.items():
        D = make_demand(cfg, 2)
        assert D.shape == (2, c["N"], c["N"]) and D.dtype == np.int32 and (D >= 0).all()
        assert (D.sum(-1) == c["tokens"] * c["top_k"]).all()
        assert D.max() <= c["tokens"] * min(c["top_k"], c["experts"] // c["N"])
    assert abs((make_demand(5, 2) == 0).mean() - 0.6) < 0.05
    assert (make_demand(3, 3) == make_demand(3, 3)).all()
