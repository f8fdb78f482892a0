"""Pins for the oracle's single-matching routines (CPU only).

The lexicographically smallest optimal permutation is checked three ways that
do not share code with the oracle's fast path: enumeration written here with
itertools, a library assignment solver (scipy) for the optimal value, and the
oracle's own enumeration / forced-assignment tiers against its dual-based tier.
"""
import itertools

import numpy as np
import pytest
from scipy.optimize import linear_sum_assignment

import oracle
from paper_2605_26845_b200.workload import random_matrices


def brute_max_weight(W):
    N = W.shape[0]
    best, arg = None, None
    for s in itertools.permutations(range(N)):      # lexicographic order
        w = sum(int(W[i, s[i]]) for i in range(N))
        if best is None or w > best:
            best, arg = w, s
    return best, list(arg)


def brute_support(A):
    N = A.shape[0]
    for s in itertools.permutations(range(N)):
        if all(A[i, s[i]] > 0 for i in range(N)):
            return list(s)
    return None


KINDS = [dict(kind="uniform", high=50), dict(kind="ties"), dict(kind="uniform", high=9, zero_frac=0.6)]


@pytest.mark.parametrize("N", [1, 2, 3, 4, 5, 6])
@pytest.mark.parametrize("kw", KINDS)
def test_max_weight_perm_against_python_enumeration(N, kw):
    mats = random_matrices(40, N, seed=11 + N, **kw)
    for W in mats:
        best, arg = brute_max_weight(W)
        assert oracle.assignment_max(W) == best
        for tier in (0, 1, 2):
            assert list(oracle.max_weight_perm(W, tier)) == arg, (tier, W)


@pytest.mark.parametrize("N", [2, 3, 4, 5, 6])
def test_support_perm_against_python_enumeration(N):
    mats = random_matrices(60, N, seed=23 + N, kind="uniform", high=5, zero_frac=0.45)
    seen_some = False
    for A in mats:
        A = A + np.eye(N, dtype=np.int32)[:, ::-1]       # anti-diagonal keeps a perfect matching
        arg = brute_support(A)
        seen_some |= arg is not None
        for tier in (0, 1, 2):
            got = oracle.support_perm(A, tier)
            assert list(got) == arg, (tier, A)
    assert seen_some


def test_support_perm_reports_missing_matching():
    A = np.array([[1, 1, 0], [0, 0, 0], [1, 0, 1]])
    for tier in (0, 1, 2):
        assert oracle.support_perm(A, tier) is None


@pytest.mark.parametrize("kw", KINDS)
def test_tier1_equals_enumeration_at_n8(kw):
    for N in (7, 8):
        mats = random_matrices(300, N, seed=5 + N, **kw)
        for W in mats:
            assert list(oracle.max_weight_perm(W, 1)) == list(oracle.max_weight_perm(W, 0))
            A = W + np.eye(N, dtype=np.int32)
            assert list(oracle.support_perm(A, 1)) == list(oracle.support_perm(A, 0))


@pytest.mark.parametrize("N", [12, 17, 24])
@pytest.mark.parametrize("kw", KINDS)
def test_tier1_equals_forced_assignment(N, kw):
    mats = random_matrices(12, N, seed=100 + N, **kw)
    for W in mats:
        assert list(oracle.max_weight_perm(W, 1)) == list(oracle.max_weight_perm(W, 2))
        A = W + np.eye(N, dtype=np.int32)
        assert list(oracle.support_perm(A, 1)) == list(oracle.support_perm(A, 2))


@pytest.mark.parametrize("N", [8, 33, 64, 128])
def test_optimal_weight_matches_library_solver(N):
    """The oracle's assignment optimum equals scipy's (a textbook routine)."""
    for kw in KINDS + [dict(kind="uniform", high=65536)]:
        for W in random_matrices(6, N, seed=7 * N, **kw):
            r, c = linear_sum_assignment(W, maximize=True)
            assert oracle.assignment_max(W) == int(W[r, c].sum())
            p = oracle.max_weight_perm(W, 1)
            assert sorted(p) == list(range(N))
            assert int(W[np.arange(N), p].sum()) == int(W[r, c].sum())


def test_lexicographic_rule_on_a_worked_case():
    # Two optimal matchings of weight 4: (0->0, 1->1) and (0->1, 1->0).
    # "Lowest row, then lowest column": row 0 takes column 0.
    W = np.array([[2, 2], [2, 2]])
    assert list(oracle.max_weight_perm(W, 1)) == [0, 1]
    # Row 0 cannot take column 0 in any optimal matching here (that would cost the 9).
    W = np.array([[1, 9, 0], [5, 5, 0], [0, 0, 0]])
    assert list(oracle.max_weight_perm(W, 1)) == [1, 0, 2]
    # Zero entries are ordinary weight-0 edges: the matching is always a full permutation.
    W = np.array([[0, 0, 3], [0, 0, 0], [0, 0, 0]])
    assert list(oracle.max_weight_perm(W, 1)) == [2, 0, 1]


def test_pins_separate_plausible_mistakes():
    """Plausible wrong variants of the rule give a different answer on these inputs,
    so a test above fails if the oracle implements one of them."""
    W = np.array([[1, 9, 0], [0, 0, 0], [5, 5, 0]])
    _, arg = brute_max_weight(W)
    assert arg == [1, 2, 0] and list(oracle.max_weight_perm(W, 1)) == arg
    assert list(oracle.max_weight_perm(W.T.copy(), 1)) != arg      # transposed operand
    assert list(oracle.max_weight_perm(-W, 1)) != arg              # minimising instead of maximising
    # row-by-row argmax is not an optimal matching: rows 0 and 1 both want column 0
    W2 = np.array([[5, 4, 0], [5, 0, 0], [0, 0, 1]])
    assert list(oracle.max_weight_perm(W2, 1)) == [1, 0, 2]
    # highest column on ties would give [1, 0]
    assert list(oracle.max_weight_perm(np.array([[3, 3], [3, 3]]), 1)) == [0, 1]


def test_forced_assignment_agrees_at_64_ranks_on_workload_matrices():
    """Tier 2 (forced assignment: uses optimal VALUES only, no tight graph, no alternating cycles) against
    tier 1 at the headline size, where the big comparisons otherwise rest on tier 1 alone: the first
    matchings of the greedy and of the Birkhoff decomposition of two matrices of configuration 3."""
    from paper_2605_26845_b200.workload import make_demand
    D = make_demand(3, 2)
    K = 6
    a = oracle.mw_decompose(D, K, tier=1, threads=2)
    b = oracle.mw_decompose(D, K, tier=2, threads=2)
    assert (a["count"] == K).all() and (b["count"] == K).all()
    assert (a["perm"] == b["perm"]).all() and (a["dur"] == b["dur"]).all()
    assert (a["residual"] == b["residual"]).all()
    K = 8
    a = oracle.bvn_decompose(D, K, tier=1, threads=2)
    b = oracle.bvn_decompose(D, K, tier=2, threads=2)
    assert (a["count"] == K).all() and (b["count"] == K).all()
    assert (a["perm"] == b["perm"]).all() and (a["coef"] == b["coef"]).all()
