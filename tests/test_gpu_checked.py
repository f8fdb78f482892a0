"""The range-checked build of the library (libmoesched_checked.so, -DMOESCHED_CHECKED).

No memory checker can be run on the kernels here, so the library has a build in which every index
the kernels derive from the matching state (a matched row or column, a path predecessor, a search
level, a rank) is range-checked, counted when out of range and replaced by 0. This test takes that
build through every kernel at sizes around each layout boundary, compares the results with the CPU
oracle, and requires the counter to stay at zero."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_26845_b200 as ms
from paper_2605_26845_b200 import build as cuda_build
from paper_2605_26845_b200.workload import DEFAULT_MODEL, bvn_capacity, make_demand, random_matrices

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def checked():
    assert ms.debug_index_faults() == -1                 # the regular build has no checks compiled in
    ms.use_library(cuda_build.build(checked=True))
    try:
        assert ms.debug_index_faults() == 0
        yield ms
        assert ms.debug_index_faults() == 0
    finally:
        ms.use_library(None)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def same(gpu, ref, key):
    count = gpu.count.cpu().numpy()
    assert (gpu.status.cpu().numpy() == ref["status"]).all() and (count == ref["count"]).all()
    kk = np.arange(gpu.perm.shape[1])[None, :] < count[:, None]
    assert (gpu.perm.cpu().numpy()[kk] == ref["perm"][kk]).all()
    assert (gpu.dur.cpu().numpy()[kk] == ref[key][kk]).all()


@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 17, 32, 33, 48, 64, 65, 100, 128, 129, 200, 233, 256])
def test_every_kernel_stays_in_bounds_and_agrees_with_the_oracle(checked, N):
    kinds = [dict(kind="uniform", high=1000), dict(kind="ties"), dict(kind="uniform", high=9, zero_frac=0.6)]
    for q, kw in enumerate(kinds):
        D = random_matrices(3, N, seed=12000 + 10 * N + q, **kw)
        if q == 0 and N >= 48:
            D[1] *= 200                                      # one matrix beyond 16 bits: the int32 / cluster paths
        d = dev(D)
        k_mw = N * N + 1 if N <= 33 else 12
        k_bvn = bvn_capacity(N) if N <= 33 else 40
        g = checked.mw_decompose(d, k_mw)
        rg = oracle.mw_decompose(D, k_mw, threads=8)
        same(g, rg, "dur")
        for scratch in (True, False):
            v = checked.bvn_decompose(d, k_bvn, scratch=scratch)
            same(v, oracle.bvn_decompose(D, k_bvn, threads=8), "coef")
        for prefix in (False, True):
            s = checked.schedule_eval(d, g.perm, g.dur, g.count, DEFAULT_MODEL, prefix=prefix)
            rs = oracle.schedule_eval(D, rg["perm"], rg["dur"], rg["count"], DEFAULT_MODEL, threads=8)
            for name in ms.SCORE_FIELDS:
                assert (s[name].cpu().numpy() == rs[name]).all(), name
        if k_mw <= ms.ORDER_MAX_K:
            od = checked.schedule_order(d, g.perm, g.dur, g.count, dict(DEFAULT_MODEL, expert_ps_per_token=400_000))
            ro = oracle.schedule_order(D, rg["perm"], rg["dur"], rg["count"],
                                       dict(DEFAULT_MODEL, expert_ps_per_token=400_000), threads=8)
            assert (od["order"].cpu().numpy() == ro["order"]).all()
        sk = checked.sinkhorn_scale(d, 10, 0.5, 20)
        rk = oracle.sinkhorn_scale(D, 10, 0.5, 20, threads=8)
        assert (sk["scaled"].cpu().numpy() == rk["scaled"]).all()
        rb = checked.bvn_real_decompose(sk["scaled"], k_bvn, 1e-9)
        rr = oracle.bvn_real_decompose(rk["scaled"], k_bvn, tol=1e-9, threads=8)
        assert (rb["count"].cpu().numpy() == rr["count"]).all()
        assert (rb["sum_lambda"].cpu().numpy() == rr["sum_lambda"]).all()
        checked.ideal_a2a(d, DEFAULT_MODEL)
    assert checked.debug_index_faults() == 0


@pytest.mark.parametrize("cfg,B", [(3, 160), (5, 3)])
def test_complete_decompositions_stay_in_bounds(checked, cfg, B):
    """The late, sparse phase of a complete Birkhoff run, and a complete greedy run at 256 ranks (one
    CTA per matrix), under the checks."""
    D = make_demand(cfg, B)
    d = dev(D)
    N = D.shape[1]
    v = checked.bvn_decompose(d, bvn_capacity(N))
    g = checked.mw_decompose(d, 4 * N)
    regular = None
    ms.use_library(None)
    try:
        regular = (ms.bvn_decompose(d, bvn_capacity(N)), ms.mw_decompose(d, 4 * N))
    finally:
        ms.use_library(cuda_build.LIB_CHECKED)
    for a, b in ((v, regular[0]), (g, regular[1])):
        kk = torch.arange(a.perm.shape[1], device="cuda")[None, :] < a.count[:, None]
        assert (a.count == b.count).all() and (a.status == b.status).all() and (a.status == 0).all()
        assert (a.perm[kk] == b.perm[kk]).all() and (a.dur[kk] == b.dur[kk]).all()
    assert checked.debug_index_faults() == 0
