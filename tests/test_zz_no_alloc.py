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


def test_static_entry_point_rejects_oversized_batches():
    # 300 matrices of 128 x 128 need 19.7 MB of working copy: beyond the 16 MiB array
    d = torch.zeros((300, 128, 128), dtype=torch.int32, device="cuda")
    with pytest.raises(ms.MoeschedError, match="too large"):
        ms.bvn_decompose_static(d, _outputs(d, 4))
    ok = torch.zeros((256, 128, 128), dtype=torch.int32, device="cuda")    # exactly 16 MiB: accepted
    out = ms.bvn_decompose_static(ok, _outputs(ok, 4))
    torch.cuda.synchronize()
    assert (out.count == 0).all() and (out.status == 0).all()
