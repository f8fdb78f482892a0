"""ctypes access to the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
import this package. The product package never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moesched_oracle.cpp")
_SO = os.path.join(_HERE, "libmoesched_oracle.so")

MODEL_FIELDS = ("bytes_per_token", "link_gbps", "reconfig_ns", "expert_fixed_ns", "expert_ps_per_token",
                "expert_knee_tokens")


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no CUDA involved)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", "-pthread", "-o", _SO, _SRC]
        subprocess.run(cmd, check=True)
    return _SO


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_assignment_max.restype = ctypes.c_int64
    return _lib


def hardware_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def mw_decompose(demand, k_max, tier=1, threads=1, want_residual=True):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    perm = np.zeros((B, k_max, N), np.uint8)
    dur = np.zeros((B, k_max), np.int32)
    count = np.zeros(B, np.int32)
    status = np.zeros(B, np.int32)
    residual = np.zeros_like(d) if want_residual else None
    rc = lib().oracle_mw_decompose(B, N, _p(d), k_max, _p(perm), _p(dur), _p(count), _p(residual),
                                   _p(status), tier, threads)
    if rc != 0:
        raise ValueError("oracle_mw_decompose rejected its arguments")
    return dict(perm=perm, dur=dur, count=count, residual=residual, status=status)


def bvn_decompose(demand, k_max, tier=1, threads=1, want_aug=True):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    perm = np.zeros((B, k_max, N), np.uint8)
    coef = np.zeros((B, k_max), np.int32)
    count = np.zeros(B, np.int32)
    status = np.zeros(B, np.int32)
    aug = np.zeros_like(d) if want_aug else None
    rc = lib().oracle_bvn_decompose(B, N, _p(d), k_max, _p(perm), _p(coef), _p(count), _p(aug),
                                    _p(status), tier, threads)
    if rc != 0:
        raise ValueError("oracle_bvn_decompose rejected its arguments")
    return dict(perm=perm, coef=coef, count=count, aug=aug, status=status)


def schedule_eval(demand, perm, dur, count, model, threads=1):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    perm = np.ascontiguousarray(perm, dtype=np.uint8)
    dur = np.ascontiguousarray(dur, dtype=np.int32)
    count = np.ascontiguousarray(count, dtype=np.int32)
    k_stride = perm.shape[1]
    m = np.array([int(model.get(f, 0)) for f in MODEL_FIELDS], np.int64)
    out = {k: np.zeros(B, np.int64) for k in
           ("makespan_overlap_ns", "makespan_serial_ns", "compute_idle_ns", "link_idle_tokens",
            "unserved_tokens")}
    status = np.zeros(B, np.int32)
    rc = lib().oracle_schedule_eval(B, N, _p(d), k_stride, _p(perm), _p(dur), _p(count), _p(m),
                                    _p(out["makespan_overlap_ns"]), _p(out["makespan_serial_ns"]),
                                    _p(out["compute_idle_ns"]), _p(out["link_idle_tokens"]),
                                    _p(out["unserved_tokens"]), _p(status), threads)
    if rc != 0:
        raise ValueError("oracle_schedule_eval rejected its arguments")
    out["status"] = status
    return out


def schedule_prefix_eval(demand, perm, dur, count, model, threads=1):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    perm = np.ascontiguousarray(perm, dtype=np.uint8)
    dur = np.ascontiguousarray(dur, dtype=np.int32)
    count = np.ascontiguousarray(count, dtype=np.int32)
    K = perm.shape[1]
    m = np.array([int(model.get(f, 0)) for f in MODEL_FIELDS], np.int64)
    po = np.zeros((B, K), np.int64)
    pu = np.zeros((B, K), np.int64)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_schedule_prefix_eval(B, N, _p(d), K, _p(perm), _p(dur), _p(count), _p(m), _p(po), _p(pu),
                                           _p(status), threads)
    if rc != 0:
        raise ValueError("oracle_schedule_prefix_eval rejected its arguments")
    return dict(prefix_overlap_ns=po, prefix_unserved_tokens=pu, status=status)


def schedule_order(demand, perm, dur, count, model, threads=1):
    """Best-of-several order of the matchings on fixed job times (see order_one in the C++ source)."""
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    perm = np.ascontiguousarray(perm, dtype=np.uint8)
    dur = np.ascontiguousarray(dur, dtype=np.int32)
    count = np.ascontiguousarray(count, dtype=np.int32)
    K = perm.shape[1]
    m = np.array([int(model.get(f, 0)) for f in MODEL_FIELDS], np.int64)
    order = np.zeros((B, K), np.int32)
    best = np.zeros(B, np.int64)
    emission = np.zeros(B, np.int64)
    rule = np.zeros(B, np.int32)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_schedule_order(B, N, _p(d), K, _p(perm), _p(dur), _p(count), _p(m), _p(order), _p(best),
                                     _p(emission), _p(rule), _p(status), threads)
    if rc != 0:
        raise ValueError("oracle_schedule_order rejected its arguments")
    return dict(order=order, makespan_ns=best, emission_ns=emission, rule=rule, status=status)


def best_budget(count, prefix_overlap_ns, prefix_unserved_tokens, ns_per_unserved_token):
    count = np.ascontiguousarray(count, dtype=np.int32)
    po = np.ascontiguousarray(prefix_overlap_ns, dtype=np.int64)
    pu = np.ascontiguousarray(prefix_unserved_tokens, dtype=np.int64)
    B, K = po.shape
    best_k = np.zeros(B, np.int32)
    best_cost = np.zeros(B, np.int64)
    rc = lib().oracle_best_budget(B, K, _p(count), _p(po), _p(pu), ctypes.c_int64(int(ns_per_unserved_token)),
                                  _p(best_k), _p(best_cost))
    if rc != 0:
        raise ValueError("oracle_best_budget rejected its arguments")
    return dict(best_k=best_k, best_cost=best_cost)


def ideal_a2a(demand, model):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    m = np.array([int(model.get(f, 0)) for f in MODEL_FIELDS], np.int64)
    comm = np.zeros(B, np.int64)
    mk = np.zeros(B, np.int64)
    status = np.zeros(B, np.int32)
    if lib().oracle_ideal_a2a(B, N, _p(d), _p(m), _p(comm), _p(mk), _p(status)) != 0:
        raise ValueError("oracle_ideal_a2a rejected its arguments")
    return dict(comm_ns=comm, makespan_ns=mk, status=status)


def sinkhorn_scale(demand, iters, smooth, scale_bits, threads=1):
    d = np.ascontiguousarray(demand, dtype=np.int32)
    B, N, _ = d.shape
    scaled = np.zeros((B, N, N), np.float64)
    fixed = np.zeros((B, N, N), np.int32)
    stretch = np.zeros(B, np.float64)
    row_err = np.zeros(B, np.float64)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_sinkhorn_scale(B, N, _p(d), int(iters), ctypes.c_double(smooth), int(scale_bits), _p(scaled),
                                     _p(fixed), _p(stretch), _p(row_err), _p(status), threads)
    if rc != 0:
        raise ValueError("oracle_sinkhorn_scale rejected its arguments")
    return dict(scaled=scaled, fixed=fixed, stretch=stretch, row_err=row_err, status=status)


def bvn_real_decompose(matrix, k_max, tol=1e-12, threads=1):
    """Real-valued Birkhoff-von Neumann decomposition (see bvn_real_one in the C++ source)."""
    a = np.ascontiguousarray(matrix, dtype=np.float64)
    B, N, _ = a.shape
    perm = np.zeros((B, k_max, N), np.uint8)
    lam = np.zeros((B, k_max), np.float64)
    count = np.zeros(B, np.int32)
    total = np.zeros(B, np.float64)
    left = np.zeros(B, np.float64)
    status = np.zeros(B, np.int32)
    rc = lib().oracle_bvn_real_decompose(B, N, _p(a), ctypes.c_double(tol), int(k_max), _p(perm), _p(lam), _p(count),
                                         _p(total), _p(left), _p(status), threads)
    if rc != 0:
        raise ValueError("oracle_bvn_real_decompose rejected its arguments")
    return dict(perm=perm, lam=lam, count=count, sum_lambda=total, max_left=left, status=status)


def sinkhorn_durations(coef, count, stretch, scale_bits):
    coef = np.ascontiguousarray(coef, dtype=np.int32)
    count = np.ascontiguousarray(count, dtype=np.int32)
    stretch = np.ascontiguousarray(stretch, dtype=np.float64)
    B, K = coef.shape
    dur = np.zeros((B, K), np.int32)
    if lib().oracle_sinkhorn_durations(B, K, _p(coef), _p(count), _p(stretch), int(scale_bits), _p(dur)) != 0:
        raise ValueError("oracle_sinkhorn_durations rejected its arguments")
    return dur


def max_weight_perm(W, tier):
    W = np.ascontiguousarray(W, dtype=np.int64)
    N = W.shape[0]
    perm = np.zeros(N, np.int32)
    rc = lib().oracle_max_weight_perm(N, _p(W), _p(perm), tier)
    return perm if rc == 0 else None


def support_perm(A, tier):
    A = np.ascontiguousarray(A, dtype=np.int64)
    N = A.shape[0]
    perm = np.zeros(N, np.int32)
    rc = lib().oracle_support_perm(N, _p(A), _p(perm), tier)
    return perm if rc == 0 else None


def assignment_max(W):
    W = np.ascontiguousarray(W, dtype=np.int64)
    return int(lib().oracle_assignment_max(W.shape[0], _p(W)))


def augment(D):
    D = np.ascontiguousarray(D, dtype=np.int32)
    A = np.zeros(D.shape, np.int64)
    rc = lib().oracle_augment(D.shape[0], _p(D), _p(A))
    return A if rc == 0 else None
