"""Python binding of libmoesched (argument marshalling only).

Every step of the path -- greedy max-weight decomposition (paper Sec. 3.2),
Birkhoff-von Neumann decomposition (Sec. 3.1) and schedule scoring (Sec. 4.1) --
runs in the CUDA kernels behind the C ABI declared in include/moesched.h.
PyTorch is used for device memory and streams only. There is no CPU fallback:
a missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from .workload import DEFAULT_MODEL, PROFILED_MODEL, bvn_capacity  # noqa: F401  (re-exported)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmoesched.so")

ST_OK, ST_TRUNCATED, ST_BAD_INPUT, ST_INTERNAL = 0, 1, -1, -2
WORK_FIELDS = 10
MAX_N = 256


class MoeschedError(RuntimeError):
    pass


class _Model(ctypes.Structure):
    _fields_ = [("bytes_per_token", ctypes.c_int64), ("link_gbps", ctypes.c_int64),
                ("reconfig_ns", ctypes.c_int64), ("expert_fixed_ns", ctypes.c_int64),
                ("expert_ps_per_token", ctypes.c_int64), ("expert_knee_tokens", ctypes.c_int64)]


_lib = None


def _open(path):
    if not os.path.exists(path):
        raise MoeschedError(f"{path} is missing: run `python -m paper_2605_26845_b200.build` "
                            "(there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    lib.moesched_strerror.restype = ctypes.c_char_p
    lib.moesched_status_str.restype = ctypes.c_char_p
    lib.moesched_workspace_bytes.restype = ctypes.c_size_t
    for name in ("moesched_mw_decompose", "moesched_bvn_decompose", "moesched_bvn_decompose_static",
                 "moesched_schedule_eval", "moesched_schedule_prefix_eval", "moesched_ideal_a2a",
                 "moesched_sinkhorn_scale", "moesched_sinkhorn_durations", "moesched_last_cuda_error",
                 "moesched_schedule_order", "moesched_schedule_permute", "moesched_best_budget",
                 "moesched_bvn_real_decompose"):
        getattr(lib, name).restype = ctypes.c_int
    lib.moesched_bvn_scratch_bytes.restype = ctypes.c_size_t
    lib.moesched_order_scratch_bytes.restype = ctypes.c_size_t
    lib.moesched_probe_int_ops.restype = ctypes.c_longlong
    lib.moesched_debug_index_faults.restype = ctypes.c_longlong
    return lib


def load_library():
    """dlopen libmoesched.so (built in-tree by paper_2605_26845_b200/build.py)."""
    global _lib
    if _lib is None:
        _lib = _open(LIB_PATH)
    return _lib


def use_library(path=None):
    """Route every call of this binding through another build of the library, e.g. the checked one
    (libmoesched_checked.so, see build.py); None goes back to the regular library. Returns the path."""
    global _lib
    path = LIB_PATH if path is None else path
    _lib = _open(path)
    return path


def debug_index_faults() -> int:
    """Out-of-range indices the checked build has caught on the current device (-1: no checks compiled in)."""
    return int(load_library().moesched_debug_index_faults())


def _check(rc, what):
    if rc != 0:
        lib = load_library()
        msg = lib.moesched_strerror(rc).decode()
        raise MoeschedError(f"{what}: {msg} (rc={rc}, cuda error {lib.moesched_last_cuda_error()})")


def _dev(t, dtype, what):
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise MoeschedError(f"{what} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype or not t.is_contiguous():
        raise MoeschedError(f"{what} must be contiguous {dtype}")
    return t


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _stream(device):
    return ctypes.c_void_p(torch.cuda.current_stream(device).cuda_stream)


@dataclass
class Schedule:
    """Ordered matchings of a batch: perm [B, k_max, N] uint8 (perm[b, k, i] = destination of
    source i), dur [B, k_max] int32 tokens, count [B], status [B]; extra = residual (greedy) or
    augmented matrix (BvN) if requested; work = per-matrix work counters if requested."""
    perm: torch.Tensor
    dur: torch.Tensor
    count: torch.Tensor
    status: torch.Tensor
    extra: torch.Tensor | None = None
    work: torch.Tensor | None = None


def _new_schedule(demand, k_max, want_extra, want_work):
    B, N, _ = demand.shape
    dev = demand.device
    return Schedule(perm=torch.empty((B, k_max, N), dtype=torch.uint8, device=dev),
                    dur=torch.empty((B, k_max), dtype=torch.int32, device=dev),
                    count=torch.empty(B, dtype=torch.int32, device=dev),
                    status=torch.empty(B, dtype=torch.int32, device=dev),
                    extra=torch.empty_like(demand) if want_extra else None,
                    work=torch.empty((B, WORK_FIELDS), dtype=torch.int64, device=dev) if want_work else None)


def _check_demand(demand):
    demand = _dev(demand, torch.int32, "demand")
    if demand.dim() != 3 or demand.shape[1] != demand.shape[2]:
        raise MoeschedError("demand must have shape [B, N, N]")
    return demand


def mw_decompose(demand, k_max, want_residual=False, want_work=False, out=None) -> Schedule:
    """Greedy max-weight decomposition of every matrix of `demand` [B, N, N] int32 (CUDA)."""
    lib = load_library()
    demand = _check_demand(demand)
    B, N, _ = demand.shape
    dev = demand.device
    if out is None:
        out = _new_schedule(demand, int(k_max), want_residual, want_work)
    with torch.cuda.device(dev):
        rc = lib.moesched_mw_decompose(B, N, _ptr(demand), int(k_max), _ptr(out.perm), _ptr(out.dur),
                                       _ptr(out.count), _ptr(out.extra), _ptr(out.status), _ptr(out.work),
                                       _stream(dev))
    _check(rc, "moesched_mw_decompose")
    return out


def bvn_scratch_bytes(B, N) -> int:
    return int(load_library().moesched_bvn_scratch_bytes(int(B), int(N)))


def workspace_bytes(B, N, k_max) -> int:
    """Device working memory a pass of the whole path can use beyond its inputs and outputs."""
    return int(load_library().moesched_workspace_bytes(int(B), int(N), int(k_max)))


def status_str(status) -> str:
    """Text for one per-matrix status value."""
    return load_library().moesched_status_str(int(status)).decode()


def bvn_decompose(demand, k_max=None, want_aug=False, want_work=False, out=None, scratch=True) -> Schedule:
    """Birkhoff-von Neumann decomposition; k_max defaults to N^2 - 2N + 2 (always enough).

    scratch: True allocates the working buffer of the fast path, a uint8 CUDA tensor of at least
    bvn_scratch_bytes(B, N) bytes is used as given, False / None selects the shared-memory path."""
    lib = load_library()
    demand = _check_demand(demand)
    B, N, _ = demand.shape
    dev = demand.device
    if k_max is None:
        k_max = bvn_capacity(N)
    if out is None:
        out = _new_schedule(demand, int(k_max), want_aug, want_work)
    if scratch is True:
        scratch = torch.empty(max(1, bvn_scratch_bytes(B, N)), dtype=torch.uint8, device=dev)
    elif scratch is False:
        scratch = None
    if scratch is not None:
        _dev(scratch, torch.uint8, "scratch")
        if scratch.numel() < bvn_scratch_bytes(B, N):
            raise MoeschedError("scratch is smaller than bvn_scratch_bytes(B, N)")
    with torch.cuda.device(dev):
        rc = lib.moesched_bvn_decompose(B, N, _ptr(demand), int(k_max), _ptr(out.perm), _ptr(out.dur),
                                        _ptr(out.count), _ptr(out.extra), _ptr(scratch), _ptr(out.status),
                                        _ptr(out.work), _stream(dev))
    _check(rc, "moesched_bvn_decompose")
    return out


STATIC_SCRATCH_BYTES = 16 * 1024 * 1024


def bvn_decompose_static(demand, out: Schedule) -> Schedule:
    """BvN decomposition through the entry point that allocates nothing: for callers that may
    not allocate device memory (a host framework owns the pool, or an allocation would stall a
    latency-critical loop). `out` must be a complete, caller-made Schedule; the working copy sits
    in the library's built-in 16 MiB array, so B * N * roundup(N, 8) * 4 must fit in it. Calls
    that may overlap on one GPU share that array and must be serialised."""
    lib = load_library()
    demand = _check_demand(demand)
    B, N, _ = demand.shape
    dev = demand.device
    with torch.cuda.device(dev):
        rc = lib.moesched_bvn_decompose_static(B, N, _ptr(demand), int(out.perm.shape[1]), _ptr(out.perm),
                                               _ptr(out.dur), _ptr(out.count), _ptr(out.extra),
                                               _ptr(out.status), _ptr(out.work), _stream(dev))
    _check(rc, "moesched_bvn_decompose_static")
    return out


def probe_int_rate(device=None, blocks=148 * 8, iters=20000, reps=3) -> float:
    """Measured integer lane-operations per second of the GPU (add / min / logic mix)."""
    lib = load_library()
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    out = torch.empty(blocks * 256, dtype=torch.int32, device=dev)
    best = 0.0
    with torch.cuda.device(dev):
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ops = lib.moesched_probe_int_ops(blocks, iters, _ptr(out), _stream(dev))
            e1.record()
            if ops < 0:
                _check(int(ops), "moesched_probe_int_ops")
            e1.synchronize()
            best = max(best, ops / (e0.elapsed_time(e1) * 1e-3))
    return best


def sinkhorn_scale(demand, iters=20, smooth=0.5, scale_bits=20, out=None) -> dict:
    """Sinkhorn-Knopp scaling of a batch (paper Sec. 3.1). Returns scaled [B, N, N] float64, fixed
    [B, N, N] int32 (= round(scaled * 2^scale_bits), the input of bvn_decompose), stretch [B], row_err [B]
    float64 and status [B]; `out` may hand back the dict of an earlier call of the same shape for reuse."""
    demand = _check_demand(demand)
    B, N, _ = demand.shape
    dev = demand.device
    if out is None:
        out = dict(scaled=torch.empty((B, N, N), dtype=torch.float64, device=dev),
                   fixed=torch.empty((B, N, N), dtype=torch.int32, device=dev),
                   stretch=torch.empty(B, dtype=torch.float64, device=dev),
                   row_err=torch.empty(B, dtype=torch.float64, device=dev),
                   status=torch.empty(B, dtype=torch.int32, device=dev))
    else:
        _dev(out["scaled"], torch.float64, "out['scaled']")
        _dev(out["fixed"], torch.int32, "out['fixed']")
        if out["scaled"].shape != demand.shape or out["fixed"].shape != demand.shape:
            raise MoeschedError("out has the wrong shape")
    rc = load_library().moesched_sinkhorn_scale(B, N, _ptr(demand), int(iters), ctypes.c_double(float(smooth)),
                                                int(scale_bits), _ptr(out["scaled"]), _ptr(out["fixed"]),
                                                _ptr(out["stretch"]), _ptr(out["row_err"]), _ptr(out["status"]),
                                                _stream(dev))
    _check(rc, "moesched_sinkhorn_scale")
    return out


def sinkhorn_durations(coef, count, stretch, scale_bits=20, out=None) -> torch.Tensor:
    """Token length of each matching of a decomposition of sinkhorn_scale(...)["fixed"]:
    ceil(coef * stretch / 2^scale_bits) for the first count[b] matchings of every schedule."""
    coef = _dev(coef, torch.int32, "coef")
    count = _dev(count, torch.int32, "count")
    stretch = _dev(stretch, torch.float64, "stretch")
    B, K = coef.shape
    if out is None:
        out = torch.zeros_like(coef)
    rc = load_library().moesched_sinkhorn_durations(B, K, _ptr(coef), _ptr(count), _ptr(stretch), int(scale_bits),
                                                    _ptr(_dev(out, torch.int32, "out")), _stream(coef.device))
    _check(rc, "moesched_sinkhorn_durations")
    return out


def bvn_real_decompose(matrix, k_max=None, tol=1e-12) -> dict:
    """Real-valued Birkhoff-von Neumann decomposition A = sum_k lambda_k P_k (paper Sec. 3.1) of [B, N, N]
    float64 matrices, e.g. sinkhorn_scale(...)["scaled"]. Returns perm [B, k_max, N] uint8, lam [B, k_max]
    float64, count, sum_lambda, max_left (largest entry remaining) and status [B]."""
    lib = load_library()
    matrix = _dev(matrix, torch.float64, "matrix")
    if matrix.dim() != 3 or matrix.shape[1] != matrix.shape[2]:
        raise MoeschedError("matrix must have shape [B, N, N]")
    B, N, _ = matrix.shape
    dev = matrix.device
    k_max = bvn_capacity(N) if k_max is None else int(k_max)
    out = dict(perm=torch.empty((B, k_max, N), dtype=torch.uint8, device=dev),
               lam=torch.empty((B, k_max), dtype=torch.float64, device=dev),
               count=torch.empty(B, dtype=torch.int32, device=dev),
               sum_lambda=torch.empty(B, dtype=torch.float64, device=dev),
               max_left=torch.empty(B, dtype=torch.float64, device=dev),
               status=torch.empty(B, dtype=torch.int32, device=dev))
    scratch = torch.empty(max(1, B * N * ((N + 7) // 8 * 8)), dtype=torch.float64, device=dev)
    with torch.cuda.device(dev):
        rc = lib.moesched_bvn_real_decompose(B, N, _ptr(matrix), ctypes.c_double(float(tol)), k_max, _ptr(out["perm"]),
                                             _ptr(out["lam"]), _ptr(out["count"]), _ptr(out["sum_lambda"]),
                                             _ptr(out["max_left"]), _ptr(scratch), _ptr(out["status"]), _stream(dev))
    _check(rc, "moesched_bvn_real_decompose")
    return out


def _model(model):
    return _Model(**{k: int(v) for k, v in (model or DEFAULT_MODEL).items()})


def ideal_a2a(demand, model=None) -> dict:
    """Idealised congestion-free all-to-all of every matrix: 'comm_ns' (one exchange at line rate of
    the busiest port), 'makespan_ns' (dispatch + compute + combine, run to completion), 'status'."""
    lib = load_library()
    demand = _check_demand(demand)
    B, N, _ = demand.shape
    dev = demand.device
    m = _model(model)
    out = torch.empty((2, B), dtype=torch.int64, device=dev)
    status = torch.empty(B, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        rc = lib.moesched_ideal_a2a(B, N, _ptr(demand), ctypes.byref(m), _ptr(out[0]), _ptr(out[1]), _ptr(status),
                                    _stream(dev))
    _check(rc, "moesched_ideal_a2a")
    return {"comm_ns": out[0], "makespan_ns": out[1], "status": status}


SCORE_FIELDS = ("makespan_overlap_ns", "makespan_serial_ns", "compute_idle_ns", "link_idle_tokens",
                "unserved_tokens")


def schedule_eval(demand, perm, dur, count, model=None, out=None, status=None, prefix=False) -> dict:
    """Score schedules under the dispatch-compute-combine model. Returns a dict of [B] int64
    tensors (SCORE_FIELDS) plus 'status' [B] int32; `out` may supply a [5, B] int64 tensor and
    `status` a [B] int32 tensor. With prefix=True the dict also holds 'prefix_overlap_ns' and
    'prefix_unserved_tokens', [B, k_stride] int64: the scores of the schedule cut after each
    matching (-1 beyond count)."""
    lib = load_library()
    demand = _dev(demand, torch.int32, "demand")
    perm = _dev(perm, torch.uint8, "perm")
    dur = _dev(dur, torch.int32, "dur")
    count = _dev(count, torch.int32, "count")
    B, N, _ = demand.shape
    if perm.dim() != 3 or perm.shape[0] != B or perm.shape[2] != N or dur.shape != perm.shape[:2]:
        raise MoeschedError("perm must be [B, k_stride, N] and dur [B, k_stride]")
    m = _model(model)
    dev = demand.device
    scores = out if out is not None else torch.empty((5, B), dtype=torch.int64, device=dev)
    if status is None:
        status = torch.empty(B, dtype=torch.int32, device=dev)
    K = int(perm.shape[1])
    pre = torch.empty((2, B, K), dtype=torch.int64, device=dev) if prefix else None
    with torch.cuda.device(dev):
        args = (B, N, _ptr(demand), K, _ptr(perm), _ptr(dur), _ptr(count), ctypes.byref(m), _ptr(scores[0]),
                _ptr(scores[1]), _ptr(scores[2]), _ptr(scores[3]), _ptr(scores[4]), _ptr(status))
        if prefix:
            rc = lib.moesched_schedule_prefix_eval(*args, _ptr(pre[0]), _ptr(pre[1]), _stream(dev))
        else:
            rc = lib.moesched_schedule_eval(*args, _stream(dev))
    _check(rc, "moesched_schedule_eval")
    res = {name: scores[i] for i, name in enumerate(SCORE_FIELDS)}
    if prefix:
        res["prefix_overlap_ns"], res["prefix_unserved_tokens"] = pre[0], pre[1]
    res["status"] = status
    return res


ORDER_MAX_K = 1024


def schedule_order(demand, perm, dur, count, model=None) -> dict:
    """Best of five orders of the matchings on the job times of the emission-order replay (paper
    Sec. 3.3). Returns 'order' [B, k_stride] int32 (position -> original index, -1 beyond count),
    'makespan_ns', 'emission_ns' [B] int64, 'rule', 'status' [B] int32."""
    lib = load_library()
    demand = _check_demand(demand)
    perm = _dev(perm, torch.uint8, "perm")
    dur = _dev(dur, torch.int32, "dur")
    count = _dev(count, torch.int32, "count")
    B, N, _ = demand.shape
    K = int(perm.shape[1])
    if perm.dim() != 3 or perm.shape[0] != B or perm.shape[2] != N or dur.shape != perm.shape[:2]:
        raise MoeschedError("perm must be [B, k_stride, N] and dur [B, k_stride]")
    dev = demand.device
    m = _model(model)
    order = torch.empty((B, K), dtype=torch.int32, device=dev)
    times = torch.empty((2, B), dtype=torch.int64, device=dev)
    small = torch.empty((2, B), dtype=torch.int32, device=dev)
    scratch = torch.empty(max(8, int(lib.moesched_order_scratch_bytes(B, K))), dtype=torch.uint8, device=dev)
    with torch.cuda.device(dev):
        rc = lib.moesched_schedule_order(B, N, _ptr(demand), K, _ptr(perm), _ptr(dur), _ptr(count), ctypes.byref(m),
                                         _ptr(order), _ptr(times[0]), _ptr(times[1]), _ptr(small[0]), _ptr(small[1]),
                                         _ptr(scratch), _stream(dev))
    _check(rc, "moesched_schedule_order")
    return {"order": order, "makespan_ns": times[0], "emission_ns": times[1], "rule": small[0], "status": small[1]}


def schedule_permute(perm, dur, order):
    """(perm, dur) with the matchings in the given order; positions whose order entry is -1 hold zeros."""
    lib = load_library()
    perm = _dev(perm, torch.uint8, "perm")
    dur = _dev(dur, torch.int32, "dur")
    order = _dev(order, torch.int32, "order")
    B, K, N = perm.shape
    perm_out, dur_out = torch.zeros_like(perm), torch.zeros_like(dur)
    with torch.cuda.device(perm.device):
        rc = lib.moesched_schedule_permute(B, N, K, _ptr(perm), _ptr(dur), _ptr(order), _ptr(perm_out), _ptr(dur_out),
                                           _stream(perm.device))
    _check(rc, "moesched_schedule_permute")
    return perm_out, dur_out


def best_budget(count, prefix_overlap_ns, prefix_unserved_tokens, ns_per_unserved_token) -> dict:
    """Number of matchings (1..count) minimising prefix makespan + price * unserved tokens."""
    lib = load_library()
    count = _dev(count, torch.int32, "count")
    po = _dev(prefix_overlap_ns, torch.int64, "prefix_overlap_ns")
    pu = _dev(prefix_unserved_tokens, torch.int64, "prefix_unserved_tokens")
    B, K = po.shape
    best_k = torch.empty(B, dtype=torch.int32, device=po.device)
    best_cost = torch.empty(B, dtype=torch.int64, device=po.device)
    with torch.cuda.device(po.device):
        rc = lib.moesched_best_budget(B, K, _ptr(count), _ptr(po), _ptr(pu), ctypes.c_int64(int(ns_per_unserved_token)),
                                      _ptr(best_k), _ptr(best_cost), _stream(po.device))
    _check(rc, "moesched_best_budget")
    return {"best_k": best_k, "best_cost": best_cost}


class Path:
    """The whole path for batches of one shape: greedy max-weight and BvN decomposition, both scored.

    All buffers (schedules, scores, BvN scratch) are allocated once here. The two decompositions do not
    depend on each other: run() forks them onto two streams -- BvN and its scoring first, greedy and its
    scoring second -- and joins them back into the caller's current stream, so that the greedy warps fill
    the SMs as the BvN matrices finish at different times (measured on a B200, headline workload: 70 ms
    per step against 77 ms on one stream). run(overlap=False) keeps everything on the current stream."""

    def __init__(self, B, N, k_mw, k_bvn=None, device=None, want_work=False):
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.device, self.B, self.N = dev, B, N
        self.k_mw, self.k_bvn = int(k_mw), int(bvn_capacity(N) if k_bvn is None else k_bvn)

        def sched(k):
            return Schedule(perm=torch.empty((B, k, N), dtype=torch.uint8, device=dev),
                            dur=torch.empty((B, k), dtype=torch.int32, device=dev),
                            count=torch.empty(B, dtype=torch.int32, device=dev),
                            status=torch.empty(B, dtype=torch.int32, device=dev),
                            work=torch.zeros((B, WORK_FIELDS), dtype=torch.int64, device=dev) if want_work else None)

        self.mw, self.bvn = sched(self.k_mw), sched(self.k_bvn)
        self.score_mw = torch.empty((5, B), dtype=torch.int64, device=dev)
        self.score_bvn = torch.empty((5, B), dtype=torch.int64, device=dev)
        self.eval_status_mw = torch.empty(B, dtype=torch.int32, device=dev)
        self.eval_status_bvn = torch.empty(B, dtype=torch.int32, device=dev)
        self.scratch = torch.empty(max(1, bvn_scratch_bytes(B, N)), dtype=torch.uint8, device=dev)
        self._side = (torch.cuda.Stream(dev), torch.cuda.Stream(dev))
        self._fork = torch.cuda.Event()
        self._join = (torch.cuda.Event(), torch.cuda.Event())

    def outputs(self):
        return [self.mw.perm, self.mw.dur, self.mw.count, self.mw.status, self.bvn.perm, self.bvn.dur,
                self.bvn.count, self.bvn.status, self.score_mw, self.score_bvn]

    def _greedy(self, demand, model):
        mw_decompose(demand, self.k_mw, out=self.mw)
        schedule_eval(demand, self.mw.perm, self.mw.dur, self.mw.count, model, out=self.score_mw,
                      status=self.eval_status_mw)

    def _bvn(self, demand, model):
        bvn_decompose(demand, self.k_bvn, out=self.bvn, scratch=self.scratch)
        schedule_eval(demand, self.bvn.perm, self.bvn.dur, self.bvn.count, model, out=self.score_bvn,
                      status=self.eval_status_bvn)

    def run_graph(self, demand, model=None):
        """The same launches replayed from a CUDA graph: for small matrices the step is a handful of
        microsecond kernels and the cost of launching them one by one dominates. The graph is captured
        on first use and again whenever the demand tensor's address or the model changes."""
        key = (demand.data_ptr(), tuple(sorted((model or DEFAULT_MODEL).items())))
        if getattr(self, "_graph_key", None) != key:
            self.run(demand, model)                      # first-use set-up outside the capture
            torch.cuda.current_stream(self.device).synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                self.run(demand, model)
            self._graph, self._graph_key, self._graph_demand = graph, key, demand
        self._graph.replay()
        return self

    def run(self, demand, model=None, overlap=True):
        """Enqueue the four kernels; results are ready when the caller's current stream reaches this point."""
        if not overlap:
            self._greedy(demand, model)
            self._bvn(demand, model)
            return self
        cur = torch.cuda.current_stream(self.device)
        self._fork.record(cur)
        for side, work, done in ((self._side[0], self._bvn, self._join[0]), (self._side[1], self._greedy, self._join[1])):
            side.wait_event(self._fork)
            with torch.cuda.stream(side):
                work(demand, model)
                done.record(side)
        for done in self._join:
            cur.wait_event(done)
        return self


class HostPipeline:
    """The whole path for batches that live in host memory, double-buffered.

    submit() enqueues, for one batch: the copy of the demand from (pinned) host memory to the device
    on an upload stream, the four kernels on a compute stream, and the copy of all schedules and scores
    back to pinned host memory on a download stream. With two slots the download of one batch and the
    upload of the next overlap the kernels of the batch in between, so a stream of batches runs at the
    speed of the slowest of the three stages instead of their sum."""

    def __init__(self, B, N, k_mw, k_bvn=None, device=None, slots=2):
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
        self.device, self.slots = dev, slots
        self.paths = [Path(B, N, k_mw, k_bvn, device=dev) for _ in range(slots)]
        self.d_in = [torch.empty((B, N, N), dtype=torch.int32, device=dev) for _ in range(slots)]
        self.h_out = [[torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in p.outputs()] for p in self.paths]
        self.up, self.compute, self.down = (torch.cuda.Stream(dev) for _ in range(3))
        self.ev_in = [torch.cuda.Event() for _ in range(slots)]
        self.ev_done = [torch.cuda.Event() for _ in range(slots)]
        self.ev_out = [torch.cuda.Event() for _ in range(slots)]
        self._next = 0
        self.h2d_bytes = B * N * N * 4
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.paths[0].outputs())

    def submit(self, demand_host, model=None) -> int:
        """Enqueue one batch (a [B, N, N] int32 CPU tensor, ideally pinned); returns its slot."""
        s = self._next
        self._next = (s + 1) % self.slots
        self.ev_out[s].synchronize()            # the slot's previous results must have left the device
        self.up.wait_event(self.ev_done[s])     # and its previous kernels must be done with the input
        with torch.cuda.stream(self.up):
            self.d_in[s].copy_(demand_host, non_blocking=True)
            self.ev_in[s].record(self.up)
        self.compute.wait_event(self.ev_in[s])
        with torch.cuda.stream(self.compute):
            self.paths[s].run(self.d_in[s], model)
            self.ev_done[s].record(self.compute)
        self.down.wait_event(self.ev_done[s])
        with torch.cuda.stream(self.down):
            for h, t in zip(self.h_out[s], self.paths[s].outputs()):
                h.copy_(t, non_blocking=True)
            self.ev_out[s].record(self.down)
        return s

    def result(self, slot):
        """Block until the slot's results are in host memory; returns the pinned host tensors in the
        order of Path.outputs(). They are overwritten when the slot is submitted again."""
        self.ev_out[slot].synchronize()
        return self.h_out[slot]
