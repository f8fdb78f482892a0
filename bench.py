"""Benchmark: demand-matrix decompositions per second on the headline workload.

One step = one pass of the whole path over one batch of B demand matrices:
greedy max-weight decomposition (k_max = 64), Birkhoff-von Neumann decomposition
(capacity N^2-2N+2) and the scoring of both schedules -- four kernel launches.
A "decomposition" is one demand matrix taken through all of it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched through torch.distributed.run) every rank processes its own
B matrices; there is no exchange step, so no collective touches the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2605_26845_b200.workload import CONFIGS, DEFAULT_MODEL, SEED, bvn_capacity, make_demand  # noqa: E402

METRIC = "demand-matrix decompositions/sec at N=64 (greedy+BvN)"
UNIT = "decompositions/s"
CFG = 3        # the headline workload; --config selects another of the five
K_MW = 64      # greedy budget = the largest k_max of the configuration
FALLBACK_HBM_GBS = 6650.0
SINKHORN_ITERS = 20


def metric_name():
    return METRIC.replace("N=64", f"N={CONFIGS[CFG]['N']}")


def select_config(cfg):
    global CFG, K_MW
    CFG = cfg
    K_MW = max(CONFIGS[cfg]["k_max"])


# Issue-rate ceiling for plain integer work: 148 SMs x 4 warp schedulers x 32 lanes, one
# instruction per scheduler per clock, at the SM clock sampled during the run.
ALU_LANES_PER_CLK = 148 * 4 * 32


def workload_name(B):
    c = CONFIGS[CFG]
    skew = (f"Zipf s={c['s']}" + (" reshuffled per matrix" if c.get("reshuffle") else "")) if c["kind"] == "zipf" \
        else f"Dirichlet({c['alpha']}) per rank, {int(100 * c['hot_prob'])}% hot experts"
    if "allowed_prob" in c:
        skew += f", {int(100 * (1 - c['allowed_prob']))}% of destinations closed per rank"
    return (f"config {CFG}: N={c['N']}, B={B}, {c['tokens']} tokens/rank, {c['experts']} experts top-{c['top_k']}, "
            f"{skew}; greedy k_max={K_MW} + BvN (capacity {bvn_capacity(c['N'])}), both scored")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.proc = None

    def __enter__(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *exc):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v == "Active":
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS, "sm_max_mhz": 1965.0}, "fallback"


def captured_traffic(name):
    """DRAM bytes per launch from the committed ncu capture, or None once the kernel's source has
    changed since the counters were taken."""
    import hashlib
    src = {"bvn_decompose": "bvn_kernel.cu", "mw_decompose": "mw_kernel.cu", "schedule_eval(bvn)": "eval_kernel.cu"}
    path = os.path.join(ROOT, "profiles", "dram_traffic_config3.txt")
    if name not in src or not os.path.exists(path):
        return None
    csrc = os.path.join(ROOT, "paper_2605_26845_b200", "csrc")
    h = hashlib.sha256()
    for f in ("common.cuh", src[name]):
        with open(os.path.join(csrc, f), "rb") as fh:
            h.update(fh.read())
    for line in open(path):
        parts = line.split()
        if len(parts) == 3 and parts[0] == name:
            return int(parts[1]) if parts[2] == h.hexdigest()[:16] else None
    return None


def algorithmic_ops(work_mw, work_bvn, N):
    """Integer lane-operations of the DATA-PARALLEL formulation the kernels run, from their work counters:
    a search level is taken by all lanes over all mask words (4 N W), a column scan costs 6 N, and so on.
    This counts what a lane-parallel machine has to issue for the method, not what a scalar one would."""
    W = (N + 31) // 32
    mw = (6 * N * work_mw[:, 0] + 4 * work_mw[:, 1] + 4 * N * work_mw[:, 2] + 4 * N * W * work_mw[:, 4]
          + 6 * N * work_mw[:, 5] + 4 * N * work_mw[:, 6] + 4 * N * work_mw[:, 3])
    bvn = (4 * N * W * work_bvn[:, 0] + 4 * work_bvn[:, 1] + 4 * N * W * work_bvn[:, 4] + 6 * N * work_bvn[:, 5]
           + 6 * N * work_bvn[:, 6] + 4 * N * work_bvn[:, 3])
    return float(mw.sum()), float(bvn.sum())


def scalar_model_ops(work_mw, work_bvn, N):
    """Integer operations of the method itself under the scalar cost model: per scanned column an add
    pair, a min-update and a compare-select (4 N per scan S), 2 N per dual update U, N/32 word
    operations per frontier row L popped by a canonicalisation search, 3 N per matching K for serve
    and emit; Birkhoff: 2 N per augmenting-path step, the same search and emit terms, 4 N^2 once for
    the sums and the padding. Counters: greedy S = field 0, U = field 1 (one dual update per
    augmentation), L = field 8, K = field 6; Birkhoff path steps = field 1, L = field 8, K = field 6."""
    mw = 4 * N * work_mw[:, 0] + 2 * N * work_mw[:, 1] + (N / 32) * work_mw[:, 8] + 3 * N * work_mw[:, 6]
    bvn = 2 * N * work_bvn[:, 1] + (N / 32) * work_bvn[:, 8] + 3 * N * work_bvn[:, 6] + 4 * N * N
    return float(mw.sum()), float(bvn.sum())


WORK_NAMES_MW = ("column_scans", "augmentations", "rows_bid", "searches", "search_levels", "rotation_steps",
                 "matchings", "rows_matched_on_tight_edges", "frontier_pops", "settled_groups")
WORK_NAMES_BVN = ("repair_levels", "repair_path_steps", "canonical_repairs", "searches", "search_levels",
                  "rotation_steps", "matchings", "rows_skipped_as_prefix", "frontier_pops", "repair_fallbacks")


def per_matching(work, names):
    k = max(1.0, float(work[:, 6].sum()))
    return {n: float(work[:, i].sum()) / k for i, n in enumerate(names) if n not in ("unused", "matchings")}


def rank_demand(rank, B):
    """Every rank works on its own B matrices (weak scaling): same recipe, rank-specific seed."""
    return make_demand(CFG, B, seed=SEED + rank)


def max_over_ranks(values, device, world):
    """Element-wise maximum of per-rank timings (the slowest rank defines the step)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_value(world, B, steps, total_ms):
    """Whole-job throughput: all ranks' matrices over the slowest rank's time."""
    return world * B * steps / (total_ms * 1e-3)


def oracle_rate(D, threads, k_bvn):
    """Whole path on the CPU checker: matrices per second (wall clock)."""
    import oracle
    t0 = time.perf_counter()
    g = oracle.mw_decompose(D, K_MW, threads=threads, want_residual=False)
    v = oracle.bvn_decompose(D, k_bvn, threads=threads, want_aug=False)
    oracle.schedule_eval(D, g["perm"], g["dur"], g["count"], DEFAULT_MODEL, threads=threads)
    oracle.schedule_eval(D, v["perm"], v["coef"], v["count"], DEFAULT_MODEL, threads=threads)
    return D.shape[0] / (time.perf_counter() - t0)


def run_reference(args, rank):
    """The CPU checker as it stands, on the host cores, a bounded sample per step."""
    if rank != 0:
        return
    import oracle
    oracle.build()
    threads = oracle.hardware_threads()
    N = CONFIGS[CFG]["N"]
    sample = max(threads, 16) if N <= 64 else threads
    D = make_demand(CFG, sample)
    cap = bvn_capacity(N) if N <= 64 else min(bvn_capacity(N), 400)
    for _ in range(args.warmup):
        oracle_rate(D[:threads], threads, cap)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_rate(D, threads, cap)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    what = f"first {sample} matrices of the workload per step" + (
        "" if N <= 64 else " with the BvN budget cut to 400 matchings")
    print(json.dumps({
        "impl": "reference", "metric": metric_name(), "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int32", "data": "synthetic",
        "config": {"workload": workload_name(CONFIGS[CFG]["B"]), "sample": what},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=None, help="matrices per GPU (default: the configuration's B)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="replay the step from a CUDA graph (pays off when the kernels take microseconds)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="keep greedy and BvN on one stream instead of forking them onto two")
    ap.add_argument("--sweep", action="store_true",
                    help="also time the greedy decomposition at every budget of the configuration (rates_by_k_max)")
    ap.add_argument("--config", type=int, default=3, choices=sorted(CONFIGS),
                    help="workload configuration (default 3: N=64, the one the metric is quoted on)")
    args = ap.parse_args()
    select_config(args.config)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist

    import paper_2605_26845_b200 as ms

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    ms.load_library()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    cfg = CONFIGS[CFG]
    N = cfg["N"]
    B = args.batch or cfg["B"]
    cap = bvn_capacity(N)
    warm = max(args.warmup, 3)
    D_host = rank_demand(rank, B)
    dev = torch.device("cuda", local_rank)
    d = torch.from_numpy(D_host).to(dev)
    stream = torch.cuda.current_stream()

    path = ms.Path(B, N, K_MW, cap, device=dev)
    mw, bv = path.mw, path.bvn
    score_mw, score_bv, scratch = path.score_mw, path.score_bvn, path.scratch
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)

    names = ["mw_decompose", "schedule_eval(mw)", "bvn_decompose", "schedule_eval(bvn)"]

    def step(events=None):
        """The whole path as a user runs it (ms.Path): greedy and BvN forked on two streams, joined."""
        if events is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
        if args.graph:
            path.run_graph(d, DEFAULT_MODEL)
        else:
            path.run(d, DEFAULT_MODEL, overlap=not args.no_overlap)
        if events is not None:
            e1.record(stream)
            events.append((e0, e1))

    def serial_step(events=None):
        """The same four launches one after the other on one stream: per-kernel durations."""
        marks = [torch.cuda.Event(enable_timing=True) for _ in range(5)] if events is not None else None
        if marks: marks[0].record(stream)
        ms.mw_decompose(d, K_MW, out=mw)
        if marks: marks[1].record(stream)
        ms.schedule_eval(d, mw.perm, mw.dur, mw.count, DEFAULT_MODEL, out=score_mw)
        if marks: marks[2].record(stream)
        ms.bvn_decompose(d, cap, out=bv, scratch=scratch)
        if marks: marks[3].record(stream)
        ms.schedule_eval(d, bv.perm, bv.dur, bv.count, DEFAULT_MODEL, out=score_bv)
        if marks:
            marks[4].record(stream)
            events.append(marks)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warm):
        step()
    barrier()

    # ---- device-resident timing: K steps, L2 flushed (untimed) between steps ----
    events = []
    with ClockSampler(local_rank) as clocks:
        barrier()
        for _ in range(args.steps):
            flush.fill_(1)
            step(events)
        barrier()
    total_ms = sum(e0.elapsed_time(e1) for e0, e1 in events)

    # ---- per-kernel durations (for the roofline): the same launches, serial, same flush ----
    kev = []
    for _ in range(args.steps):
        flush.fill_(1)
        serial_step(kev)
    barrier()
    per_kernel = np.zeros(4)
    for marks in kev:
        for i in range(4):
            per_kernel[i] += marks[i].elapsed_time(marks[i + 1])
    per_kernel /= args.steps

    # ---- the all-to-all yardstick (not part of the step): one streaming pass over the demand ----
    a2a_ms = []
    for _ in range(5):
        flush.fill_(1)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        ms.ideal_a2a(d, DEFAULT_MODEL)
        a1.record(stream)
        a1.synchronize()
        a2a_ms.append(a0.elapsed_time(a1))
    a2a_ms = float(np.median(a2a_ms))

    # ---- Sinkhorn-Knopp scaling (the paper's preprocessing for BvN; not part of the step either) ----
    sk_ms = []
    sk = ms.sinkhorn_scale(d, SINKHORN_ITERS, 0.5, 20)          # allocates the outputs once, untimed
    for _ in range(3):
        flush.fill_(1)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        ms.sinkhorn_scale(d, SINKHORN_ITERS, 0.5, 20, out=sk)
        a1.record(stream)
        a1.synchronize()
        sk_ms.append(a0.elapsed_time(a1))
    sk_ms = float(np.median(sk_ms))
    sk_ok = bool((sk["status"] == 0).all())
    del sk

    # ---- order of the matchings (not part of the step): best of five orders of the greedy schedule ----
    compute_bound = dict(DEFAULT_MODEL, expert_ps_per_token=400_000)     # an expert token costs more than its transfer
    ordering = {}
    if K_MW <= ms.ORDER_MAX_K:
        fixed_list = cfg.get("expert_fixed_ns", (DEFAULT_MODEL["expert_fixed_ns"],))
        models = [("fixed_%dus" % (f // 1000), dict(DEFAULT_MODEL, expert_fixed_ns=f)) for f in fixed_list]
        models.append(("compute_bound_400ns_per_token", compute_bound))
        for name, model in models:
            ms.schedule_order(d, mw.perm, mw.dur, mw.count, model)          # allocations and first-use set-up
            flush.fill_(1)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            od = ms.schedule_order(d, mw.perm, mw.dur, mw.count, model)
            a1.record(stream)
            a1.synchronize()
            gain = ((od["emission_ns"] - od["makespan_ns"]).double() / od["emission_ns"].double().clamp(min=1)).mean()
            ordering[name] = {"ms": a0.elapsed_time(a1), "mean_makespan_gain_frac": float(gain),
                              "schedules_reordered_frac": float((od["rule"] != 0).double().mean())}

    # ---- greedy at every budget of the configuration (--sweep), scored ----
    rates_by_k = {}
    if args.sweep:
        for kb in cfg["k_max"]:
            sch = ms._new_schedule(d, kb, False, False)
            ts = []
            for _ in range(3):
                flush.fill_(1)
                a0, a1, a2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                a0.record(stream)
                ms.mw_decompose(d, kb, out=sch)
                a1.record(stream)
                sc = ms.schedule_eval(d, sch.perm, sch.dur, sch.count, DEFAULT_MODEL)
                a2.record(stream)
                a2.synchronize()
                ts.append((a0.elapsed_time(a1), a1.elapsed_time(a2)))
            t_mw, t_ev = (float(np.median([t[i] for t in ts])) for i in (0, 1))
            entry = {"greedy_ms": t_mw, "scoring_ms": t_ev, "greedy_per_s": B / (t_mw * 1e-3),
                     "mean_unserved_frac": float((sc["unserved_tokens"].double() / d.sum((1, 2)).double()).mean()),
                     "mean_makespan_overlap_us": float(sc["makespan_overlap_ns"].double().mean()) / 1e3}
            for f in cfg.get("expert_fixed_ns", ()):
                sf = ms.schedule_eval(d, sch.perm, sch.dur, sch.count, dict(DEFAULT_MODEL, expert_fixed_ns=f))
                entry["mean_makespan_overlap_us_fixed_%dus" % (f // 1000)] = \
                    float(sf["makespan_overlap_ns"].double().mean()) / 1e3
            rates_by_k[str(kb)] = entry
            del sch

    # ---- end to end: pinned host demand in, schedules and scores back to pinned host memory, every step;
    # the public double-buffered runner overlaps one step's copies with the next step's kernels ----
    h_in = torch.from_numpy(D_host).pin_memory()
    pipe = ms.HostPipeline(B, N, K_MW, cap, device=dev)
    h2d, d2h = pipe.h2d_bytes, pipe.d2h_bytes
    for _ in range(2):
        pipe.result(pipe.submit(h_in, DEFAULT_MODEL))
    barrier()
    e2e_steps = max(10, args.steps)      # enough batches that filling and draining the pipeline do not dominate
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(pipe.up)
    last = 0
    for _ in range(e2e_steps):
        last = pipe.submit(h_in, DEFAULT_MODEL)
    pipe.result(last)
    e1.record(pipe.down)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ok = bool((pipe.h_out[last][2] == mw.count.cpu()).all() and (pipe.h_out[last][6] == bv.count.cpu()).all())

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dev, world)

    ok = bool((mw.status >= 0).all() and (bv.status == 0).all())
    # the kernels' work counters (for the algorithmic-operation count) come from one more, untimed pass:
    # the timed steps run the kernels without them
    wk = torch.zeros((2, B, ms.WORK_FIELDS), dtype=torch.int64, device=dev)
    ms.mw_decompose(d, K_MW, out=ms.Schedule(mw.perm, mw.dur, mw.count, mw.status, work=wk[0]))
    ms.bvn_decompose(d, cap, out=ms.Schedule(bv.perm, bv.dur, bv.count, bv.status, work=wk[1]), scratch=scratch)
    barrier()
    work_mw = wk[0].cpu().numpy().astype(np.float64)
    work_bv = wk[1].cpu().numpy().astype(np.float64)

    if rank == 0:
        value = aggregate_value(world, B, args.steps, total_ms)
        ck = clocks.summary()
        peaks, peak_kind = measured_peaks()
        sm_mhz = ck["sm_mhz"] or peaks.get("sm_max_mhz", 1965.0)
        ops_mw, ops_bvn = algorithmic_ops(work_mw, work_bv, N)
        sc_mw, sc_bvn = scalar_model_ops(work_mw, work_bv, N)
        dom = int(np.argmax(per_kernel))
        dom_ops = ops_bvn if dom == 2 else ops_mw
        dom_scalar = sc_bvn if dom == 2 else sc_mw
        alu_peak = ALU_LANES_PER_CLK * sm_mhz * 1e6 / 1e9          # G lane-ops/s at the sampled clock
        alu_measured = ms.probe_int_rate(dev) / 1e9                 # add / min / logic mix, measured now
        achieved_par = dom_ops / (per_kernel[dom] * 1e-3) / 1e9
        achieved = dom_scalar / (per_kernel[dom] * 1e-3) / 1e9
        other = 0 if dom == 2 else 2
        other_scalar = sc_mw if dom == 2 else sc_bvn
        other_par = ops_mw if dom == 2 else ops_bvn
        k_bv = float(bv.count.double().mean())
        k_mw = float(mw.count.double().mean())
        bytes_bvn = B * (4 * N * N + k_bv * (N + 4) + 8)
        out = {
            "metric": metric_name(), "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "int32", "data": "synthetic",
            "config": {"workload": workload_name(B), "l2": "flushed between timed steps (256 MiB write, untimed)",
                       "matchings_per_matrix": {"greedy": k_mw, "bvn": k_bv}, "all_status_ok": ok,
                       "streams": "one" if args.no_overlap else "greedy and BvN forked on two streams, joined",
                       "launch": "CUDA graph replay" if args.graph else "direct",
                       "seed": SEED},
            "kernels_ms": {n: float(t) for n, t in zip(names, per_kernel)},
            "kernels_ms_note": "per-kernel events from a second, identical serial pass",
            "rates": {"greedy_per_s": B / (per_kernel[0] * 1e-3), "bvn_per_s": B / (per_kernel[2] * 1e-3)},
            # frac: the method's own integer operations (scalar cost model, see scalar_model_ops) over the
            # issue-rate peak; frac_parallel_formulation: the lane-operations of the data-parallel formulation
            # (algorithmic_ops: a search level costs all lanes over all mask words, whether or not a lane's
            # rows are in the frontier) over the same peak. Both can be recomputed from work_per_matching.
            "roofline": {"kernel": names[dom], "bound": "alu", "achieved": achieved, "peak": alu_peak,
                         "unit": "Gop/s", "frac": achieved / alu_peak,
                         "ops_per_launch": dom_scalar, "ops_model": "scalar: 4NS+2NU+(N/32)L+3NK (greedy), "
                         "2N*path_steps+(N/32)L+3NK+4N^2 (BvN)",
                         "frac_parallel_formulation": achieved_par / alu_peak,
                         "ops_per_launch_parallel_formulation": dom_ops,
                         "traffic": captured_traffic(names[dom]) if CFG == 3 else None,
                         "peak_source": f"148 SMs x 4 schedulers x 32 lanes x {sm_mhz:.0f} MHz (sampled)",
                         "peak_measured_int_mix": alu_measured, "frac_of_measured_int_mix": achieved / alu_measured,
                         "frac_parallel_formulation_of_measured_int_mix": achieved_par / alu_measured,
                         "work_per_matching": {"greedy": per_matching(work_mw, WORK_NAMES_MW),
                                               "bvn": per_matching(work_bv, WORK_NAMES_BVN)},
                         "other_decomposer": {"kernel": names[other],
                                              "frac": other_scalar / (per_kernel[other] * 1e-3) / 1e9 / alu_peak,
                                              "frac_parallel_formulation":
                                                  other_par / (per_kernel[other] * 1e-3) / 1e9 / alu_peak,
                                              "ops_per_launch": other_scalar},
                         "scoring_kernel_hbm": {"kernel": names[3], "bound": "hbm",
                                                "algorithmic_bytes": B * (4 * N * N + k_bv * (N + 4) + 48),
                                                "achieved_gbs": B * (4 * N * N + k_bv * (N + 4) + 48)
                                                / (per_kernel[3] * 1e-3) / 1e9,
                                                "frac": B * (4 * N * N + k_bv * (N + 4) + 48)
                                                / (per_kernel[3] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                "traffic": captured_traffic(names[3]) if CFG == 3 else None,
                                                "peak_kind": f"of {peak_kind}"},
                         "hbm_side": {"algorithmic_bytes": bytes_bvn,
                                      "gbs": bytes_bvn / (per_kernel[2] * 1e-3) / 1e9,
                                      "peak_gbs": peaks["hbm_gbs"], "peak_kind": f"of {peak_kind}"}},
            "ideal_a2a_kernel": {"ms": a2a_ms, "bound": "hbm", "achieved": 4.0 * B * N * N / (a2a_ms * 1e-3) / 1e9,
                                 "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": 4.0 * B * N * N / (a2a_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                 "peak_kind": f"of {peak_kind}"},
            # algorithmic bytes of the scaling: demand in, scaled (double) and fixed-point matrix out;
            # the kernel itself streams the matrix four times per sweep through L2
            "sinkhorn_kernel": {"ms": sk_ms, "sweeps": SINKHORN_ITERS, "bound": "hbm",
                                "achieved": 16.0 * B * N * N / (sk_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                "unit": "GB/s", "frac": 16.0 * B * N * N / (sk_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                "peak_kind": f"of {peak_kind}", "all_status_ok": sk_ok},
            "ordering": ordering,
            "e2e": {"value": aggregate_value(world, B, e2e_steps, e2e_ms), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "how": "HostPipeline: upload, kernels and download on three streams, two slots",
                    "results_match_device_run": e2e_ok},
            # per step: greedy, BvN and two scoring launches; from N = 48 up the greedy and scoring entry
            # points each add a class pre-pass and a second (wide-class) launch
            "gpu_launches": (4 if N < 48 else 10) * args.steps,
            "clocks": ck,
        }
        if rates_by_k:
            out["rates_by_k_max"] = rates_by_k
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            threads = oracle.hardware_threads()
            sample = min(B, max(threads, 16) * 2 if N <= 64 else threads)
            rate = oracle_rate(D_host[:sample], threads, cap if N <= 64 else min(cap, 400))
            out["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                                   "sample": f"first {sample} matrices of the same batch, whole path"
                                   + ("" if N <= 64 else " with the BvN budget cut to 400 matchings")}
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
