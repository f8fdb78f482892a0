"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import oracle
import paper_2605_26845_b200 as ms
from paper_2605_26845_b200.workload import (CONFIGS, DEFAULT_MODEL, PROFILED_MODEL, bvn_capacity, make_demand,
                                            random_matrices, structured_cases)

pytestmark = pytest.mark.gpu

KINDS = [dict(kind="uniform", high=1000), dict(kind="ties"), dict(kind="uniform", high=9, zero_frac=0.6)]


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_schedule_equal(gpu, ref, key):
    """perm / dur are compared on the first count[b] matchings only (the rest is unspecified)."""
    count = gpu.count.cpu().numpy()
    status = gpu.status.cpu().numpy()
    assert (status == ref["status"]).all(), (status, ref["status"])
    assert (count == ref["count"]).all(), (count, ref["count"])
    perm = gpu.perm.cpu().numpy()
    dur = gpu.dur.cpu().numpy()
    kk = np.arange(perm.shape[1])[None, :] < count[:, None]
    assert (perm[kk] == ref["perm"][kk]).all()
    assert (dur[kk] == ref[key][kk]).all()


def check_all(D, k_mw, k_bvn, model=DEFAULT_MODEL, threads=8):
    d = dev(D)
    g = ms.mw_decompose(d, k_mw, want_residual=True)
    rg = oracle.mw_decompose(D, k_mw, threads=threads)
    assert_schedule_equal(g, rg, "dur")
    ok = rg["status"] >= 0
    assert (g.extra.cpu().numpy()[ok] == rg["residual"][ok]).all()
    rv = oracle.bvn_decompose(D, k_bvn, threads=threads)
    ok = rv["status"] >= 0
    for scratch in (True, False):       # global working copy / shared-memory (cluster) path
        v = ms.bvn_decompose(d, k_bvn, want_aug=True, scratch=scratch)
        assert_schedule_equal(v, rv, "coef")
        assert (v.extra.cpu().numpy()[ok] == rv["aug"][ok]).all()
    for sched, ref, key in ((g, rg, "dur"), (v, rv, "coef")):
        good = dev(ref["status"] >= 0)
        count = torch.where(good, sched.count, torch.zeros_like(sched.count))
        # rows beyond count are never read, so uninitialised memory there is fine
        s = ms.schedule_eval(d, sched.perm, sched.dur, count, model)
        cnt = np.where(ref["status"] >= 0, ref["count"], 0).astype(np.int32)
        rs = oracle.schedule_eval(D, ref["perm"], ref[key], cnt, model, threads=threads)
        for name in ms.SCORE_FIELDS + ("status",):
            assert (s[name].cpu().numpy() == rs[name]).all(), name
    return g, v


@pytest.mark.parametrize("N", [1, 2, 3, 5, 8, 13, 17, 31, 32, 33, 48, 64])
@pytest.mark.parametrize("kw", KINDS)
def test_small_matrices_full_decompositions(N, kw):
    D = random_matrices(5, N, seed=1000 + N, **kw)
    check_all(D, N * N + 1, bvn_capacity(N))


@pytest.mark.parametrize("N", [65, 96, 100, 128, 129, 192, 232, 233, 256])
@pytest.mark.parametrize("kw", KINDS)
def test_large_matrices_prefix(N, kw):
    """The oracle needs O(N^3) per matching, so large sizes are compared on a schedule prefix."""
    D = random_matrices(3, N, seed=2000 + N, **kw)
    check_all(D, 6, 10)


@pytest.mark.parametrize("N,kw", [(129, KINDS[0]), (200, KINDS[2]), (256, KINDS[0]), (256, KINDS[1])])
def test_team_kernel_deep_prefix(N, kw):
    """Above 128 ranks a small batch runs the Birkhoff kernel that puts a CTA of eight warps on each
    matrix: several hundred matchings deep against the oracle, and against the one-warp kernel
    (shared-memory placement) on the same inputs."""
    D = random_matrices(2, N, seed=7000 + N, **kw)
    d = dev(D)
    K = 400
    rv = oracle.bvn_decompose(D, K, threads=8)
    team = ms.bvn_decompose(d, K, want_aug=True, scratch=True)
    warp = ms.bvn_decompose(d, K, want_aug=True, scratch=False)
    for v in (team, warp):
        assert_schedule_equal(v, rv, "coef")
        assert (v.extra.cpu().numpy() == rv["aug"]).all()


@pytest.mark.parametrize("N,kw", [(129, KINDS[2]), (256, KINDS[0])])
def test_one_warp_kernel_above_128_ranks_in_a_large_batch(N, kw):
    """Above 128 ranks a batch of at least eight matrices per SM keeps one warp per matrix, with the
    working copy in global memory and the search records in shared memory; a small batch of the same
    matrices takes the CTA-per-matrix kernel. Both against the oracle on a sample, and against each
    other on every matrix."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    base = random_matrices(37, N, seed=8100 + N, **kw)
    reps = -(-8 * sms // base.shape[0])
    D = np.concatenate([base] * reps)
    assert D.shape[0] >= 8 * sms
    K = 24
    wide = ms.bvn_decompose(dev(D), K, want_aug=True)
    small = ms.bvn_decompose(dev(base), K, want_aug=True)
    rv = oracle.bvn_decompose(base, K, threads=8)
    assert_schedule_equal(small, rv, "coef")
    for q in range(reps):
        part = ms.Schedule(*(getattr(wide, f)[q * 37:(q + 1) * 37] for f in ("perm", "dur", "count", "status")))
        assert_schedule_equal(part, rv, "coef")
    assert (wide.extra[:37].cpu().numpy() == rv["aug"]).all()


@pytest.mark.parametrize("N,per_sm", [(16, 14), (64, 13), (64, 27)])
def test_paced_launch_of_a_resident_batch_gives_the_same_schedules(N, per_sm):
    """From twelve matrices per SM up, when the whole batch is resident at once, the warps that share a
    scheduler pace one another (a warp that is ahead sleeps). Timing only: the complete schedules must equal
    those of the same matrices decomposed in a small, unpaced batch, and the oracle's."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    base = random_matrices(29, N, seed=8300 + N, **(KINDS[2] if N == 16 else KINDS[0]))
    reps = -(-per_sm * sms // base.shape[0])
    D = np.concatenate([base] * reps)
    assert D.shape[0] >= 12 * sms
    K = bvn_capacity(N)
    rv = oracle.bvn_decompose(base, K, threads=8)
    small = ms.bvn_decompose(dev(base), K)
    assert_schedule_equal(small, rv, "coef")
    for _ in range(2):   # twice: entries of the pacing table left by the first launch must not matter
        wide = ms.bvn_decompose(dev(D), K)
        torch.cuda.synchronize()
        for q in range(reps):
            part = ms.Schedule(*(getattr(wide, f)[q * 29:(q + 1) * 29] for f in ("perm", "dur", "count", "status")))
            assert_schedule_equal(part, rv, "coef")


@pytest.mark.parametrize("N", [233, 256])
def test_wide_entries_above_232_ranks_run_deep_on_the_cluster_path(N):
    """Entries beyond 16 bits at N > 232 put the matrix (as int32) across the two CTAs of a cluster, for
    the greedy decomposition and for the scoring alike: 70 matchings deep against the oracle."""
    D = random_matrices(3, N, seed=8300 + N, kind="uniform", high=400000, zero_frac=0.5)
    D[2] = np.minimum(D[2], 65535)                       # one narrow matrix in the same batch
    d = dev(D)
    K = 70
    g = ms.mw_decompose(d, K, want_residual=True)
    rg = oracle.mw_decompose(D, K, threads=8)
    assert_schedule_equal(g, rg, "dur")
    assert (g.extra.cpu().numpy() == rg["residual"]).all() and (rg["count"] == K).all()
    for model in (DEFAULT_MODEL, PROFILED_MODEL):
        s = ms.schedule_eval(d, g.perm, g.dur, g.count, model, prefix=True)
        rs = oracle.schedule_eval(D, rg["perm"], rg["dur"], rg["count"], model, threads=8)
        for name in ms.SCORE_FIELDS + ("status",):
            assert (s[name].cpu().numpy() == rs[name]).all(), name
        rp = oracle.schedule_prefix_eval(D, rg["perm"], rg["dur"], rg["count"], model, threads=8)
        assert (s["prefix_overlap_ns"].cpu().numpy() == rp["prefix_overlap_ns"]).all()
        assert (s["prefix_unserved_tokens"].cpu().numpy() == rp["prefix_unserved_tokens"]).all()


@pytest.mark.parametrize("N", [1, 2, 5, 8, 17, 64, 100])
def test_closed_form_cases(N):
    cases = structured_cases(N, m=7)
    D = np.stack(list(cases.values()))
    g, v = check_all(D, N + 2, N + 2)
    names = list(cases)
    gc = g.count.cpu().numpy()
    vc = v.count.cpu().numpy()
    assert gc[names.index("zero")] == 0 and vc[names.index("zero")] == 0
    assert gc[names.index("scaled_permutation")] == 1 and vc[names.index("scaled_permutation")] == 1
    assert gc[names.index("uniform")] == N and vc[names.index("uniform")] == N
    assert gc[names.index("hot_column")] == N and gc[names.index("diagonal")] == 1


def test_bad_inputs_and_budget():
    D = make_demand(1, 6)
    D[1, 2, 3] = -1
    D[4, 0, 0] = 2**31 - 1          # entry above 2^28 (greedy) and row sum beyond 31 bits (BvN)
    check_all(D, 8, 50)
    check_all(D, 1, 1)
    check_all(D, 3, 7)


def test_eval_rejects_bad_schedules():
    D = make_demand(1, 4)
    d = dev(D)
    g = ms.mw_decompose(d, 8)
    perm = g.perm.cpu().numpy().copy()
    dur = g.dur.cpu().numpy().copy()
    count = g.count.cpu().numpy().copy()
    perm[0, 1, 3] = perm[0, 1, 2]   # repeated column
    perm[1, 0, 0] = 200             # out of range
    dur[2, 0] = -4
    count[3] = 9                    # beyond the stride
    s = ms.schedule_eval(d, dev(perm), dev(dur), dev(count))
    r = oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL)
    assert list(r["status"]) == [-1, -1, -1, -1]
    for name in ms.SCORE_FIELDS + ("status",):
        assert (s[name].cpu().numpy() == r[name]).all(), name


@pytest.mark.parametrize("gbps", [1, 2, 3, 7, 400, 1000, 4099, 65536, 2**20 - 1, 2**20])
def test_link_time_for_any_link_speed_and_token_size(gbps):
    """The kernel divides by the link speed with a multiply-high by a constant made on the host; the
    quotient must equal the plain ceiling division of the definition for every speed and size in range."""
    N = 5
    rng = np.random.default_rng(gbps)
    durs = np.array([1, 2, 3, 25, 2**31 - 1, 2**30 + 1, 999_983, 2**20, 2**20 + 1, 123_456_789], dtype=np.int32)
    K = len(durs)
    B = 4
    D = rng.integers(0, 2**31 - 1, size=(B, N, N), dtype=np.int64).astype(np.int32)
    perm = np.stack([np.stack([rng.permutation(N) for _ in range(K)]) for _ in range(B)]).astype(np.uint8)
    dur = np.stack([rng.permutation(durs) for _ in range(B)]).astype(np.int32)
    count = np.full(B, K, dtype=np.int32)
    for nbytes in (1, 50, 14336, 2**20 - 1, 2**20):
        model = dict(DEFAULT_MODEL, link_gbps=gbps, bytes_per_token=nbytes)
        s = ms.schedule_eval(dev(D), dev(perm), dev(dur), dev(count), model, prefix=True)
        r = oracle.schedule_eval(D, perm, dur, count, model)
        assert (r["status"] == 0).all()
        for name in ms.SCORE_FIELDS + ("status",):
            assert (s[name].cpu().numpy() == r[name]).all(), (name, nbytes)
        rp = oracle.schedule_prefix_eval(D, perm, dur, count, model)
        assert (s["prefix_overlap_ns"].cpu().numpy() == rp["prefix_overlap_ns"]).all()


@pytest.mark.parametrize("N", [100, 129, 200, 256])
def test_large_matrix_scoring_rejects_bad_schedules_and_scores_long_ones(N):
    """Few large matrices are scored by the kernel that puts one CTA on each matrix: faulty schedules,
    a mix of narrow and wide matrices, and a schedule several chunks long, all against the oracle."""
    D = random_matrices(6, N, seed=9000 + N, kind="uniform", high=3000)
    D[5, 1, 2] = 70000                        # one wide matrix: scored by the one-warp kernel
    d = dev(D)
    K = 75
    g = ms.mw_decompose(d, K)
    perm = g.perm.cpu().numpy().copy()
    dur = g.dur.cpu().numpy().copy()
    count = g.count.cpu().numpy().copy()
    assert (count > 64).all()
    perm[0, 40, 3] = perm[0, 40, 2]           # repeated column, in the second chunk
    perm[1, 0, 0] = 255 if N < 256 else perm[1, 0, 1]   # out of range (N = 256 has no such byte: repeat instead)
    dur[2, 65] = -4
    count[3] = K + 1                          # beyond the stride
    for model in (DEFAULT_MODEL, PROFILED_MODEL):
        s = ms.schedule_eval(d, dev(perm), dev(dur), dev(count), model)
        r = oracle.schedule_eval(D, perm, dur, count, model, threads=8)
        assert list(r["status"]) == [-1, -1, -1, -1, 0, 0]
        for name in ms.SCORE_FIELDS + ("status",):
            assert (s[name].cpu().numpy() == r[name]).all(), name


@pytest.mark.parametrize("N", [4, 64, 200])
def test_stage_sums_out_of_range_are_rejected_like_the_oracle_does(N):
    """Slowest link, largest token: transfer times that add up beyond 2^60 ns give BAD_INPUT, not a wrapped
    makespan; just below the limit the 64-bit sums are still exact (one-warp and CTA-per-matrix kernels)."""
    K = 600
    D = random_matrices(3, N, seed=31 + N, kind="uniform", high=100)
    perm = np.tile(np.arange(N, dtype=np.uint8), (3, K, 1))
    dur = np.zeros((3, K), np.int32)
    dur[0, :128] = 2**31 - 1
    dur[1, :32] = 2**31 - 1
    dur[2, 500:] = 2**31 - 1                       # the sum leaves its range late in the schedule
    count = np.array([K, K, K], np.int32)
    model = dict(DEFAULT_MODEL, bytes_per_token=2**20, link_gbps=1)
    for prefix in (False, True):
        s = ms.schedule_eval(dev(D), dev(perm), dev(dur), dev(count), model, prefix=prefix)
        r = oracle.schedule_eval(D, perm, dur, count, model)
        assert list(r["status"]) == [-1, 0, -1]
        for name in ms.SCORE_FIELDS + ("status",):
            assert (s[name].cpu().numpy() == r[name]).all(), name


def test_argument_errors_are_reported():
    d = dev(make_demand(1, 2))
    with pytest.raises(ms.MoeschedError):
        ms.mw_decompose(d, 0)
    with pytest.raises(ms.MoeschedError):
        ms.mw_decompose(d.cpu(), 8)
    with pytest.raises(ms.MoeschedError):
        ms.schedule_eval(d, torch.zeros((2, 1, 8), dtype=torch.uint8, device="cuda"),
                         torch.zeros((2, 1), dtype=torch.int32, device="cuda"),
                         torch.zeros(2, dtype=torch.int32, device="cuda"), dict(DEFAULT_MODEL, link_gbps=0))
    too_big = torch.zeros((1, 257, 257), dtype=torch.int32, device="cuda")
    with pytest.raises(ms.MoeschedError):
        ms.mw_decompose(too_big, 4)


def test_runs_are_deterministic_and_stream_ordered():
    D = make_demand(2, 64)
    d = dev(D)
    a = ms.bvn_decompose(d)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        b = ms.bvn_decompose(d)
    side.synchronize()
    torch.cuda.synchronize()
    assert (a.count == b.count).all() and (a.status == b.status).all()
    kk = (torch.arange(a.perm.shape[1], device="cuda")[None, :] < a.count[:, None])
    assert (a.perm[kk] == b.perm[kk]).all() and (a.dur[kk] == b.dur[kk]).all()


@pytest.mark.parametrize("N", [1, 5, 16, 33, 64, 100, 256])
def test_ideal_all_to_all_and_knee_model(N):
    from paper_2605_26845_b200.workload import PROFILED_MODEL
    D = random_matrices(6, N, seed=4000 + N, kind="uniform", high=3000, zero_frac=0.3)
    D[1] = 0
    D[2, 0, 0] = -1
    d = dev(D)
    for model in (DEFAULT_MODEL, PROFILED_MODEL, dict(PROFILED_MODEL, expert_knee_tokens=50, expert_fixed_ns=7)):
        got = ms.ideal_a2a(d, model)
        ref = oracle.ideal_a2a(D, model)
        for name in ("comm_ns", "makespan_ns", "status"):
            assert (got[name].cpu().numpy() == ref[name]).all(), name
        D2 = D.copy()
        D2[2, 0, 0] = 1
        check_all(D2, 4, 6, model=model)              # the knee enters the scores of both schedules


def test_ideal_all_to_all_rejects_port_overflow():
    D = np.zeros((2, 4, 4), np.int32)
    D[0, 0, :2] = 2**30                               # row sum 2^31: beyond the port range
    D[1, 0, 0] = 2**31 - 1
    got = ms.ideal_a2a(dev(D), DEFAULT_MODEL)
    ref = oracle.ideal_a2a(D, DEFAULT_MODEL)
    assert list(ref["status"]) == [-1, 0]
    for name in ("comm_ns", "makespan_ns", "status"):
        assert (got[name].cpu().numpy() == ref[name]).all(), name


@pytest.mark.parametrize("overlap", [True, False])
def test_path_runner_matches_separate_calls(overlap):
    D = make_demand(2, 96)
    d = dev(D)
    N = D.shape[1]
    path = ms.Path(96, N, 16)
    for _ in range(2):                                   # buffers are reused from run to run
        path.run(d, DEFAULT_MODEL, overlap=overlap)
    torch.cuda.current_stream().synchronize()
    g = ms.mw_decompose(d, 16)
    v = ms.bvn_decompose(d)
    for a, b in ((path.mw, g), (path.bvn, v)):
        kk = torch.arange(a.perm.shape[1], device="cuda")[None, :] < b.count[:, None]
        assert (a.count == b.count).all() and (a.status == b.status).all()
        assert (a.perm[kk] == b.perm[kk]).all() and (a.dur[kk] == b.dur[kk]).all()
    sg = ms.schedule_eval(d, g.perm, g.dur, g.count)
    sv = ms.schedule_eval(d, v.perm, v.dur, v.count)
    for i, name in enumerate(ms.SCORE_FIELDS):
        assert (path.score_mw[i] == sg[name]).all() and (path.score_bvn[i] == sv[name]).all()
    ref = oracle.schedule_eval(D, g.perm.cpu().numpy(), g.dur.cpu().numpy(), g.count.cpu().numpy(), DEFAULT_MODEL)
    assert (path.score_mw[0].cpu().numpy() == ref["makespan_overlap_ns"]).all()


@pytest.mark.parametrize("N", [4, 8, 64, 128])
def test_values_at_the_top_of_the_range(N):
    """Entries up to 2^28 (greedy range) and sums up to 2^31-1 (BvN range): no 32-bit overflow."""
    rng = np.random.default_rng(77 + N)
    D = rng.integers(0, 2**28 + 1, size=(4, N, N)).astype(np.int32)
    D[0, 0, 0] = 2**28                                   # exactly the greedy limit
    D[1] = D[1] // (N * 2)                               # sums stay below 2^31: BvN accepts this one
    D[2] = np.where(rng.random((N, N)) < 0.8, 0, D[2])   # sparse with huge entries
    D[3, 1, 1] = 2**28 + 1                               # one above the limit: greedy rejects matrix 3
    check_all(D, 12, 12)


def test_empty_batch_is_a_no_op():
    d = torch.zeros((0, 8, 8), dtype=torch.int32, device="cuda")
    g = ms.mw_decompose(d, 4)
    v = ms.bvn_decompose(d, 4)
    s = ms.schedule_eval(d, g.perm, g.dur, g.count)
    a = ms.ideal_a2a(d)
    torch.cuda.synchronize()
    assert g.count.numel() == 0 and v.count.numel() == 0 and s["status"].numel() == 0 and a["status"].numel() == 0


def test_block_diagonal_and_staircase_matrices():
    """Decomposable supports: several independent blocks, and a triangular staircase."""
    N = 24
    D = np.zeros((3, N, N), np.int32)
    for k in range(0, N, 6):
        D[0, k:k + 6, k:k + 6] = np.arange(1, 37).reshape(6, 6) + k
    D[1] = np.triu(np.full((N, N), 5)) + np.eye(N, dtype=np.int32)
    D[2] = np.tril(np.arange(N * N).reshape(N, N) % 7)
    check_all(D, N * N, ms.bvn_capacity(N))


def test_host_pipeline_returns_the_same_results_in_order():
    batches = [make_demand(2, 64, seed=s) for s in (1, 2, 3, 4, 5)]
    pipe = ms.HostPipeline(64, 16, 16)
    slots = []
    got = []
    for i, D in enumerate(batches):
        h = torch.from_numpy(D).pin_memory()
        slots.append(pipe.submit(h))
        if i >= 1:                                       # consume the previous batch while this one runs
            got.append([t.clone() for t in pipe.result(slots[i - 1])])
    got.append([t.clone() for t in pipe.result(slots[-1])])
    for D, out in zip(batches, got):
        ref = oracle.mw_decompose(D, 16, threads=4)
        rv = oracle.bvn_decompose(D, ms.bvn_capacity(16), threads=4)
        count, bcount = out[2].numpy(), out[6].numpy()
        assert (count == ref["count"]).all() and (bcount == rv["count"]).all()
        kk = np.arange(16)[None, :] < count[:, None]
        assert (out[0].numpy()[kk] == ref["perm"][kk]).all() and (out[1].numpy()[kk] == ref["dur"][kk]).all()
        kk = np.arange(rv["perm"].shape[1])[None, :] < bcount[:, None]
        assert (out[4].numpy()[kk] == rv["perm"][kk]).all() and (out[5].numpy()[kk] == rv["coef"][kk]).all()
        sc = oracle.schedule_eval(D, rv["perm"], rv["coef"], rv["count"], DEFAULT_MODEL)
        assert (out[9].numpy()[0] == sc["makespan_overlap_ns"]).all()


@pytest.mark.parametrize("N", [3, 16, 33, 64, 128, 256])
def test_prefix_scores(N):
    D = random_matrices(5, N, seed=6000 + N, kind="uniform", high=500, zero_frac=0.4)
    d = dev(D)
    k = min(12, N * N)
    for sched, key in ((ms.mw_decompose(d, k), "dur"), (ms.bvn_decompose(d, k), "coef")):
        perm = sched.perm.cpu().numpy().copy()
        dur = sched.dur.cpu().numpy().copy()
        count = sched.count.cpu().numpy().copy()
        kk = np.arange(k)[None, :] < count[:, None]
        perm[~kk] = 0
        dur[~kk] = 0
        perm[4, 0, 0] = perm[4, 0, N - 1] if N > 1 else 200          # matrix 4: a bad schedule
        if N == 1:
            perm[4, 0, 0] = 200
        if count[4] == 0:
            count[4] = 1
        got = ms.schedule_eval(d, dev(perm), dev(dur), dev(count), DEFAULT_MODEL, prefix=True)
        ref = oracle.schedule_prefix_eval(D, perm, dur, count, DEFAULT_MODEL, threads=4)
        plain = oracle.schedule_eval(D, perm, dur, count, DEFAULT_MODEL, threads=4)
        assert (got["status"].cpu().numpy() == ref["status"]).all() and ref["status"][4] == -1
        for name in ("prefix_overlap_ns", "prefix_unserved_tokens"):
            assert (got[name].cpu().numpy() == ref[name]).all(), name
        for name in ms.SCORE_FIELDS:
            assert (got[name].cpu().numpy() == plain[name]).all(), name


@pytest.mark.parametrize("N", [48, 64, 100, 200, 256])
def test_mixed_16_bit_and_wide_matrices_in_one_batch(N):
    """The greedy path holds matrices whose entries fit 16 bits in a narrower layout; a batch may mix both."""
    D = random_matrices(6, N, seed=7000 + N, kind="uniform", high=60000, zero_frac=0.3)
    D[1] *= 3                                          # entries up to 180000: wide
    D[2, 5 % N, 7 % N] = 65535                         # the largest narrow value
    D[3, 5 % N, 7 % N] = 65536                         # the smallest wide value
    D[4] = 0
    D[5, 0, 0] = -2                                    # bad input goes through the wide path
    check_all(D, 5, 5)


def test_graph_replay_gives_the_same_schedules():
    D = make_demand(1, 64)
    d = dev(D)
    path = ms.Path(64, 8, 8)
    for _ in range(3):
        path.run_graph(d, DEFAULT_MODEL)
    d2 = dev(make_demand(1, 64, seed=5))                 # another tensor: the graph is captured again
    other = ms.Path(64, 8, 8).run(d2)
    path.run_graph(d2, DEFAULT_MODEL)
    torch.cuda.synchronize()
    for a, b in ((path.mw, other.mw), (path.bvn, other.bvn)):
        kk = torch.arange(a.perm.shape[1], device="cuda")[None, :] < b.count[:, None]
        assert (a.count == b.count).all() and (a.perm[kk] == b.perm[kk]).all() and (a.dur[kk] == b.dur[kk]).all()
    assert (path.score_bvn == other.score_bvn).all() and (path.score_mw == other.score_mw).all()
