"""Host-side logic of the multi-rank benchmark path, with two gloo ranks on CPU.

Matrices are independent, so N ranks run N replicas on different inputs (weak scaling):
no collective touches the data path, only the timings are combined (maximum over ranks).
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        D = bench.rank_demand(rank, 4)
        digest = int(np.asarray(D, dtype=np.int64).sum() % (1 << 31)) ^ int(D[0, 0, 1])
        # the slower rank defines the step time
        total_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 30.0 - 3.0 * rank], torch.device("cpu"), world)
        gathered = [None] * world
        dist.all_gather_object(gathered, digest)
        out.put((rank, total_ms, e2e_ms, gathered, D.shape))
    finally:
        dist.destroy_process_group()


def test_two_ranks_take_different_matrices_and_the_slowest_rank_sets_the_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, total_ms, e2e_ms, digests, shape in results:
        assert total_ms == 15.0 and e2e_ms == 30.0          # max over ranks, on every rank
        assert digests[0] != digests[1]                      # each rank has its own inputs
        assert shape == (4, 64, 64)
    # whole-job value: all ranks' matrices over the slowest rank's time
    assert bench.aggregate_value(2, 4096, 5, 500.0) == 2 * 4096 * 5 / 0.5


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks([1.0, 2.0], torch.device("cpu"), 1) == [1.0, 2.0]
    assert (bench.rank_demand(0, 2) == bench.rank_demand(0, 2)).all()
    assert (bench.rank_demand(0, 2) != bench.rank_demand(1, 2)).any()
