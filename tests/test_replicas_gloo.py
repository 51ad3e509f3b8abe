"""The N > 1 path of the benchmark is "replicas only": every rank runs the same independent workload,
a barrier brackets the timed region, the slowest rank's time is the job's time and the job's
throughput is N times the per-rank work over that time.  Checked here with two gloo ranks on CPU
(the ranks time the CPU oracle's step instead of the CUDA step; the aggregation logic is what is
under test)."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    steps, batch = 3, 64
    ms_local = 10.0 * (rank + 1)                       # rank 1 is the slow one
    value, ms = bench.aggregate_over_ranks(ms_local, steps, batch, world, device="cpu")
    if rank == 0:
        out.put((value, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_work():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    value, ms = out.get()
    assert ms == pytest.approx(20.0)                                   # max over ranks
    assert value == pytest.approx(2 * 3 * 64 / 20e-3)                  # whole-job samples/s


def test_single_process_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    value, ms = bench.aggregate_over_ranks(5.0, 10, 256, 1)
    assert ms == 5.0 and value == pytest.approx(10 * 256 / 5e-3)
