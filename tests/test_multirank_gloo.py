"""The N > 1 path of the benchmark on CPU: two gloo ranks on 127.0.0.1.  GEMM problems are independent, so
ranks share nothing on the data path; what the ranks do share is the timing protocol -- every rank its own
seeded problem, the step time is the max over ranks, rank 0 reports the whole-job aggregate."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2512_19018_b200 import workloads as W
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    case = W.config0().with_(M=64, N=48, K=32)
    mine = bench.rank_case(case, rank)
    A, B, _ = W.make_inputs(mine)
    digest = int(np.bitwise_xor.reduce(A.astype(np.uint64).ravel() * 1315423911 % (1 << 61)))
    fake_ms = 10.0 + 5.0 * rank                         # rank 1 is the slow one
    max_ms = bench.reduce_max(fake_ms, dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine.seed, digest))
    value = bench.aggregate_value(case, world, steps=4, max_ms=max_ms)
    dist.barrier()
    if rank == 0:
        out.put((max_ms, value, gathered, case.flops))
    dist.destroy_process_group()


def test_two_ranks_weak_scaling_protocol():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    max_ms, value, gathered, flops = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert max_ms == 15.0                                # the slowest rank defines the time
    assert abs(value - 2 * flops * 4 / 15e-3 / 1e12) < 1e-12
    (seed0, dig0), (seed1, dig1) = gathered
    assert seed0 != seed1 and dig0 != dig1               # every rank ran its own problem


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, None) == 3.5
    assert not dist.is_initialized()
