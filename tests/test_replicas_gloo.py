"""The multi-GPU mode of the benchmark is N independent replicas (no data-path collective);
the only cross-rank step is the MAX-over-ranks timing.  Checked here with two gloo ranks on
the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 1 is the slower replica: both ranks must report its time and the sum of the tokens
    ms, value = bench.aggregate_replicas(10.0 * (rank + 1), steps=5, tokens_per_rank=1000,
                                         dist=dist, device=torch.device("cpu"))
    out[rank] = (ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_take_the_slowest_time_and_add_their_tokens():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        port = 29500 + os.getpid() % 2000
        procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        res = dict(out)
    for r in range(2):
        ms, value = res[r]
        assert abs(ms - 4.0) < 1e-9                      # 20 ms (rank 1) / 5 steps
        assert abs(value - 2 * 1000 / 4.0e-3) < 1e-6     # tokens of both ranks over that time


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    ms, value = bench.aggregate_replicas(12.0, 3, 500, None, torch.device("cpu"))
    assert ms == 4.0 and abs(value - 125000.0) < 1e-9
