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


def test_bench_starts_its_own_replicas_when_not_under_torchrun():
    """`bench.py --gpus 2` outside torchrun starts two ranks itself; here they run the CPU
    self-test of the replica plumbing (gloo) instead of the GPU benchmark."""
    import json
    import subprocess

    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2",
                          "--selftest-replicas"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                               # rank 0 alone prints
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2
    assert abs(rec["ms_per_step"] - 4.0) < 1e-9          # the slower rank's 20 ms over 5 steps
    assert abs(rec["value"] - 2 * 1000 / 4.0e-3) < 1e-6


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    ms, value = bench.aggregate_replicas(12.0, 3, 500, None, torch.device("cpu"))
    assert ms == 4.0 and abs(value - 125000.0) < 1e-9
