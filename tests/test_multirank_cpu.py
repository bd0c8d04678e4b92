"""The N > 1 path of the benchmark on CPU: two gloo ranks.  The hot path does not shard across
GPUs (replicas only), so what N > 1 adds is the rendezvous, the barrier, the max-over-ranks
timing and "rank 0 alone reports"; those are exercised here without a GPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    dist.barrier()
    mine = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
    slowest = bench.max_over_ranks(mine, world)
    value = bench.whole_job_value(1e9, slowest, world)
    # the reference arm: rank 0 alone works and prints, the others return at once
    class A:
        gpus, steps, warmup = world, 1, 0
    from paper_2607_06202_b200 import workload as W
    import contextlib, io
    buf = io.StringIO()
    with contextlib.redirect_stdout(buf):
        bench.run_reference(A, W.CONFIGS["tiny"], rank)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{slowest} {value}\n{buf.getvalue()}")
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_replica(tmp_path):
    world, port = 2, 29731
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    import json
    r0 = open(tmp_path / "r0.txt").read().splitlines()
    r1 = open(tmp_path / "r1.txt").read().splitlines()
    for first in (r0[0], r1[0]):
        slowest, value = map(float, first.split())
        assert slowest == 15.0                                   # max over ranks, on every rank
        assert abs(value - 2 * 1e9 / 15e-3 / 1e9) < 1e-9         # whole job = both replicas
    assert len(r1) == 1                                          # rank 1 printed nothing
    line = json.loads(r0[1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
