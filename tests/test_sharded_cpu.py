"""Host-side logic of the path for ranks on different GPUs, on CPU with three gloo ranks: the
token partition agrees with the oracle's source-rank rule, and the routing all-gather gives
every rank the table of the whole batch although the shares differ in size."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2607_06202_b200 import sharded
from paper_2607_06202_b200 import workload as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
CFG = W.Config("shares", T=37, H=64, E=12, R=3, k=3, seed=6100)


def test_token_ranges_are_the_oracles_source_ranks():
    for T, S in ((37, 3), (5, 8), (512, 32), (1, 1), (0, 4), (4096, 72)):
        owner = np.full(T, -1)
        for s in range(S):
            b0, b1 = sharded.token_range(s, T, S)
            assert 0 <= b0 <= b1 <= T
            owner[b0:b1] = s
        assert [int(v) for v in owner] == [oracle.source_rank(t, T, S) for t in range(T)]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = W.make_workload(CFG)
    b0, b1 = sharded.token_range(rank, CFG.T, world)
    idx, w = sharded.gather_routing(torch.from_numpy(wl.topk_idx[b0:b1].copy()),
                                    torch.from_numpy(wl.topk_w[b0:b1].copy()), CFG.T)
    ok = (idx.dtype == torch.int32 and w.dtype == torch.float32
          and np.array_equal(idx.numpy(), wl.topk_idx)
          and np.array_equal(w.numpy().view(np.int32), wl.topk_w.view(np.int32)))   # weights bit for bit
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.barrier()
    dist.destroy_process_group()


def test_three_gloo_ranks_gather_the_whole_routing_table(tmp_path):
    world, port = 3, 29741
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert open(tmp_path / f"r{r}.txt").read() == "ok"
