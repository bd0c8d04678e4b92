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


# ------------------------------------------------------------------ the driver's order of steps

class _FakeBuffer:
    """Stand-in for binding.Buffer: views of the right shapes in host memory, no library behind it."""

    def __init__(self, *, num_ranks, num_experts, hidden, topk, max_tokens, rows_per_rank_cap, dedup=0, payload=0,
                 device=0, arena=None, **_):
        self.arena, self.handle = arena, object()
        self.recv_x = torch.zeros((num_ranks, rows_per_rank_cap, hidden * (1 if payload else 2)), dtype=torch.uint8)
        self.recv_scale = torch.zeros((num_ranks, rows_per_rank_cap, max(hidden // 128, 1)))
        self.num_rows_per_rank = torch.zeros(num_ranks, dtype=torch.int32)

    def status(self):
        return 0


class _FakeBackend:
    """Records every call the driver makes on the C ABI, with what it was given."""
    UBEP_ERR_ARG = -1
    UbepError = RuntimeError

    def __init__(self, log):
        self.log = log
        self.Buffer = _FakeBuffer

    def ubep_config_t(self, *a):
        return a

    def ubep_buffer_bytes(self, cfg):
        return 4096

    def ubep_set_peers(self, handle, rank, ptrs):
        self.log.append(("set_peers", rank, tuple(ptrs)))

    def ubep_dispatch_sharded(self, handle, x_local, idx, w, T):
        self.log.append(("dispatch", tuple(x_local.shape), idx.clone(), w.clone(), T))

    def ubep_wait_arrivals(self, handle):
        self.log.append(("wait",))

    def ubep_combine_sharded(self, handle, y_ptrs, w, T, out_local):
        self.log.append(("combine", tuple(y_ptrs.tolist()), tuple(out_local.shape), T))


def _driver_worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []

    def alloc(nbytes, device, group):
        """Host memory, and its 'address' on every rank: exchanged through the group like the real
        rendezvous does, so that a rank passing the wrong list shows."""
        t = torch.zeros(nbytes, dtype=torch.uint8)
        mine = torch.tensor([1000 * (rank + 1) + len([e for e in log if e[0] == "alloc"])], dtype=torch.int64)
        parts = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(parts, mine)
        log.append(("alloc", nbytes))
        return t, [int(p.item()) for p in parts]

    class Logged(sharded.ShardedEP):
        def fence(self):
            log.append(("fence",))
            super().fence()

    cfg = W.Config("drv", T=21, H=128, E=8, R=world, k=2, seed=6200)
    wl = W.make_workload(cfg)
    b0, b1 = sharded.token_range(rank, cfg.T, world)
    ep = Logged(num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T, rows_per_rank_cap=32,
                device=torch.device("cpu"), alloc=alloc, backend=_FakeBackend(log))
    x = torch.zeros((b1 - b0, cfg.H), dtype=torch.bfloat16)
    ep.dispatch(x, torch.from_numpy(wl.topk_idx[b0:b1].copy()), torch.from_numpy(wl.topk_w[b0:b1].copy()), cfg.T)
    out = ep.combine()
    kinds = [e[0] for e in log]
    ok = kinds == ["alloc", "set_peers", "alloc", "fence", "dispatch", "wait", "fence", "combine", "fence"]
    peers = log[1]
    ok = ok and peers[1] == rank and peers[2] == tuple(1000 * (r + 1) for r in range(world))   # arena of every rank
    d = log[4]
    ok = ok and d[1] == (b1 - b0, cfg.H) and d[4] == cfg.T
    ok = ok and np.array_equal(d[2].numpy(), wl.topk_idx) and np.array_equal(d[3].numpy(), wl.topk_w)   # whole table
    cmb = log[7]
    ok = ok and cmb[1] == tuple(1000 * (r + 1) + 1 for r in range(world)) and cmb[2] == (b1 - b0, cfg.H)
    ok = ok and tuple(out.shape) == (b1 - b0, cfg.H)
    with open(os.path.join(out_dir, f"d{rank}.txt"), "w") as f:
        f.write("ok" if ok else "mismatch " + repr(kinds))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_run_the_drivers_steps_in_order(tmp_path):
    """ShardedEP with stand-ins for the allocator and the library: the arenas' addresses are exchanged
    and passed on in rank order, every rank dispatches its own token range with the table of the whole
    batch, the arrival wait follows the dispatch, and combine sits between two fences."""
    world, port = 2, 29743
    mp.spawn(_driver_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        assert open(tmp_path / f"d{r}.txt").read() == "ok"
