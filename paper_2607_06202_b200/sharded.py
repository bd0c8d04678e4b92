"""One process per GPU, rank = GPU: the expert-parallel group over NVLink peer memory.

``ShardedEP`` is the thin driver around the sharded entry points of the C ABI
(``ubep_set_peers``, ``ubep_dispatch_sharded``, ``ubep_wait_arrivals``, ``ubep_combine_sharded``):
it obtains an arena and an expert-output buffer that the other GPUs can address
(``torch.distributed._symmetric_memory``: peer-to-peer mappings, no multicast is used),
exchanges their addresses, all-gathers the routing table (the one collective of the path,
8 bytes per slot) and orders the steps across ranks where memory is reused.  Every byte of a
row travels in the library's kernels as plain stores to / loads from peer memory.

Only the host-side logic (token partition, routing all-gather) can run without several GPUs;
the kernels are exercised on one GPU with every rank's arena as a separate allocation (see the
GPU tests).  Launch with torchrun, one rank per GPU, backend nccl.
"""
from __future__ import annotations

import os
from typing import Callable, List, Optional, Tuple

import torch
import torch.distributed as dist

from . import binding as B


def token_range(rank: int, T: int, world: int) -> Tuple[int, int]:
    """Tokens [begin, end) of the global batch that source rank `rank` owns (Sec. 2.3: contiguous
    shares that differ by at most one token)."""
    return rank * T // world, (rank + 1) * T // world


def gather_routing(idx_local: torch.Tensor, w_local: torch.Tensor, T: int, group=None):
    """All-gather of the routing table: every rank contributes the rows of its own tokens and gets
    topk_idx int32 [T, k] and topk_w fp32 [T, k] of the whole batch.  Shares differ by at most one
    token, so every rank pads its share to the largest one."""
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    k = idx_local.shape[1]
    b0, b1 = token_range(rank, T, world)
    assert idx_local.shape[0] == b1 - b0 and w_local.shape == idx_local.shape
    most = max(token_range(r, T, world)[1] - token_range(r, T, world)[0] for r in range(world))
    # one buffer for both arrays: the weights travel as their bit patterns
    mine = torch.full((most, 2 * k), -1, dtype=torch.int32, device=idx_local.device)
    mine[:b1 - b0, :k] = idx_local.to(torch.int32)
    mine[:b1 - b0, k:] = w_local.to(torch.float32).contiguous().view(torch.int32)
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    rows = [parts[r][:token_range(r, T, world)[1] - token_range(r, T, world)[0]] for r in range(world)]
    table = torch.cat(rows, dim=0)
    return table[:, :k].contiguous(), table[:, k:].contiguous().view(torch.float32)


def symmetric_alloc(nbytes: int, device: torch.device, group) -> Tuple[torch.Tensor, List[int]]:
    """nbytes of device memory that every rank of the group can address, and the address of every
    rank's copy as seen from this GPU."""
    os.environ.setdefault("TORCH_SYMM_MEM_DISABLE_MULTICAST", "1")   # plain peer mappings are all we use
    import torch.distributed._symmetric_memory as symm_mem
    t = symm_mem.empty(nbytes, dtype=torch.uint8, device=device)
    handle = symm_mem.rendezvous(t, group if group is not None else dist.group.WORLD)
    return t, [int(p) for p in handle.buffer_ptrs]


class ShardedEP:
    """This process's rank of an expert-parallel group: R = world size, experts p of rank p // L."""

    def __init__(self, *, num_experts: int, hidden: int, topk: int, max_tokens: int, rows_per_rank_cap: int,
                 dedup: int = 0, payload: int = 0, group=None, device: Optional[torch.device] = None,
                 alloc: Callable = symmetric_alloc, backend=B):
        """`alloc(nbytes, device, group)` returns memory every rank can address and its address on every
        rank; `backend` is the binding module.  Both can be replaced by stand-ins, which is how the
        order of the steps is tested on CPU ranks."""
        B = backend  # noqa: N806  (the names below are the binding's)
        self.B = backend
        self.group = group
        self.rank, self.world = dist.get_rank(group), dist.get_world_size(group)
        self.device = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        self.H, self.k, self.cap, self.payload = hidden, topk, rows_per_rank_cap, payload
        cfg = B.ubep_config_t(self.world, num_experts, hidden, topk, max_tokens, rows_per_rank_cap, 0, payload, dedup,
                              self.device.index or 0, 0, 0)
        nbytes = B.ubep_buffer_bytes(cfg)
        if nbytes == 0:
            raise B.UbepError(B.UBEP_ERR_ARG, "ubep_buffer_bytes")
        arena, arena_ptrs = alloc(nbytes, self.device, group)
        self.buf = B.Buffer(num_ranks=self.world, num_experts=num_experts, hidden=hidden, topk=topk,
                            max_tokens=max_tokens, rows_per_rank_cap=rows_per_rank_cap, dedup=dedup, payload=payload,
                            device=self.device.index or 0, arena=arena)
        B.ubep_set_peers(self.buf.handle, self.rank, arena_ptrs)
        # expert outputs, laid out like the receive regions; this rank fills region `rank`
        y_raw, y_ptrs = alloc(self.world * rows_per_rank_cap * hidden * 2, self.device, group)
        self.y = y_raw.view(torch.bfloat16).view(self.world, rows_per_rank_cap, hidden)
        self.y_ptrs = torch.tensor(y_ptrs, dtype=torch.int64, device=self.device)
        self._token = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.T = 0
        self.fence()     # every rank's arena is initialised before anybody stores into it

    def fence(self):
        """Stream-ordered barrier of the group (a one-word all-reduce on the current stream)."""
        if self.world > 1:
            dist.all_reduce(self._token, group=self.group)

    @property
    def region(self):
        """The rows this rank received (num_rows_per_rank[rank] of them are valid): bf16 [cap, H], or for
        FP8 rows the pair (e4m3 bytes [cap, H], fp32 scales [cap, H / 128])."""
        if self.payload:
            return self.buf.recv_x[self.rank], self.buf.recv_scale[self.rank]
        return self.buf.recv_x[self.rank].view(torch.bfloat16).view(self.cap, self.H)

    def dispatch(self, x_local: torch.Tensor, idx_local: torch.Tensor, w_local: torch.Tensor, T: int):
        """Routes this rank's tokens; returns when (on the stream) this rank's region is complete."""
        self.T = T
        self.idx, self.w = gather_routing(idx_local, w_local, T, self.group)
        self.B.ubep_dispatch_sharded(self.buf.handle, x_local.contiguous(), self.idx, self.w, T)
        self.B.ubep_wait_arrivals(self.buf.handle)
        return self.region, self.buf.num_rows_per_rank[self.rank]

    def combine(self, out_local: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Weighted sum of the expert outputs (self.y of every rank) for this rank's tokens."""
        b0, b1 = token_range(self.rank, self.T, self.world)
        if out_local is None:
            out_local = torch.empty((b1 - b0, self.H), dtype=torch.bfloat16, device=self.device)
        self.fence()     # every rank's y is complete
        self.B.ubep_combine_sharded(self.buf.handle, self.y_ptrs, self.w, self.T, out_local)
        self.fence()     # nobody overwrites a region or a y that a peer still reads
        return out_local

    def status(self) -> int:
        return self.buf.status()
