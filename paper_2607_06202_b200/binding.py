"""ctypes binding of the C-ABI library ``libubep.so`` (see ``include/ubep.h``).

The module-level ``ubep_*`` functions have the names and argument order of the C entry
points and only marshal arguments (torch tensors -> device pointers, the current torch
stream -> ``void*``).  ``Buffer`` is a small convenience holder for an arena tensor and its
views.  PyTorch supplies device memory and streams; every step of dispatch / combine runs
in the library's kernels.  There is no fallback: if the library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libubep.so")

UBEP_OK = 0
UBEP_ERR_ARG, UBEP_ERR_CUDA, UBEP_ERR_CAPACITY, UBEP_ERR_TIMEOUT, UBEP_ERR_BAD_INDEX, UBEP_ERR_ARENA = \
    -1, -2, -3, -4, -5, -6
UBEP_ERR_CHECKSUM = -7
UBEP_SYNC_SW, UBEP_SYNC_TFF, UBEP_SYNC_DC, UBEP_SYNC_SP = 0, 1, 2, 3
UBEP_SYNC_BLOCK_BYTES, UBEP_SYNC_FLAG_BYTES = 16, 4
UBEP_SYNC_DC_BLOCK_BYTES, UBEP_SYNC_DC_MARKER_BYTES = 512, 32
UBEP_SYNC_SENTINEL = 0xFFFF
SYNC_NAMES = {"sw": 0, "tff": 1, "dc": 2, "sp": 3}
SYNC_VIEW_NAMES = ["tff_wire", "sp_wire", "checksum", "counters", "times", "seq"]
_SYNC_VIEW_DTYPES = [torch.uint8, torch.uint8, torch.int64, torch.int32, torch.int64, torch.int32]
_SYNC_VIEW_RANK = [3, 3, 2, 2, 2, 1]
UBEP_PAYLOAD_BF16, UBEP_PAYLOAD_FP8_E4M3 = 0, 1
UBEP_PIPELINE_AUTO, UBEP_PIPELINE_PHASED, UBEP_PIPELINE_FUSED, UBEP_PIPELINE_LOCAL = 0, 1, 2, 3

VIEW_NAMES = ["recv_x", "recv_scale", "recv_src_idx", "recv_weight", "recv_topk_idx", "recv_topk_w",
              "expert_rows", "cnt", "src_offset", "expert_offset", "num_tokens_per_expert",
              "num_rows_per_rank", "num_tokens_per_rank", "slot_row", "arrival", "epoch", "trace", "shard_arrival"]
_VIEW_DTYPES = [torch.uint8, torch.float32, torch.int32, torch.float32, torch.int32, torch.float32,
                torch.int32, torch.int32, torch.int32, torch.int32, torch.int32, torch.int32, torch.int32,
                torch.int32, torch.int32, torch.int32, torch.int64, torch.int32]

# every symbol include/ubep.h declares
EXPORTS = ["ubep_buffer_bytes", "ubep_buffer_create", "ubep_buffer_destroy", "ubep_set_replicas",
           "ubep_set_dest_order", "ubep_get_dispatch_layout", "ubep_get_dispatch_layout_static", "ubep_dispatch", "ubep_combine", "ubep_view",
           "ubep_status", "ubep_epoch", "ubep_launch_count", "ubep_debug_withhold_flag", "ubep_debug_trace",
           "ubep_debug_set_quant_warps", "ubep_debug_set_count_warps", "ubep_debug_set_prefetch_rows", "ubep_debug_empty_launch",
           "ubep_last_cuda_error", "ubep_strerror", "ubep_map_workers",
           "ubep_sync_wire_bytes", "ubep_sync_attach", "ubep_dispatch_sync", "ubep_sync_view",
           "ubep_sync_scan_sentinel",
           "ubep_set_peers", "ubep_dispatch_sharded", "ubep_wait_arrivals", "ubep_combine_sharded"]


class ubep_config_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("num_ranks", "num_experts", "hidden", "topk", "max_tokens", "rows_per_rank_cap",
                 "num_src_ranks", "payload", "dedup", "device", "pipeline", "num_ctas")]


_lib = None


def load() -> ctypes.CDLL:
    """Load libubep.so; raises if it has not been built (no CPU or eager fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_06202_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, u32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64
    cfgp = ctypes.POINTER(ubep_config_t)
    lib.ubep_buffer_bytes.restype, lib.ubep_buffer_bytes.argtypes = ctypes.c_size_t, [cfgp]
    lib.ubep_buffer_create.restype = ctypes.c_int
    lib.ubep_buffer_create.argtypes = [cfgp, vp, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.ubep_buffer_destroy.restype, lib.ubep_buffer_destroy.argtypes = ctypes.c_int, [vp]
    lib.ubep_set_replicas.restype, lib.ubep_set_replicas.argtypes = ctypes.c_int, [vp, vp, vp, i32, i32]
    lib.ubep_set_dest_order.restype, lib.ubep_set_dest_order.argtypes = ctypes.c_int, [vp, vp]
    lib.ubep_get_dispatch_layout.restype = ctypes.c_int
    lib.ubep_get_dispatch_layout.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    lib.ubep_get_dispatch_layout_static.restype = ctypes.c_int
    lib.ubep_get_dispatch_layout_static.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp]
    lib.ubep_dispatch.restype, lib.ubep_dispatch.argtypes = ctypes.c_int, [vp, vp, vp, vp, i32, vp]
    lib.ubep_combine.restype, lib.ubep_combine.argtypes = ctypes.c_int, [vp, vp, vp, i32, vp, vp]
    lib.ubep_view.restype = ctypes.c_int
    lib.ubep_view.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_int64)]
    lib.ubep_status.restype, lib.ubep_status.argtypes = ctypes.c_int, [vp, ctypes.POINTER(i32)]
    lib.ubep_epoch.restype, lib.ubep_epoch.argtypes = u32, [vp]
    lib.ubep_launch_count.restype, lib.ubep_launch_count.argtypes = u64, []
    lib.ubep_debug_withhold_flag.restype, lib.ubep_debug_withhold_flag.argtypes = ctypes.c_int, [vp, i32]
    lib.ubep_debug_trace.restype, lib.ubep_debug_trace.argtypes = ctypes.c_int, [vp, i32]
    lib.ubep_debug_set_quant_warps.restype, lib.ubep_debug_set_quant_warps.argtypes = ctypes.c_int, [vp, i32]
    lib.ubep_debug_set_count_warps.restype, lib.ubep_debug_set_count_warps.argtypes = ctypes.c_int, [vp, i32]
    lib.ubep_debug_set_prefetch_rows.restype, lib.ubep_debug_set_prefetch_rows.argtypes = ctypes.c_int, [vp, i32]
    lib.ubep_debug_empty_launch.restype, lib.ubep_debug_empty_launch.argtypes = ctypes.c_int, [vp, i32, vp]
    lib.ubep_last_cuda_error.restype, lib.ubep_last_cuda_error.argtypes = ctypes.c_char_p, [vp]
    lib.ubep_strerror.restype, lib.ubep_strerror.argtypes = ctypes.c_char_p, [ctypes.c_int]
    lib.ubep_map_workers.restype = ctypes.c_int
    lib.ubep_map_workers.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.ubep_sync_wire_bytes.restype, lib.ubep_sync_wire_bytes.argtypes = ctypes.c_size_t, [cfgp]
    lib.ubep_sync_attach.restype, lib.ubep_sync_attach.argtypes = ctypes.c_int, [vp, vp, ctypes.c_size_t, vp]
    lib.ubep_dispatch_sync.restype = ctypes.c_int
    lib.ubep_dispatch_sync.argtypes = [vp, ctypes.c_int, vp, vp, vp, i32, vp]
    lib.ubep_sync_view.restype = ctypes.c_int
    lib.ubep_sync_view.argtypes = [vp, ctypes.c_int, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_int64)]
    lib.ubep_sync_scan_sentinel.restype = ctypes.c_int
    lib.ubep_sync_scan_sentinel.argtypes = [vp, vp, i32, ctypes.POINTER(ctypes.c_int64), vp]
    lib.ubep_set_peers.restype, lib.ubep_set_peers.argtypes = ctypes.c_int, [vp, i32, ctypes.POINTER(vp)]
    lib.ubep_dispatch_sharded.restype = ctypes.c_int
    lib.ubep_dispatch_sharded.argtypes = [vp, vp, vp, vp, i32, vp]
    lib.ubep_wait_arrivals.restype, lib.ubep_wait_arrivals.argtypes = ctypes.c_int, [vp, vp]
    lib.ubep_combine_sharded.restype = ctypes.c_int
    lib.ubep_combine_sharded.argtypes = [vp, vp, vp, i32, vp, vp]
    _lib = lib
    return lib


class UbepError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = load().ubep_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code}){' - ' + detail if detail else ''}")


def _check(code: int, where: str, buf=None):
    if code != UBEP_OK:
        detail = load().ubep_last_cuda_error(buf).decode() if (buf and code == UBEP_ERR_CUDA) else ""
        raise UbepError(code, where, detail)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


# ------------------------------------------------------------------ the C entry points

def ubep_strerror(code: int) -> str:
    return load().ubep_strerror(code).decode()


def ubep_buffer_bytes(cfg: ubep_config_t) -> int:
    return int(load().ubep_buffer_bytes(ctypes.byref(cfg)))


def ubep_buffer_create(cfg: ubep_config_t, arena: torch.Tensor) -> ctypes.c_void_p:
    out = ctypes.c_void_p()
    _check(load().ubep_buffer_create(ctypes.byref(cfg), _ptr(arena), arena.numel() * arena.element_size(),
                                     ctypes.byref(out)), "ubep_buffer_create")
    return out


def ubep_buffer_destroy(buf) -> None:
    _check(load().ubep_buffer_destroy(buf), "ubep_buffer_destroy")


def ubep_set_replicas(buf, phys: Optional[torch.Tensor], ncopies: Optional[torch.Tensor]) -> None:
    if phys is None:
        _check(load().ubep_set_replicas(buf, None, None, 0, 0), "ubep_set_replicas", buf)
        return
    assert phys.dtype == torch.int32 and ncopies.dtype == torch.int32 and phys.is_cuda
    _check(load().ubep_set_replicas(buf, _ptr(phys), _ptr(ncopies), phys.shape[0], phys.shape[1]),
           "ubep_set_replicas", buf)


def ubep_set_dest_order(buf, order) -> None:
    if order is None:
        _check(load().ubep_set_dest_order(buf, None), "ubep_set_dest_order", buf)
        return
    arr = (ctypes.c_int32 * len(order))(*[int(v) for v in order])
    _check(load().ubep_set_dest_order(buf, ctypes.cast(arr, ctypes.c_void_p)), "ubep_set_dest_order", buf)


def ubep_get_dispatch_layout(buf, topk_idx: torch.Tensor, T: int, num_tokens_per_rank, num_tokens_per_expert,
                             is_token_in_rank, stream=None) -> None:
    _check(load().ubep_get_dispatch_layout(buf, _ptr(topk_idx), T, _ptr(num_tokens_per_rank),
                                           _ptr(num_tokens_per_expert), _ptr(is_token_in_rank), _stream(stream)),
           "ubep_get_dispatch_layout", buf)


def ubep_get_dispatch_layout_static(topk_idx: torch.Tensor, T: int, topk: int, num_experts: int, num_ranks: int,
                                    num_tokens_per_rank, num_tokens_per_expert, is_token_in_rank, stream=None) -> None:
    """Counts through the entry point that needs no arena (see include/ubep.h): the caller passes only the
    routing table and the output tensors; scratch lives in a fixed array inside the library."""
    _check(load().ubep_get_dispatch_layout_static(_ptr(topk_idx), T, topk, num_experts, num_ranks,
                                                  _ptr(num_tokens_per_rank), _ptr(num_tokens_per_expert),
                                                  _ptr(is_token_in_rank), _stream(stream)),
           "ubep_get_dispatch_layout_static")


def ubep_dispatch(buf, x: torch.Tensor, topk_idx: torch.Tensor, topk_w: torch.Tensor, T: int, stream=None) -> None:
    _check(load().ubep_dispatch(buf, _ptr(x), _ptr(topk_idx), _ptr(topk_w), T, _stream(stream)),
           "ubep_dispatch", buf)


def ubep_combine(buf, y: torch.Tensor, topk_w: torch.Tensor, T: int, out: torch.Tensor, stream=None) -> None:
    _check(load().ubep_combine(buf, _ptr(y), _ptr(topk_w), T, _ptr(out), _stream(stream)), "ubep_combine", buf)


def ubep_map_workers(order: torch.Tensor, counts: torch.Tensor, n_workers: int, start_pos: torch.Tensor,
                     start_off: torch.Tensor, iters: Optional[torch.Tensor] = None, stream=None) -> None:
    assert order.dtype == torch.int32 and counts.dtype == torch.int32
    assert start_pos.dtype == torch.int32 and start_off.dtype == torch.int64
    _check(load().ubep_map_workers(_ptr(order), _ptr(counts), order.numel(), counts.numel(), n_workers,
                                   _ptr(start_pos), _ptr(start_off), _ptr(iters), _stream(stream)),
           "ubep_map_workers")


def ubep_view(buf, which: int):
    ptr = ctypes.c_void_p()
    shape = (ctypes.c_int64 * 4)()
    _check(load().ubep_view(buf, which, ctypes.byref(ptr), shape), "ubep_view", buf)
    return ptr.value, list(shape)


def ubep_status(buf) -> int:
    st = ctypes.c_int32(0)
    _check(load().ubep_status(buf, ctypes.byref(st)), "ubep_status", buf)
    return st.value


def ubep_epoch(buf) -> int:
    return int(load().ubep_epoch(buf))


def ubep_launch_count() -> int:
    return int(load().ubep_launch_count())


def ubep_debug_trace(buf, enable: bool) -> None:
    _check(load().ubep_debug_trace(buf, int(bool(enable))), "ubep_debug_trace", buf)


def ubep_debug_set_quant_warps(buf, n: int) -> None:
    _check(load().ubep_debug_set_quant_warps(buf, n), "ubep_debug_set_quant_warps", buf)


def ubep_debug_set_count_warps(buf, n: int) -> None:
    _check(load().ubep_debug_set_count_warps(buf, n), "ubep_debug_set_count_warps", buf)


def ubep_debug_set_prefetch_rows(buf, n: int) -> None:
    _check(load().ubep_debug_set_prefetch_rows(buf, n), "ubep_debug_set_prefetch_rows", buf)


def ubep_debug_empty_launch(buf, ahead: bool, stream=None) -> None:
    _check(load().ubep_debug_empty_launch(buf, int(bool(ahead)), _stream(stream)), "ubep_debug_empty_launch", buf)


def ubep_debug_withhold_flag(buf, chunk: int) -> None:
    _check(load().ubep_debug_withhold_flag(buf, chunk), "ubep_debug_withhold_flag", buf)


def ubep_sync_wire_bytes(cfg: ubep_config_t) -> int:
    return int(load().ubep_sync_wire_bytes(ctypes.byref(cfg)))


def ubep_sync_attach(buf, wire: torch.Tensor, stream=None) -> None:
    _check(load().ubep_sync_attach(buf, _ptr(wire), wire.numel() * wire.element_size(), _stream(stream)),
           "ubep_sync_attach", buf)


def ubep_dispatch_sync(buf, protocol: int, x: torch.Tensor, topk_idx: torch.Tensor, topk_w: torch.Tensor, T: int,
                       stream=None) -> None:
    _check(load().ubep_dispatch_sync(buf, protocol, _ptr(x), _ptr(topk_idx), _ptr(topk_w), T, _stream(stream)),
           "ubep_dispatch_sync", buf)


def ubep_sync_view(buf, which: int):
    ptr = ctypes.c_void_p()
    shape = (ctypes.c_int64 * 4)()
    _check(load().ubep_sync_view(buf, which, ctypes.byref(ptr), shape), "ubep_sync_view", buf)
    return ptr.value, list(shape)


def ubep_sync_scan_sentinel(buf, x: torch.Tensor, T: int, stream=None) -> int:
    n = ctypes.c_int64(0)
    _check(load().ubep_sync_scan_sentinel(buf, _ptr(x), T, ctypes.byref(n), _stream(stream)),
           "ubep_sync_scan_sentinel", buf)
    return n.value


def ubep_set_peers(buf, my_rank: int, peer_arena_ptrs) -> None:
    """peer_arena_ptrs: R integers, the device address of every rank's arena as this GPU sees it."""
    arr = (ctypes.c_void_p * len(peer_arena_ptrs))(*[int(v) for v in peer_arena_ptrs])
    _check(load().ubep_set_peers(buf, my_rank, arr), "ubep_set_peers", buf)


def ubep_dispatch_sharded(buf, x_local: torch.Tensor, topk_idx: torch.Tensor, topk_w: torch.Tensor, T: int,
                          stream=None) -> None:
    _check(load().ubep_dispatch_sharded(buf, _ptr(x_local), _ptr(topk_idx), _ptr(topk_w), T, _stream(stream)),
           "ubep_dispatch_sharded", buf)


def ubep_wait_arrivals(buf, stream=None) -> None:
    _check(load().ubep_wait_arrivals(buf, _stream(stream)), "ubep_wait_arrivals", buf)


def ubep_combine_sharded(buf, y_peers: torch.Tensor, topk_w: torch.Tensor, T: int, out_local: torch.Tensor,
                         stream=None) -> None:
    """y_peers: int64 device tensor of R addresses (every rank's expert-output buffer)."""
    assert y_peers.dtype == torch.int64 and y_peers.is_cuda
    _check(load().ubep_combine_sharded(buf, _ptr(y_peers), _ptr(topk_w), T, _ptr(out_local), _stream(stream)),
           "ubep_combine_sharded", buf)


# ------------------------------------------------------------------------ convenience

class Buffer:
    """An arena tensor plus the library handle laid out inside it."""

    def __init__(self, *, num_ranks, num_experts, hidden, topk, max_tokens, rows_per_rank_cap,
                 num_src_ranks=0, payload=0, dedup=0, device=0, pipeline=0, num_ctas=0, fill: Optional[int] = None,
                 arena: Optional[torch.Tensor] = None):
        self.cfg = ubep_config_t(num_ranks, num_experts, hidden, topk, max_tokens, rows_per_rank_cap,
                                 num_src_ranks, payload, dedup, device, pipeline, num_ctas)
        nbytes = ubep_buffer_bytes(self.cfg)
        if nbytes == 0:
            raise UbepError(UBEP_ERR_ARG, "ubep_buffer_bytes")
        dev = torch.device("cuda", device)
        if arena is not None:      # memory the caller obtained elsewhere (e.g. mapped for peer access)
            assert arena.dtype == torch.uint8 and arena.numel() >= nbytes and arena.is_cuda
        self.arena = arena if arena is not None else torch.empty(nbytes, dtype=torch.uint8, device=dev)
        if fill is not None:
            self.arena.fill_(fill)
        self.handle = ubep_buffer_create(self.cfg, self.arena)
        self.views = {}
        base = self.arena.data_ptr()
        for which, (name, dt) in enumerate(zip(VIEW_NAMES, _VIEW_DTYPES)):
            ptr, shape = ubep_view(self.handle, which)
            if not ptr:
                self.views[name] = None
                continue
            shape = [s for s in shape if s > 0]
            rank = {"recv_x": 3, "recv_scale": 3, "recv_topk_idx": 3, "recv_topk_w": 3}.get(name)
            if rank is None:
                rank = 1 if name in ("expert_offset", "num_tokens_per_expert", "num_rows_per_rank",
                                     "num_tokens_per_rank", "epoch", "shard_arrival") else 2
            shape = shape[:rank]
            n = 1
            for s in shape:
                n *= s
            esz = torch.empty(0, dtype=dt).element_size()
            self.views[name] = self.arena[ptr - base: ptr - base + n * esz].view(dt).view(shape)

    def __getattr__(self, name):
        views = self.__dict__.get("views", {})
        if name in views:
            return views[name]
        raise AttributeError(name)

    def set_replicas(self, phys, ncopies):
        self._phys, self._ncopies = phys, ncopies     # keep the tensors alive
        ubep_set_replicas(self.handle, phys, ncopies)

    def set_dest_order(self, order):
        ubep_set_dest_order(self.handle, order)

    def get_dispatch_layout(self, topk_idx, stream=None):
        T = topk_idx.shape[0]
        R, E = self.cfg.num_ranks, self.cfg.num_experts
        dev = self.arena.device
        npr = torch.empty(R, dtype=torch.int32, device=dev)
        npe = torch.empty(E, dtype=torch.int32, device=dev)
        itr = torch.empty((T, R), dtype=torch.uint8, device=dev)
        ubep_get_dispatch_layout(self.handle, topk_idx, T, npr, npe, itr, stream)
        return npr, npe, itr

    def dispatch(self, x, topk_idx, topk_w, stream=None):
        ubep_dispatch(self.handle, x, topk_idx, topk_w, x.shape[0], stream)

    def combine(self, y, topk_w, out=None, stream=None):
        T = topk_w.shape[0]
        if out is None:
            out = torch.empty((T, self.cfg.hidden), dtype=torch.bfloat16, device=self.arena.device)
        ubep_combine(self.handle, y, topk_w, T, out, stream)
        return out

    def status(self) -> int:
        return ubep_status(self.handle)

    def attach_sync(self, fill: Optional[int] = None, stream=None):
        """Allocates and attaches the wire buffer of the readiness-protocol dispatch."""
        nbytes = ubep_sync_wire_bytes(self.cfg)
        if nbytes == 0:
            raise UbepError(UBEP_ERR_ARG, "ubep_sync_wire_bytes")
        self.wire = torch.empty(nbytes, dtype=torch.uint8, device=self.arena.device)
        if fill is not None:
            self.wire.fill_(fill)
        ubep_sync_attach(self.handle, self.wire, stream)
        self.sync_views = {}
        base = self.wire.data_ptr()
        for which, (name, dt, rank) in enumerate(zip(SYNC_VIEW_NAMES, _SYNC_VIEW_DTYPES, _SYNC_VIEW_RANK)):
            ptr, shape = ubep_sync_view(self.handle, which)
            shape = shape[:rank]
            n = 1
            for s in shape:
                n *= s
            esz = torch.empty(0, dtype=dt).element_size()
            self.sync_views[name] = self.wire[ptr - base: ptr - base + n * esz].view(dt).view(shape)
        return self.sync_views

    def dispatch_sync(self, protocol, x, topk_idx, topk_w, stream=None):
        if isinstance(protocol, str):
            protocol = SYNC_NAMES[protocol]
        ubep_dispatch_sync(self.handle, protocol, x, topk_idx, topk_w, x.shape[0], stream)

    def scan_sentinel(self, x, stream=None) -> int:
        return ubep_sync_scan_sentinel(self.handle, x, x.shape[0], stream)

    def close(self):
        if getattr(self, "handle", None):
            ubep_buffer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
