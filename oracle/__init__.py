"""ctypes front end of the CPU oracle (``ubep_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline / reference legs.  The CUDA library and its Python
binding never import this package, and this package never imports them.

Every function takes and returns plain numpy arrays; argument marshalling is the
only thing done in Python.  The arithmetic lives in the C file, which cites the
passages of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ubep_oracle.c")
_LIB = os.path.join(_HERE, "libubep_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no fp contraction)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-std=c11", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
           "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    build()
    lib = ctypes.CDLL(_LIB)
    c_i32p = ctypes.POINTER(ctypes.c_int32)
    lib.orc_f32_to_e4m3.restype = ctypes.c_uint8
    lib.orc_f32_to_e4m3.argtypes = [ctypes.c_float]
    lib.orc_e4m3_to_f32.restype = ctypes.c_float
    lib.orc_e4m3_to_f32.argtypes = [ctypes.c_uint8]
    lib.orc_f32_to_bf16.restype = ctypes.c_uint16
    lib.orc_f32_to_bf16.argtypes = [ctypes.c_float]
    lib.orc_bf16_to_f32.restype = ctypes.c_float
    lib.orc_bf16_to_f32.argtypes = [ctypes.c_uint16]
    lib.orc_source_rank.restype = ctypes.c_int
    lib.orc_source_rank.argtypes = [ctypes.c_int] * 3
    for name in ("orc_resolve_ids", "orc_layout", "orc_fp8_quantize_row", "orc_dispatch",
                 "orc_combine", "orc_quaternary_search"):
        getattr(lib, name).restype = ctypes.c_int
    lib.orc_hop_distribution.restype = None
    lib.orc_stride_remap.restype = None
    lib.orc_equal_slices.restype = None
    _ = c_i32p
    _lib = lib
    return lib


def _p(a: Optional[np.ndarray]):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def host_cores() -> int:
    return len(os.sched_getaffinity(0))


# ------------------------------------------------------------------ scalars

def f32_to_e4m3(v: float) -> int:
    return int(_load().orc_f32_to_e4m3(ctypes.c_float(v)))


def e4m3_to_f32(c: int) -> float:
    return float(_load().orc_e4m3_to_f32(ctypes.c_uint8(c)))


def f32_to_bf16(v: float) -> int:
    return int(_load().orc_f32_to_bf16(ctypes.c_float(v)))


def bf16_to_f32(b: int) -> float:
    return float(_load().orc_bf16_to_f32(ctypes.c_uint16(b)))


def source_rank(t: int, T: int, S: int) -> int:
    return int(_load().orc_source_rank(t, T, S))


# ------------------------------------------------------------------- layout

def resolve_ids(topk_idx: np.ndarray, phys: np.ndarray, ncopies: np.ndarray) -> np.ndarray:
    T, k = topk_idx.shape
    E_log, C = phys.shape
    topk_idx = np.ascontiguousarray(topk_idx, np.int32)
    phys = np.ascontiguousarray(phys, np.int32)
    ncopies = np.ascontiguousarray(ncopies, np.int32)
    out = np.empty((T, k), np.int32)
    rc = _load().orc_resolve_ids(_p(topk_idx), T, k, _p(phys), _p(ncopies), E_log, C, _p(out))
    if rc:
        raise ValueError(f"orc_resolve_ids failed: {rc}")
    return out


@dataclass
class Layout:
    cnt: np.ndarray
    num_tokens_per_expert: np.ndarray
    is_token_in_rank: np.ndarray
    num_tokens_per_rank: np.ndarray
    expert_offset: np.ndarray
    src_offset: np.ndarray
    num_rows_per_rank: np.ndarray
    slot_row: np.ndarray
    expert_rows: Optional[np.ndarray]


def layout(ids: np.ndarray, E: int, R: int, S: int, dedup: int, er_cap: int = 0) -> Layout:
    """Counts, prefix-sum offsets and destination rows of every slot."""
    ids = np.ascontiguousarray(ids, np.int32)
    T, k = ids.shape
    cnt = np.empty((S, E), np.int32)
    npe = np.empty(E, np.int32)
    itr = np.empty((T, R), np.uint8)
    npr = np.empty(R, np.int32)
    eo = np.empty(E, np.int32)
    so = np.empty((S, E), np.int32)
    nrr = np.empty(R, np.int32)
    sr = np.empty((T, k), np.int32)
    er = None
    if dedup:
        if er_cap <= 0:
            er_cap = max(1, T * min(k, E // R))
        er = np.full((R, er_cap), -1, np.int32)
    rc = _load().orc_layout(_p(ids), T, k, E, R, S, int(dedup), _p(cnt), _p(npe), _p(itr), _p(npr),
                            _p(eo), _p(so), _p(nrr), _p(sr), _p(er), int(er_cap))
    if rc:
        raise ValueError(f"orc_layout failed: {rc}")
    return Layout(cnt, npe, itr, npr, eo, so, nrr, sr, er)


# --------------------------------------------------------------------- FP8

def fp8_quantize_rows(x_bf16: np.ndarray):
    """x_bf16: uint16 [n, H] -> (uint8 [n, H], float32 [n, H/128])."""
    x_bf16 = np.ascontiguousarray(x_bf16, np.uint16)
    n, H = x_bf16.shape
    q = np.empty((n, H), np.uint8)
    sc = np.empty((n, H // 128), np.float32)
    lib = _load()
    for i in range(n):
        rc = lib.orc_fp8_quantize_row(_p(x_bf16[i]), H, _p(q[i]), _p(sc[i]))
        if rc:
            raise ValueError(f"orc_fp8_quantize_row failed: {rc}")
    return q, sc


# ---------------------------------------------------------------- dispatch

@dataclass
class Recv:
    recv_x: np.ndarray           # uint8 [R, cap, rowB]
    recv_scale: Optional[np.ndarray]
    recv_src_idx: np.ndarray
    recv_weight: Optional[np.ndarray]
    recv_topk_idx: Optional[np.ndarray]
    recv_topk_w: Optional[np.ndarray]


def dispatch(x_bf16: np.ndarray, ids: np.ndarray, topk_w: np.ndarray, slot_row: np.ndarray,
             E: int, R: int, cap: int, payload: int, dedup: int, fill: int = 0xA5,
             num_threads: int = 1) -> Recv:
    """Fill the R receive regions; rows past a region's count keep the fill byte."""
    x_bf16 = np.ascontiguousarray(x_bf16, np.uint16)
    ids = np.ascontiguousarray(ids, np.int32)
    topk_w = np.ascontiguousarray(topk_w, np.float32)
    slot_row = np.ascontiguousarray(slot_row, np.int32)
    T, H = x_bf16.shape
    k = ids.shape[1]
    rowB = H if payload else 2 * H
    fill32 = np.frombuffer(bytes([fill] * 4), np.int32)[0]
    fillf = np.frombuffer(bytes([fill] * 4), np.float32)[0]
    recv_x = np.full((R, cap, rowB), fill, np.uint8)
    recv_scale = np.full((R, cap, H // 128), fillf, np.float32) if payload else None
    recv_src = np.full((R, cap), fill32, np.int32)
    recv_w = None if dedup else np.full((R, cap), fillf, np.float32)
    recv_ti = np.full((R, cap, k), fill32, np.int32) if dedup else None
    recv_tw = np.full((R, cap, k), fillf, np.float32) if dedup else None
    rc = _load().orc_dispatch(_p(x_bf16), _p(ids), _p(topk_w), _p(slot_row), T, H, k, E, R, cap,
                              int(payload), int(dedup), _p(recv_x), _p(recv_scale), _p(recv_src),
                              _p(recv_w), _p(recv_ti), _p(recv_tw), int(num_threads))
    if rc:
        raise ValueError(f"orc_dispatch failed: {rc}")
    return Recv(recv_x, recv_scale, recv_src, recv_w, recv_ti, recv_tw)


# ----------------------------------------------------------------- combine

def combine(y_bf16: np.ndarray, ids: np.ndarray, topk_w: np.ndarray, slot_row: np.ndarray,
            E: int, R: int, want_f64: bool = False, num_threads: int = 1):
    """y_bf16: uint16 [R, cap, H] -> (uint16 [T, H], float64 [T, H] or None)."""
    y_bf16 = np.ascontiguousarray(y_bf16, np.uint16)
    ids = np.ascontiguousarray(ids, np.int32)
    topk_w = np.ascontiguousarray(topk_w, np.float32)
    slot_row = np.ascontiguousarray(slot_row, np.int32)
    Ry, cap, H = y_bf16.shape
    assert Ry == R
    T, k = ids.shape
    out = np.empty((T, H), np.uint16)
    out64 = np.empty((T, H), np.float64) if want_f64 else None
    rc = _load().orc_combine(_p(y_bf16), _p(ids), _p(topk_w), _p(slot_row), T, H, k, E, R, cap,
                             _p(out), _p(out64), int(num_threads))
    if rc:
        raise ValueError(f"orc_combine failed: {rc}")
    return out, out64


# ------------------------------------------------------------- Algorithm 1

def quaternary_search(order: np.ndarray, counts: np.ndarray, target: int):
    """Returns (position in `order`, offset, iterations) or None if target is past the end."""
    order = np.ascontiguousarray(order, np.int32)
    counts = np.ascontiguousarray(counts, np.int32)
    pos = ctypes.c_int32(0)
    off = ctypes.c_int64(0)
    it = ctypes.c_int32(0)
    rc = _load().orc_quaternary_search(_p(order), _p(counts), len(order), ctypes.c_int64(target),
                                       ctypes.byref(pos), ctypes.byref(off), ctypes.byref(it))
    if rc:
        return None
    return pos.value, off.value, it.value


def stride_remap(n: int, rows: int) -> np.ndarray:
    order = np.empty(n, np.int32)
    _load().orc_stride_remap(n, rows, _p(order))
    return order


def equal_slices(total: int, workers: int) -> np.ndarray:
    begin = np.empty(workers + 1, np.int64)
    _load().orc_equal_slices(ctypes.c_int64(total), workers, _p(begin))
    return begin


def hop_distribution(order: np.ndarray, counts: np.ndarray, hop_of: np.ndarray, workers: int, n_hops: int) -> np.ndarray:
    """v[w][h]: tokens of hop class h in worker w's slice of the send sequence."""
    order = np.ascontiguousarray(order, np.int32)
    counts = np.ascontiguousarray(counts, np.int32)
    hop_of = np.ascontiguousarray(hop_of, np.int32)
    v = np.empty((workers, n_hops), np.int64)
    _load().orc_hop_distribution(_p(order), _p(counts), _p(hop_of), len(order), workers, n_hops, _p(v))
    return v


# ------------------------------------------------- Sec. 3.4: Data-as-Flag encodings

def tff_blocks(row_bytes: int, block_bytes: int, flag_bytes: int) -> int:
    n = int(_load().orc_tff_blocks(row_bytes, block_bytes, flag_bytes))
    if n < 0:
        raise ValueError("orc_tff_blocks: bad arguments")
    return n


def tff_pack(row: np.ndarray, block_bytes: int, flag_bytes: int, flag: int) -> np.ndarray:
    """DataBlocks (uint8 [blocks, block_bytes]) of one row of bytes."""
    row = np.ascontiguousarray(row).view(np.uint8).reshape(-1)
    nb = tff_blocks(row.size, block_bytes, flag_bytes)
    wire = np.empty((nb, block_bytes), np.uint8)
    _load().orc_tff_pack(_p(row), row.size, block_bytes, flag_bytes, ctypes.c_uint32(flag), _p(wire))
    return wire


def tff_unpack(wire: np.ndarray, row_bytes: int, block_bytes: int, flag_bytes: int, flag: int,
               row: Optional[np.ndarray] = None):
    """Returns (row bytes, number of DataBlocks that have not arrived)."""
    wire = np.ascontiguousarray(wire).view(np.uint8).reshape(-1)
    if row is None:
        row = np.zeros(row_bytes, np.uint8)
    assert row.dtype == np.uint8 and row.size == row_bytes and row.flags["C_CONTIGUOUS"]
    missing = int(_load().orc_tff_unpack(_p(wire), row_bytes, block_bytes, flag_bytes,
                                         ctypes.c_uint32(flag), _p(row)))
    if missing < 0:
        raise ValueError("orc_tff_unpack: bad arguments")
    return row, missing


def dc_checksum(rows: np.ndarray, block_bytes: int, marker_bytes: int) -> int:
    """Accumulated marker sum (mod 2^64) of rows given as a 2-D byte-viewable array."""
    rows = np.ascontiguousarray(rows)
    b = rows.view(np.uint8).reshape(rows.shape[0], -1) if rows.shape[0] else np.zeros((0, 8), np.uint8)
    fn = _load().orc_dc_checksum
    fn.restype = ctypes.c_uint64
    return int(fn(_p(b), ctypes.c_int64(b.shape[0]), int(b.shape[1]), ctypes.c_int64(b.shape[1]),
                  block_bytes, marker_bytes))


def sp_pending(data: np.ndarray, block_bytes: int, probe_bytes: int, sentinel: int) -> int:
    data = np.ascontiguousarray(data).view(np.uint8).reshape(-1)
    fn = _load().orc_sp_pending
    fn.restype = ctypes.c_int64
    return int(fn(_p(data), ctypes.c_int64(data.size), block_bytes, probe_bytes, ctypes.c_uint16(sentinel)))


def count_f32_rounding_to_bf16(code: int) -> int:
    fn = _load().orc_count_f32_rounding_to_bf16
    fn.restype = ctypes.c_int64
    return int(fn(ctypes.c_uint16(code)))
