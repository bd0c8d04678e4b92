"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the
header declares, and rejects bad configurations without launching anything."""
import os
import re

import pytest

from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.load()


def test_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "ubep.h")).read()
    declared = sorted(set(re.findall(r"\b(ubep_[a-z_]+)\s*\(", header)))
    assert declared, "no declarations found"
    assert sorted(B.EXPORTS) == declared
    for name in declared:
        assert hasattr(lib, name), name


def test_header_is_plain_c():
    import subprocess
    src = '#include "ubep.h"\nint main(void){ ubep_config_t c; (void)c; return UBEP_OK; }\n'
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-fsyntax-only", "-I", os.path.join(ROOT, "include"),
                    "-x", "c", "-"], input=src.encode(), check=True)


def test_strerror_and_codes(lib):
    assert B.ubep_strerror(0) == "ok"
    for code in (B.UBEP_ERR_ARG, B.UBEP_ERR_CUDA, B.UBEP_ERR_CAPACITY, B.UBEP_ERR_TIMEOUT,
                 B.UBEP_ERR_BAD_INDEX, B.UBEP_ERR_ARENA, B.UBEP_ERR_CHECKSUM):
        assert B.ubep_strerror(code) not in ("ok", "unknown error")
    assert B.ubep_strerror(-99) == "unknown error"


def _cfg(**kw):
    base = dict(num_ranks=4, num_experts=16, hidden=256, topk=2, max_tokens=128, rows_per_rank_cap=128,
                num_src_ranks=0, payload=0, dedup=0, device=0, pipeline=0, num_ctas=0)
    base.update(kw)
    return B.ubep_config_t(*[base[n] for n, _ in B.ubep_config_t._fields_])


def test_buffer_bytes_validates_config(lib):
    assert B.ubep_buffer_bytes(_cfg()) > 4 * 128 * 512
    assert B.ubep_buffer_bytes(_cfg(num_experts=18)) == 0          # E % R != 0
    assert B.ubep_buffer_bytes(_cfg(hidden=100)) == 0              # H % 8 != 0
    assert B.ubep_buffer_bytes(_cfg(hidden=192, payload=1)) == 0   # FP8 needs H % 128 == 0
    assert B.ubep_buffer_bytes(_cfg(topk=33)) == 0
    assert B.ubep_buffer_bytes(_cfg(topk=0)) == 0
    assert B.ubep_buffer_bytes(_cfg(dedup=2)) == 0
    assert B.ubep_buffer_bytes(_cfg(pipeline=9)) == 0
    assert B.ubep_buffer_bytes(_cfg(max_tokens=0)) == 0
    # FP8 rows are half the size of bf16 rows
    big = dict(hidden=1024, rows_per_rank_cap=4096)
    assert B.ubep_buffer_bytes(_cfg(payload=1, **big)) < B.ubep_buffer_bytes(_cfg(**big))
    # a decode-sized arena is dominated by the receive regions
    n = B.ubep_buffer_bytes(_cfg(num_ranks=32, num_experts=256, hidden=7168, topk=8, max_tokens=512,
                                 rows_per_rank_cap=256, dedup=1))
    assert 32 * 256 * 14336 < n < 32 * 256 * 14336 * 1.05


def test_null_arguments_are_rejected_without_a_gpu(lib):
    import ctypes
    out = ctypes.c_void_p()
    cfg = _cfg()
    assert lib.ubep_buffer_create(ctypes.byref(cfg), None, 1 << 30, ctypes.byref(out)) == B.UBEP_ERR_ARG
    assert lib.ubep_buffer_destroy(None) == B.UBEP_ERR_ARG
    assert lib.ubep_dispatch(None, None, None, None, 0, None) == B.UBEP_ERR_ARG
    assert lib.ubep_combine(None, None, None, 0, None, None) == B.UBEP_ERR_ARG
    assert lib.ubep_status(None, None) == B.UBEP_ERR_ARG
    assert lib.ubep_epoch(None) == 0
    assert lib.ubep_launch_count() == 0
    assert lib.ubep_sync_attach(None, None, 0, None) == B.UBEP_ERR_ARG
    assert lib.ubep_dispatch_sync(None, 0, None, None, None, 0, None) == B.UBEP_ERR_ARG
    assert lib.ubep_sync_view(None, 0, None, None) == B.UBEP_ERR_ARG
    assert lib.ubep_sync_scan_sentinel(None, None, 0, None, None) == B.UBEP_ERR_ARG
    assert lib.ubep_set_peers(None, 0, None) == B.UBEP_ERR_ARG
    assert lib.ubep_dispatch_sharded(None, None, None, None, 0, None) == B.UBEP_ERR_ARG
    assert lib.ubep_wait_arrivals(None, None) == B.UBEP_ERR_ARG
    assert lib.ubep_combine_sharded(None, None, None, 0, None, None) == B.UBEP_ERR_ARG


def test_wire_bytes_of_the_readiness_protocols(lib):
    # decode-sized: Token-Flag blocks (16 bytes per 12 of payload) plus the sentinel wire
    kw = dict(num_ranks=32, num_experts=256, hidden=7168, topk=8, max_tokens=512, rows_per_rank_cap=256, dedup=1)
    rows = 32 * 256
    tff_row = 16 * -(-14336 // 12)
    n = B.ubep_sync_wire_bytes(_cfg(**kw))
    assert rows * (tff_row + 14336) < n < rows * (tff_row + 14336) * 1.01
    # FP8 rows: payload plus scales, 7168 + 224 bytes
    n8 = B.ubep_sync_wire_bytes(_cfg(payload=1, **kw))
    w8 = 7168 + 224
    assert rows * (16 * -(-w8 // 12) + w8) < n8 < rows * (16 * -(-w8 // 12) + w8) * 1.01
    assert B.ubep_sync_wire_bytes(_cfg(num_experts=18)) == 0
    assert (B.UBEP_SYNC_BLOCK_BYTES - B.UBEP_SYNC_FLAG_BYTES) / B.UBEP_SYNC_BLOCK_BYTES == 0.75
    header = open(os.path.join(ROOT, "include", "ubep.h")).read()
    for name in ("UBEP_SYNC_BLOCK_BYTES", "UBEP_SYNC_FLAG_BYTES", "UBEP_SYNC_DC_BLOCK_BYTES",
                 "UBEP_SYNC_DC_MARKER_BYTES"):
        assert int(re.search(rf"#define {name} (\d+)", header).group(1)) == getattr(B, name)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libubep.so"))
    with pytest.raises(RuntimeError, match="missing"):
        B.load()
