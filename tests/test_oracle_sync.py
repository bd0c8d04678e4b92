"""Pins of the oracle's Data-as-Flag encodings (Sec. 3.4 of the paper): the paper's own
figures, a hand-worked fixture, numpy slicing written independently of the C code,
invariants, and exhaustive walks where the space is small."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "tff_handworked.txt")


def read_golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            key, *vals = line.split()
            out[key] = [int(v, 0) for v in vals]
    return out


def numpy_tff(row, block, flag_bytes, flag):
    """Independent packer: pad the row to whole payloads, prepend the flag column."""
    P = block - flag_bytes
    nb = -(-row.size // P)
    padded = np.zeros(nb * P, np.uint8)
    padded[:row.size] = row
    fl = np.frombuffer(np.uint32(flag).tobytes() * (flag_bytes // 4), np.uint8)
    return np.concatenate([np.tile(fl, (nb, 1)), padded.reshape(nb, P)], axis=1)


def test_tff_handworked_fixture():
    g = read_golden()
    row = np.array(g["row"], np.uint8)
    wire = oracle.tff_pack(row, g["block_bytes"][0], g["flag_bytes"][0], g["flag"][0])
    assert wire.shape == (g["blocks"][0], g["block_bytes"][0])
    assert wire.reshape(-1).tolist() == g["wire"]
    # checksum markers of the same row: one whole word in block 0, none in the cut-short block 1
    assert oracle.dc_checksum(row.reshape(1, -1), g["dc_block"][0], g["dc_marker"][0]) == g["dc_sum"][0]


def test_tff_paper_figures():
    g = read_golden()
    blk, fl = g["paper_block"][0], g["paper_flag"][0]
    assert blk - fl == g["paper_payload"][0]
    assert oracle.tff_blocks(g["paper_row"][0], blk, fl) == g["paper_blocks"][0]
    # payload efficiency of the paper's DataBlock and of 16-byte blocks with a 4-byte flag
    assert (blk - fl) / blk == 0.9375
    assert oracle.tff_blocks(14328, 16, 4) * 16 == 14328 // 12 * 16
    assert oracle.tff_blocks(14336, 16, 4) == 1195          # 14336 = 1194 * 12 + 8
    with pytest.raises(ValueError):
        oracle.tff_blocks(64, 16, 16)
    with pytest.raises(ValueError):
        oracle.tff_blocks(64, 16, 3)


@pytest.mark.parametrize("row_bytes,block,flag_bytes", [(24, 16, 4), (512, 16, 4), (14336, 16, 4),
                                                        (14336, 512, 32), (8192, 512, 32), (40, 32, 8), (8, 16, 4)])
def test_tff_pack_matches_numpy_and_round_trips(row_bytes, block, flag_bytes):
    rng = np.random.Generator(np.random.PCG64(row_bytes * 131 + block))
    row = rng.integers(0, 256, row_bytes, dtype=np.uint8)
    flag = int(rng.integers(1, 2**32))
    wire = oracle.tff_pack(row, block, flag_bytes, flag)
    assert np.array_equal(wire, numpy_tff(row, block, flag_bytes, flag))
    back, missing = oracle.tff_unpack(wire, row_bytes, block, flag_bytes, flag)
    assert missing == 0 and np.array_equal(back, row)


def test_tff_unpack_sees_missing_blocks():
    rng = np.random.Generator(np.random.PCG64(77))
    row = rng.integers(0, 256, 480, dtype=np.uint8)
    wire = oracle.tff_pack(row, 16, 4, 9)
    stale = wire.copy()
    stale[[3, 17], 0] = 8                    # two blocks still carry the previous call's flag
    stale[5, 3] ^= 0x80                      # one block with a torn flag field
    before = np.full(480, 0xEE, np.uint8)
    back, missing = oracle.tff_unpack(stale, 480, 16, 4, 9, before.copy())
    assert missing == 3
    gone = np.zeros(480, bool)
    for b in (3, 5, 17):
        gone[b * 12:(b + 1) * 12] = True
    assert np.array_equal(back[~gone], row[~gone]) and np.all(back[gone] == 0xEE)
    # nothing has arrived under another flag value
    _, missing = oracle.tff_unpack(wire, 480, 16, 4, 10)
    assert missing == wire.shape[0]


def numpy_dc(rows, block, marker):
    if rows.shape[0] == 0:
        return 0
    rows = rows.view(np.uint8).reshape(rows.shape[0], -1)
    total = 0
    for b0 in range(0, rows.shape[1], block):
        m = rows[:, b0:b0 + min(marker, block)]
        m = m[:, :m.shape[1] // 8 * 8]
        if m.shape[1]:
            words = np.ascontiguousarray(m).view("<u8")
            total += int(words.astype(object).sum())
    return total % 2**64


@pytest.mark.parametrize("n_rows,row_bytes,block,marker", [(1, 512, 512, 32), (7, 14336, 512, 32), (33, 8192, 512, 32),
                                                           (5, 520, 512, 32), (9, 256, 64, 16), (0, 512, 512, 32)])
def test_dc_checksum_matches_numpy(n_rows, row_bytes, block, marker):
    rng = np.random.Generator(np.random.PCG64(n_rows * 7 + row_bytes))
    rows = rng.integers(0, 256, (n_rows, row_bytes), dtype=np.uint8)
    assert oracle.dc_checksum(rows, block, marker) == numpy_dc(rows, block, marker)


def test_dc_checksum_invariants():
    rng = np.random.Generator(np.random.PCG64(5))
    rows = rng.integers(0, 256, (16, 1024), dtype=np.uint8)
    base = oracle.dc_checksum(rows, 512, 32)
    # rows may arrive in any order; the sum of two batches is the sum of the sums
    assert oracle.dc_checksum(rows[rng.permutation(16)], 512, 32) == base
    assert (oracle.dc_checksum(rows[:5], 512, 32) + oracle.dc_checksum(rows[5:], 512, 32)) % 2**64 == base
    # a marker byte changes it by exactly its place value, any other byte does not
    m = rows.copy()
    m[3, 512 + 9] = (int(m[3, 512 + 9]) + 1) % 256
    delta = (oracle.dc_checksum(m, 512, 32) - base) % 2**64
    assert delta in ((1 << 8) % 2**64, (-(255 << 8)) % 2**64)
    o = rows.copy()
    o[3, 40] ^= 0xFF
    assert oracle.dc_checksum(o, 512, 32) == base
    # wrap-around: 2^63 + 2^63 = 0
    two = np.zeros((2, 8), np.uint8)
    two[:, 7] = 0x80
    assert oracle.dc_checksum(two, 8, 8) == 0


def test_sp_pending_counts_blocks_that_show_the_sentinel():
    buf = np.full(16 * 10, 0xFF, np.uint8)
    assert oracle.sp_pending(buf, 16, 16, 0xFFFF) == 10
    buf[16 * 4 + 15] = 0xFE                   # last probed byte of block 4
    buf[16 * 7] = 0                           # first byte of block 7
    assert oracle.sp_pending(buf, 16, 16, 0xFFFF) == 8
    assert oracle.sp_pending(buf, 16, 8, 0xFFFF) == 9    # an 8-byte probe does not see byte 15
    # the paper's instance: 32 probed bytes per 512-byte DataBlock
    big = np.zeros(512 * 3, np.uint8)
    big[512:512 + 32] = np.tile(np.array([0x34, 0x12], np.uint8), 16)
    assert oracle.sp_pending(big, 512, 32, 0x1234) == 1
    big[512 + 31] = 0
    assert oracle.sp_pending(big, 512, 32, 0x1234) == 0


def test_sp_collision_rate_of_a_two_byte_probe_is_one_in_2_16():
    # Sec. 3.4 gives 2^-(8 * probe bytes) under uniform data; walked in full for 2 bytes
    every = np.arange(65536, dtype="<u2")
    for sentinel in (0xFFFF, 0x7FC0, 0x0000, 0x1234):
        assert oracle.sp_pending(every, 2, 2, sentinel) == 1


def test_sentinel_code_is_never_the_rounding_of_a_number():
    # every fp32 bit pattern that is not NaN, rounded to bf16: none gives the all-ones code,
    # while an ordinary code collects its 2^16 + 1 neighbours (ties to even)
    assert oracle.count_f32_rounding_to_bf16(0xFFFF) == 0
    assert oracle.count_f32_rounding_to_bf16(0x3F80) == 65537
