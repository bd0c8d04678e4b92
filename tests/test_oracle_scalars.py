"""Pins for the oracle's scalar converters (bf16 and FP8 e4m3).

The e4m3 converter is pinned by an exhaustive nearest-code search with exact rational
arithmetic (a different algorithm from the converter's scale-and-round), by torch's CPU
float8 cast for in-range values, and by the format's fixed points.
"""
from fractions import Fraction

import numpy as np
import pytest
import torch


def _decode_table():
    """Exact values of the 2 x 127 finite e4m3fn codes (bias 7, subnormal step 2^-9)."""
    vals = {}
    for code in range(256):
        e, m = (code >> 3) & 15, code & 7
        if e == 15 and m == 7:
            continue
        mag = Fraction(m, 8) * Fraction(1, 64) if e == 0 else Fraction(8 + m, 8) * Fraction(2) ** (e - 7)
        vals[code] = -mag if code & 0x80 else mag
    return vals


TABLE = _decode_table()
POS = sorted((v, c) for c, v in TABLE.items() if c < 0x80)


def brute_nearest(v: float) -> int:
    """Nearest finite code by exhaustive search; ties to the even mantissa; saturating."""
    if v != v:
        return 0x7F
    sign = 0x80 if np.signbit(np.float32(v)) else 0
    if abs(v) == float("inf"):
        return sign | 0x7E
    a = abs(Fraction(float(v)))
    if a > 448:
        return sign | 0x7E
    best = None
    for val, code in POS:
        d = abs(val - a)
        if best is None or d < best[0] or (d == best[0] and (code & 1) == 0 and (best[1] & 1) == 1):
            best = (d, code)
    return sign | best[1]


def _sweep_values():
    vals = [0.0, -0.0, 448.0, -448.0, 449.0, 463.9, 464.0, 465.0, 1e9, -1e9, float("inf"),
            float("-inf"), 2.0 ** -9, 2.0 ** -10, 2.0 ** -10 * 1.0001, 2.0 ** -11, 1e-30, 2.0 ** -6]
    pos = [float(v) for v, _ in POS]
    for a, b in zip(pos[:-1], pos[1:]):
        mid = (a + b) / 2
        vals += [a, mid, float(np.nextafter(np.float32(mid), np.float32(np.inf))),
                 float(np.nextafter(np.float32(mid), np.float32(-np.inf))), -mid]
    rng = np.random.default_rng(7)
    vals += list(rng.standard_normal(2000).astype(np.float32) * 100)
    vals += list(rng.standard_normal(2000).astype(np.float32) * 0.01)
    return [float(np.float32(v)) for v in vals]


def test_e4m3_matches_exhaustive_nearest_code_search(orc):
    for v in _sweep_values():
        assert orc.f32_to_e4m3(v) == brute_nearest(v), v


def test_e4m3_fixed_points(orc):
    assert orc.f32_to_e4m3(float("nan")) == 0x7F
    assert orc.f32_to_e4m3(0.0) == 0x00 and orc.f32_to_e4m3(-0.0) == 0x80
    assert orc.f32_to_e4m3(448.0) == 0x7E and orc.f32_to_e4m3(-448.0) == 0xFE
    assert orc.f32_to_e4m3(1.0) == 0x38
    assert orc.f32_to_e4m3(2.0 ** -9) == 0x01      # smallest subnormal
    assert orc.f32_to_e4m3(2.0 ** -10) == 0x00     # tie between 0 and 2^-9 -> even (0)
    assert orc.f32_to_e4m3(3 * 2.0 ** -10) == 0x02  # tie between codes 1 and 2 -> even
    for code, val in TABLE.items():                 # every code is a fixed point
        if val != 0:
            assert orc.f32_to_e4m3(float(val)) == code
        assert Fraction(orc.e4m3_to_f32(code)) == val


def test_e4m3_agrees_with_torch_cpu_cast_in_range(orc):
    rng = np.random.default_rng(11)
    v = np.concatenate([rng.standard_normal(4000) * 50, rng.standard_normal(4000) * 0.02,
                        rng.uniform(-448, 448, 4000)]).astype(np.float32)
    v = v[np.abs(v) <= 448]
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([orc.f32_to_e4m3(float(x)) for x in v], np.uint8)
    assert np.array_equal(got, ref)


def test_bf16_rne_agrees_with_torch_cpu(orc):
    rng = np.random.default_rng(3)
    v = (rng.standard_normal(5000) * 10 ** rng.uniform(-3, 3, 5000)).astype(np.float32)
    ties = (np.arange(0x3F80, 0x3F80 + 64, dtype=np.uint32) << 16 | 0x8000).view(np.float32)
    v = np.concatenate([v, ties, -ties, np.array([0.0, -0.0, np.inf, -np.inf], np.float32)])
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([orc.f32_to_bf16(float(x)) for x in v], np.uint16)
    assert np.array_equal(got, ref)
    for b in (0x3F80, 0xC000, 0x0001, 0x7F7F):
        assert orc.f32_to_bf16(orc.bf16_to_f32(b)) == b
    assert orc.bf16_to_f32(0x3F80) == 1.0 and orc.bf16_to_f32(0xC000) == -2.0


def test_workload_bf16_generator_agrees_with_torch():
    from paper_2607_06202_b200 import workload as W
    rng = np.random.default_rng(5)
    v = rng.standard_normal(10000).astype(np.float32)
    ref = torch.from_numpy(v).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(W.f32_to_bf16_bits(v), ref)
    assert np.array_equal(W.bf16_bits_to_f32(ref), torch.from_numpy(v).to(torch.bfloat16).float().numpy())
