"""Host-side helpers of the measurement modules, checked against the oracle without a GPU."""
import numpy as np
import pytest

import oracle
import bench_sweeps


@pytest.mark.parametrize("n,rows", [(16, 4), (72, 4), (32, 8), (13, 4), (7, 3), (5, 1), (4, 9)])
def test_stride_order_is_the_oracles_transposition(n, rows):
    got = bench_sweeps.stride_order(n, rows)
    assert np.array_equal(got, oracle.stride_remap(n, rows))
    assert sorted(got.tolist()) == list(range(n))


@pytest.mark.parametrize("row_bytes", [512, 528, 2048, 8192, 14336])
def test_wire_ratio_follows_the_oracles_block_count(row_bytes):
    blocks = oracle.tff_blocks(row_bytes, 16, 4)
    assert bench_sweeps.wire_ratio("tff", row_bytes) == pytest.approx(16 * blocks / row_bytes)
    for proto in ("sw", "dc", "sp"):
        assert bench_sweeps.wire_ratio(proto, row_bytes) == 1.0
