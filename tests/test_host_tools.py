"""Host-side helpers of the measurement modules, checked against the oracle without a GPU."""
import numpy as np
import pytest

import oracle
import bench
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


@pytest.mark.parametrize("steps", [1, 3, 20, 256, 257, 1000])
def test_a_timed_block_holds_exactly_the_steps_asked_for(steps):
    g, full, rem = bench.block_plan(steps)
    assert g * full + rem == steps and 1 <= g <= bench.MAX_GRAPH_STEPS and 0 <= rem < g


def test_block_count_and_summary():
    assert bench.blocks_needed(0.6) == 500            # 0.3 s of 0.6 ms blocks
    assert bench.blocks_needed(100.0) == bench.MIN_BLOCKS
    assert bench.blocks_needed(1e-4) == 4000          # capped
    s = bench.summarize_blocks([2.0, 4.0, 3.0], steps=2)
    assert s["median_us"] == pytest.approx(1500.0) and s["min_us"] == pytest.approx(1000.0) and s["blocks"] == 3


def test_traffic_file_carries_the_commit_it_was_captured_at():
    traffic, commit, _ = bench.read_traffic("decode", "dispatch")
    assert traffic is not None and traffic > 0
    assert commit is not None and len(commit) >= 7
