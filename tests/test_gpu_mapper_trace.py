"""GPU parity of the scheduler's load partition (Algorithm 1) against the oracle, and the
library's phase tracing."""
import numpy as np
import pytest
import torch

import harness as Hn
import oracle
from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,workers,zero_frac", [(1, 1, 0.0), (5, 3, 0.0), (16, 48, 0.3), (256, 148, 0.0),
                                                 (288, 148, 0.2), (1300, 296, 0.5), (37, 7, 0.9)])
def test_map_workers_matches_the_oracle_search(n, workers, zero_frac):
    rng = np.random.default_rng(n * 31 + workers)
    counts = rng.integers(1, 200, n).astype(np.int32)
    counts[rng.random(n) < zero_frac] = 0
    order = oracle.stride_remap(n, 8) if n >= 8 else np.arange(n, dtype=np.int32)
    total = int(counts.sum())
    begin = oracle.equal_slices(total, workers)
    pos = torch.full((workers + 1,), -5, dtype=torch.int32, device="cuda")
    off = torch.full((workers + 1,), -5, dtype=torch.int64, device="cuda")
    its = torch.full((workers + 1,), -5, dtype=torch.int32, device="cuda")
    B.ubep_map_workers(torch.from_numpy(order).cuda(), torch.from_numpy(counts).cuda(), workers, pos, off, its)
    torch.cuda.synchronize()
    pos, off, its = pos.cpu().numpy(), off.cpu().numpy(), its.cpu().numpy()
    for w in range(workers + 1):
        ref = oracle.quaternary_search(order, counts, int(begin[w]))
        if ref is None:
            assert pos[w] == n and off[w] == 0
        else:
            assert (pos[w], off[w], its[w]) == ref, (w, pos[w], off[w], its[w], ref)
    sizes = np.diff(begin)
    assert sizes.max() - sizes.min() <= 1                   # the paper's balance guarantee


def test_map_workers_on_a_dispatch_count_table(workloads):
    """Counts of a real layout, experts visited in the stride-remapped order."""
    wl = workloads("decode")
    cfg = wl.cfg
    lay = oracle.layout(wl.topk_idx, cfg.E, cfg.R, cfg.S, 0)
    order = oracle.stride_remap(cfg.E, 148)
    counts = lay.num_tokens_per_expert.astype(np.int32)
    pos = torch.empty(149, dtype=torch.int32, device="cuda")
    off = torch.empty(149, dtype=torch.int64, device="cuda")
    B.ubep_map_workers(torch.from_numpy(order).cuda(), torch.from_numpy(counts).cuda(), 148, pos, off)
    cum = np.concatenate([[0], np.cumsum(counts[order].astype(np.int64))])
    start = cum[pos.cpu().numpy()[:148]] + off.cpu().numpy()[:148]
    assert np.array_equal(start, oracle.equal_slices(int(cum[-1]), 148)[:148])


def test_phase_trace_is_monotone_per_cta():
    cfg = W.Config("tr", T=2000, H=512, E=64, R=8, k=4, seed=5)
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap, pipeline=B.UBEP_PIPELINE_FUSED)
    x, idx, w, _, _ = Hn.device_inputs(wl)
    B.ubep_debug_trace(buf.handle, True)
    buf.dispatch(x, idx, w)
    Hn.check_dispatch(buf, wl, lay, cap, recv)
    tr = buf.trace.cpu().numpy()
    # start <= counted <= all-offsets-seen <= rows assigned <= movers released <= copies done <= end
    for a, b in [(0, 1), (1, 4), (4, 5), (5, 6), (6, 9), (9, 10)]:
        assert np.all(tr[:, a] <= tr[:, b]), (a, b)
    assert (tr[:, 10] - tr[:, 0]).max() < 5e6      # a dispatch of this size takes far less than 5 ms
    B.ubep_debug_trace(buf.handle, False)
