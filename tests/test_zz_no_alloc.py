"""The counts entry point that allocates nothing and takes no arena.

Some callers cannot allocate device memory at all: they run inside another component's
memory plan and are handed input and output tensors only, so they cannot give the library
an arena either.  `ubep_get_dispatch_layout_static` serves them from a fixed scratch array
inside the library.  This test calls it through the C ABI twice in a row (different routing
each time, so stale scratch from the first call would show) and requires exactly the output
of the ordinary entry point -- and, so that a fault shared by both would not pass, exactly the
counts of the CPU oracle.  It is collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W

pytestmark = pytest.mark.gpu


def _ordinary(cfg, wl):
    buf = B.Buffer(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T,
                   rows_per_rank_cap=8, num_src_ranks=cfg.S, payload=0, dedup=0, device=0)
    idx = torch.from_numpy(wl.topk_idx.astype(np.int32)).cuda()
    npr, npe, itr = buf.get_dispatch_layout(idx)
    torch.cuda.synchronize()
    return idx, npr, npe, itr


def test_static_scratch_entry_point_matches_the_ordinary_one_twice():
    assert torch.cuda.is_available()
    cases = [W.Config("na1", T=700, H=256, E=64, R=8, k=4, seed=31),
             W.Config("na2", T=333, H=256, E=288, R=72, k=8, seed=32)]
    for cfg in cases:
        wl = W.with_empty_slots(W.make_workload(cfg, with_x=False), 0.1, seed=cfg.seed)
        idx, npr, npe, itr = _ordinary(cfg, wl)
        got_r = torch.full((cfg.R,), -7, dtype=torch.int32, device="cuda")
        got_e = torch.full((cfg.E,), -7, dtype=torch.int32, device="cuda")
        got_m = torch.full((cfg.T, cfg.R), 9, dtype=torch.uint8, device="cuda")
        B.ubep_get_dispatch_layout_static(idx, cfg.T, cfg.k, cfg.E, cfg.R, got_r, got_e, got_m)
        torch.cuda.synchronize()
        assert torch.equal(got_r, npr) and torch.equal(got_e, npe) and torch.equal(got_m, itr)
        lay = oracle.layout(wl.topk_idx, cfg.E, cfg.R, cfg.S, 0)
        assert np.array_equal(got_r.cpu().numpy(), lay.num_tokens_per_rank)
        assert np.array_equal(got_e.cpu().numpy(), lay.num_tokens_per_expert)
        assert np.array_equal(got_m.cpu().numpy(), lay.is_token_in_rank)


def test_static_scratch_entry_point_rejects_sizes_beyond_its_array():
    idx = torch.zeros((4, 2), dtype=torch.int32, device="cuda")
    out = torch.zeros(2048, dtype=torch.int32, device="cuda")
    with pytest.raises(B.UbepError) as ei:       # 1020 + 12 bins > 1024
        B.ubep_get_dispatch_layout_static(idx, 4, 2, 1020, 12, out, out, None)
    assert ei.value.code == B.UBEP_ERR_ARG
    with pytest.raises(B.UbepError):             # E % R != 0
        B.ubep_get_dispatch_layout_static(idx, 4, 2, 10, 4, out, out, None)
