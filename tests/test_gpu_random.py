"""Seeded random sweep over shapes, payloads, schedules, chunk counts, destination tables and empty
slots: every case through the C ABI against the oracle (dispatch bit for bit, combine within the
tolerance), also through the readiness protocols and the sharded path."""
import numpy as np
import pytest
import torch

from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu


def draw(rng):
    R = int(rng.choice([1, 2, 3, 4, 8, 16, 32]))
    L = int(rng.choice([1, 2, 3, 4, 8]))
    E = R * L
    k = int(rng.integers(1, min(8, E) + 1))
    payload = int(rng.integers(0, 2))
    H = int(rng.choice([128, 256, 512, 1024])) if payload else int(rng.choice([8, 64, 136, 264, 512, 1032]))
    T = int(rng.choice([1, 5, 33, 100, 257, 700, 1500, 3000]))
    pipeline = int(rng.integers(0, 4))
    if pipeline == B.UBEP_PIPELINE_LOCAL and T * k > 8192:
        pipeline = B.UBEP_PIPELINE_AUTO
    ctas = int(rng.choice([0, 0, 0, 1, 7, 40, 148]))
    if T * k > 2000 and ctas in (1, 7):
        ctas = 40                      # a chunk's bookkeeping has to fit in shared memory
    cfg = W.Config("random", T=T, H=H, E=E, R=R, k=k, payload=payload, dedup=int(rng.integers(0, 2)),
                   seed=int(rng.integers(1 << 30)), routing=str(rng.choice(["gauss", "zipf"])))
    wl = W.make_workload(cfg)
    if rng.random() < 0.3:
        wl = W.with_empty_slots(wl, 0.2, int(rng.integers(1 << 30)))
    order = [int(v) for v in rng.permutation(R)] if rng.random() < 0.3 else None
    return cfg, wl, pipeline, ctas, order


@pytest.mark.parametrize("seed", range(6))
def test_random_cases(seed):
    rng = np.random.default_rng(9000 + seed)
    for _ in range(8):
        cfg, wl, pipeline, ctas, order = draw(rng)
        Hn.run_case(wl, pipeline=pipeline, num_ctas=ctas, dest_order=order)
        ids, lay, cap, recv = Hn.oracle_reference(wl)
        x, idx, w, _, _ = Hn.device_inputs(wl)
        buf = Hn.make_buffer(cfg, cap, num_ctas=ctas)
        buf.attach_sync()
        for proto in ("sw", "tff", "dc", "sp"):
            buf.recv_x.fill_(Hn.FILL)
            buf.dispatch_sync(proto, x, idx, w)
            Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
        if cfg.R <= 8:
            ranks = [Hn.make_buffer(cfg, cap, num_ctas=ctas) for _ in range(cfg.R)]
            ptrs = [b.arena.data_ptr() for b in ranks]
            for r, b in enumerate(ranks):
                B.ubep_set_peers(b.handle, r, ptrs)
            for s, b in enumerate(ranks):
                B.ubep_dispatch_sharded(b.handle, x[s * cfg.T // cfg.R:(s + 1) * cfg.T // cfg.R].contiguous(), idx, w,
                                        cfg.T)
            for r, b in enumerate(ranks):
                B.ubep_wait_arrivals(b.handle)
                assert b.status() == 0
                assert torch.equal(b.recv_x[r].cpu(), torch.from_numpy(recv.recv_x[r])), f"sharded region {r}: {cfg}"
