"""Helpers shared by the GPU parity tests, the smoke check and the benchmark: run one workload
through the C-ABI library and through the CPU oracle and compare every output."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W

FILL = 0xA5


def oracle_reference(wl: W.Workload, cap: int | None = None, num_threads: int = 1):
    """Everything the oracle says about a workload: resolved ids, layout, receive regions."""
    cfg = wl.cfg
    ids = wl.topk_idx if wl.phys is None else oracle.resolve_ids(wl.topk_idx, wl.phys, wl.ncopies)
    lay = oracle.layout(ids, cfg.E, cfg.R, cfg.S, cfg.dedup,
                        er_cap=(cap * min(cfg.k, cfg.L) if (cap and cfg.dedup) else 0))
    if cap is None:
        cap = W.round_up(max(1, int(lay.num_rows_per_rank.max())), 128)
        if cfg.dedup:
            lay = oracle.layout(ids, cfg.E, cfg.R, cfg.S, cfg.dedup, er_cap=cap * min(cfg.k, cfg.L))
    recv = oracle.dispatch(wl.x, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, cap, cfg.payload, cfg.dedup,
                           fill=FILL, num_threads=num_threads)
    return ids, lay, cap, recv


def make_buffer(cfg: W.Config, cap: int, pipeline: int = 0, num_ctas: int = 0, max_tokens: int | None = None,
                fill=FILL) -> B.Buffer:
    return B.Buffer(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k,
                    max_tokens=max_tokens or max(cfg.T, 1), rows_per_rank_cap=cap, num_src_ranks=cfg.S,
                    payload=cfg.payload, dedup=cfg.dedup, device=0, pipeline=pipeline, num_ctas=num_ctas,
                    fill=fill)


def to_dev(a: np.ndarray, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is torch.bfloat16:
        t = t.view(torch.int16).view(torch.bfloat16)
    return t.cuda()


def device_inputs(wl: W.Workload):
    x = to_dev(wl.x, torch.bfloat16)
    idx = to_dev(wl.topk_idx.astype(np.int32))
    w = to_dev(wl.topk_w.astype(np.float32))
    phys = ncopies = None
    if wl.phys is not None:
        phys, ncopies = to_dev(wl.phys.astype(np.int32)), to_dev(wl.ncopies.astype(np.int32))
    return x, idx, w, phys, ncopies


def _eq(name, got: torch.Tensor, want: np.ndarray):
    want_t = torch.from_numpy(np.ascontiguousarray(want)).to(got.device)
    if want_t.dtype != got.dtype:
        want_t = want_t.view(got.dtype) if want_t.element_size() == got.element_size() else want_t.to(got.dtype)
    assert got.shape == want_t.shape, f"{name}: shape {tuple(got.shape)} vs {tuple(want_t.shape)}"
    if not torch.equal(got, want_t):
        bad = (got != want_t).nonzero()
        raise AssertionError(f"{name}: {bad.shape[0]} mismatches, first at {bad[0].tolist()}: "
                             f"got {got[tuple(bad[0])].item()} want {want_t[tuple(bad[0])].item()}")


def check_dispatch(buf: B.Buffer, wl: W.Workload, lay, cap: int, recv, check_tails: bool = True,
                   arrival: bool = True):
    """Bit-exact comparison of everything dispatch leaves in the arena with the oracle."""
    cfg = wl.cfg
    T = cfg.T
    assert buf.status() == 0
    _eq("cnt", buf.cnt, lay.cnt)
    _eq("src_offset", buf.src_offset, lay.src_offset)
    _eq("expert_offset", buf.expert_offset, lay.expert_offset)
    _eq("num_tokens_per_expert", buf.num_tokens_per_expert, lay.num_tokens_per_expert)
    _eq("num_rows_per_rank", buf.num_rows_per_rank, lay.num_rows_per_rank)
    _eq("num_tokens_per_rank", buf.num_tokens_per_rank, lay.num_tokens_per_rank)
    _eq("slot_row", buf.slot_row[:T], lay.slot_row)
    # the oracle leaves the fill byte in rows past a region's count, so whole arrays compare
    if check_tails:
        _eq("recv_x", buf.recv_x, recv.recv_x)
        _eq("recv_src_idx", buf.recv_src_idx, recv.recv_src_idx)
        if cfg.payload:
            _eq("recv_scale", buf.recv_scale.view(torch.int32), recv.recv_scale.view(np.int32))
        if cfg.dedup:
            _eq("recv_topk_idx", buf.recv_topk_idx, recv.recv_topk_idx)
            _eq("recv_topk_w", buf.recv_topk_w.view(torch.int32), recv.recv_topk_w.view(np.int32))
        else:
            _eq("recv_weight", buf.recv_weight.view(torch.int32), recv.recv_weight.view(np.int32))
    else:
        for r in range(cfg.R):
            n = int(lay.num_rows_per_rank[r])
            _eq(f"recv_x[{r}]", buf.recv_x[r, :n], recv.recv_x[r, :n])
            _eq(f"recv_src_idx[{r}]", buf.recv_src_idx[r, :n], recv.recv_src_idx[r, :n])
    if cfg.dedup:
        er = buf.expert_rows.cpu().numpy()
        for r in range(cfg.R):
            n = int(lay.num_tokens_per_expert[r * cfg.L:(r + 1) * cfg.L].sum())
            assert np.array_equal(er[r, :n], lay.expert_rows[r, :n]), f"expert_rows[{r}]"
    if arrival:   # (the readiness-protocol dispatch keeps its own counters)
        got = buf.arrival.cpu().numpy()[int(buf.epoch.item()) & 1]
        assert np.array_equal(got, 8 * lay.num_rows_per_rank), "arrival counters"


def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    def key(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


def check_combine(out: torch.Tensor, want_bits: np.ndarray):
    """GPU combine vs the oracle's fp32 accumulation: at most 1 bf16 ulp and relative error
    <= 2^-7 per element; returns the fraction of bit-identical elements."""
    got = out.view(torch.int16).cpu().numpy().view(np.uint16)
    assert got.shape == want_bits.shape
    d = bf16_ulp_distance(got, want_bits)
    assert d.max() <= 1, f"combine: {int((d > 1).sum())} elements off by more than 1 bf16 ulp (max {d.max()})"
    gf, wf = W.bf16_bits_to_f32(got).astype(np.float64), W.bf16_bits_to_f32(want_bits).astype(np.float64)
    rel = np.abs(gf - wf) <= 2.0 ** -7 * np.abs(wf) + 1e-38
    assert rel.all()
    return float((d == 0).mean())


def run_case(wl: W.Workload, pipeline: int = 0, num_ctas: int = 0, y_bits: np.ndarray | None = None,
             dest_order=None, threads: int = 1, check_tails: bool = True):
    """dispatch (+ combine) one workload on the GPU and compare everything with the oracle."""
    cfg = wl.cfg
    ids, lay, cap, recv = oracle_reference(wl, num_threads=threads)
    buf = make_buffer(cfg, cap, pipeline, num_ctas)
    x, idx, w, phys, ncopies = device_inputs(wl)
    if phys is not None:
        buf.set_replicas(phys, ncopies)
    if dest_order is not None:
        buf.set_dest_order(dest_order)
    buf.dispatch(x, idx, w)
    check_dispatch(buf, wl, lay, cap, recv, check_tails)
    exact = None
    if y_bits is None:
        y_bits = W.make_expert_outputs(cfg, cap)
    y = to_dev(y_bits, torch.bfloat16)
    out = buf.combine(y, w)
    want, _ = oracle.combine(y_bits, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, num_threads=threads)
    exact = check_combine(out, want)
    assert buf.status() == 0
    return buf, lay, cap, exact
