"""Pins for the oracle's FP8 payload, row contents and combine.

FP8 rows: numpy float32 library arithmetic + torch's CPU float8 cast reproduce payload and
scales; closed-form error bound; the group's largest element lands on +-448.
Dispatch rows: definitional byte equality through recv_src_idx, untouched tails, the
permutation-invariant set of rows per expert.
Combine: closed forms (y == 1, one-hot weights, identity experts), a float64 error bound and
torch CPU gather / multiply / sum as a library cross-check.
"""
import numpy as np
import pytest
import torch

from paper_2607_06202_b200 import workload as W


def _small_cfg(payload, dedup, T=96, H=256, E=16, R=4, k=4, seed=42):
    return W.Config("small", T=T, H=H, E=E, R=R, k=k, payload=payload, dedup=dedup, seed=seed)


def _prepare(orc, cfg, empty=0.0):
    wl = W.make_workload(cfg)
    if empty:
        wl = W.with_empty_slots(wl, empty, 9)
    ids = wl.topk_idx if wl.phys is None else orc.resolve_ids(wl.topk_idx, wl.phys, wl.ncopies)
    lay = orc.layout(ids, cfg.E, cfg.R, cfg.S, cfg.dedup)
    cap = W.round_up(max(1, int(lay.num_rows_per_rank.max())), 8)
    return wl, ids, lay, cap


# ------------------------------------------------------------------------ FP8

def test_fp8_rows_match_numpy_float32_and_torch_cast(orc):
    rng = np.random.default_rng(21)
    x = W.normal_bf16(rng, (64, 512))
    x[3, 128:256] = 0                       # an all-zero group -> amax floor
    x[4, :128] = W.f32_to_bf16_bits(np.full(128, 3e-6, np.float32))   # below the floor
    q, sc = orc.fp8_quantize_rows(x)
    xf = W.bf16_bits_to_f32(x).reshape(64, 4, 128)
    a = np.maximum(np.abs(xf).max(-1), np.float32(1e-4)).astype(np.float32)
    scale = (a / np.float32(448.0)).astype(np.float32)
    inv = (np.float32(448.0) / a).astype(np.float32)
    assert np.array_equal(sc, scale)
    prod = (xf * inv[..., None]).astype(np.float32)
    assert np.abs(prod).max() <= 448.0 * (1 + 2 ** -22)
    ref = torch.from_numpy(np.clip(prod, -448, 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(q, ref.reshape(64, 512))


def test_fp8_error_bound_and_extreme_element(orc):
    rng = np.random.default_rng(22)
    x = W.normal_bf16(rng, (32, 1024))
    q, sc = orc.fp8_quantize_rows(x)
    xf = W.bf16_bits_to_f32(x).astype(np.float64).reshape(32, 8, 128)
    deq = np.array([orc.e4m3_to_f32(int(c)) for c in q.ravel()], np.float64).reshape(32, 8, 128)
    err = np.abs(deq * sc.astype(np.float64)[..., None] - xf)
    # half the grid spacing at the quantised magnitude (spacing 2^(e-3), at least 2^-9), plus fp32 slack
    mag = np.maximum(np.abs(deq), 2.0 ** -6)
    half_step = 2.0 ** (np.floor(np.log2(mag)) - 3) / 2
    assert np.all(err <= sc[..., None] * half_step * (1 + 1e-5) + 1e-7)
    # the largest magnitude of each group maps to code 0x7E / 0xFE
    qg = q.reshape(32, 8, 128)
    arg = np.abs(xf).argmax(-1)
    top = np.take_along_axis(qg, arg[..., None], -1)[..., 0]
    assert np.all((top & 0x7F) == 0x7E)


# ------------------------------------------------------------------- dispatch

@pytest.mark.parametrize("payload", [0, 1])
@pytest.mark.parametrize("dedup", [0, 1])
def test_dispatch_rows_are_the_source_rows(orc, payload, dedup):
    cfg = _small_cfg(payload, dedup)
    wl, ids, lay, cap = _prepare(orc, cfg, empty=0.1)
    rv = orc.dispatch(wl.x, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, cap, payload, dedup, fill=0xA5)
    if payload:
        q, sc = orc.fp8_quantize_rows(wl.x)
    n_checked = 0
    for r in range(cfg.R):
        n = int(lay.num_rows_per_rank[r])
        src = rv.recv_src_idx[r, :n]
        assert src.min(initial=0) >= 0 and src.max(initial=0) < cfg.T
        if payload:
            assert np.array_equal(rv.recv_x[r, :n], q[src])
            assert np.array_equal(rv.recv_scale[r, :n], sc[src])
        else:
            assert np.array_equal(rv.recv_x[r, :n].view(np.uint16), wl.x[src])
        assert np.all(rv.recv_x[r, n:] == 0xA5)              # tails untouched
        assert np.all(rv.recv_src_idx[r, n:].view(np.uint8) == 0xA5)
        n_checked += n
        if dedup:
            assert np.all(np.diff(src) > 0)                   # ascending tokens, one row each
            for row in range(n):
                t = src[row]
                here = (ids[t] >= 0) & (ids[t] // cfg.L == r)
                assert np.array_equal(rv.recv_topk_idx[r, row], np.where(here, ids[t] % cfg.L, -1))
                assert np.array_equal(rv.recv_topk_w[r, row], np.where(here, wl.topk_w[t], 0).astype(np.float32))
        else:
            # permutation-invariant check: each expert's segment holds exactly its tokens
            for l in range(cfg.L):
                p = r * cfg.L + l
                seg = slice(lay.expert_offset[p], lay.expert_offset[p] + lay.num_tokens_per_expert[p])
                toks = np.nonzero((ids == p).any(1))[0]
                assert sorted(src[seg].tolist()) == toks.tolist()
                assert np.array_equal(src[seg], toks)          # and the stable order
                j = np.argmax(ids[toks] == p, axis=1)
                assert np.array_equal(rv.recv_weight[r, seg], wl.topk_w[toks, j])
    assert n_checked == lay.num_rows_per_rank.sum()


def test_dispatch_reports_capacity_overflow(orc):
    cfg = _small_cfg(0, 0)
    wl, ids, lay, cap = _prepare(orc, cfg)
    with pytest.raises(ValueError):
        orc.dispatch(wl.x, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, int(lay.num_rows_per_rank.max()) - 1, 0, 0)


# -------------------------------------------------------------------- combine

def _bf16_ulp_distance(a_bits, b_bits):
    def key(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, -(u & 0x7FFF), u & 0x7FFF)
    return np.abs(key(a_bits) - key(b_bits))


@pytest.mark.parametrize("dedup", [0, 1])
def test_combine_closed_forms(orc, dedup):
    cfg = _small_cfg(0, dedup)
    wl, ids, lay, cap = _prepare(orc, cfg, empty=0.1)
    T, k, H = cfg.T, cfg.k, cfg.H
    ones = np.full((cfg.R, cap, H), 0x3F80, np.uint16)
    # y == 1 with weights 1/8 on every valid slot: exact sum (valid slots) / 8
    w = np.full((T, k), 0.125, np.float32)
    out, _ = orc.combine(ones, ids, w, lay.slot_row, cfg.E, cfg.R)
    expect = (ids >= 0).sum(1).astype(np.float32) / 8
    assert np.array_equal(W.bf16_bits_to_f32(out), np.repeat(expect[:, None], H, 1))
    # one-hot weights pick exactly one expert's row
    y = W.normal_bf16(np.random.default_rng(1), (cfg.R, cap, H))
    for j in range(k):
        w = np.zeros((T, k), np.float32)
        w[:, j] = 1.0
        out, _ = orc.combine(y, ids, w, lay.slot_row, cfg.E, cfg.R)
        valid = ids[:, j] >= 0
        rows = y[ids[valid, j] // cfg.L, lay.slot_row[valid, j]]
        assert np.array_equal(out[valid], rows)
        assert np.all(W.bf16_bits_to_f32(out[~valid]) == 0)


@pytest.mark.parametrize("dedup", [0, 1])
def test_round_trip_identity_experts(orc, dedup):
    """dispatch -> identity experts -> combine with weights summing to one returns x (<= 1 bf16 ulp)."""
    cfg = _small_cfg(0, dedup, T=80, H=384, k=4, seed=77)
    wl, ids, lay, cap = _prepare(orc, cfg)
    rv = orc.dispatch(wl.x, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, cap, 0, dedup)
    y = rv.recv_x.view(np.uint16).reshape(cfg.R, cap, cfg.H)
    assert np.allclose(wl.topk_w.sum(1), 1.0, atol=1e-6)
    out, _ = orc.combine(y, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R)
    assert _bf16_ulp_distance(out, wl.x).max() <= 1


@pytest.mark.parametrize("dedup", [0, 1])
def test_combine_float64_bound_and_torch_cross_check(orc, dedup):
    cfg = _small_cfg(0, dedup, T=64, H=512, k=8, E=32, R=4, seed=5)
    wl, ids, lay, cap = _prepare(orc, cfg, empty=0.05)
    y = W.normal_bf16(np.random.default_rng(2), (cfg.R, cap, cfg.H))
    out, out64 = orc.combine(y, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, want_f64=True)
    got = W.bf16_bits_to_f32(out).astype(np.float64)
    # fp32 accumulation of k terms then one bf16 rounding
    absum = np.zeros_like(out64)
    yt = torch.from_numpy(W.bf16_bits_to_f32(y))
    valid = ids >= 0
    g = (ids // cfg.L).clip(0) * cap + lay.slot_row.clip(0)
    rows = yt.reshape(-1, cfg.H)[torch.from_numpy(g.astype(np.int64))]          # [T, k, H]
    wt = torch.from_numpy(np.where(valid, wl.topk_w, 0).astype(np.float32))
    ref32 = (rows * wt[..., None]).sum(1).numpy().astype(np.float64)
    absum = (rows.abs() * wt[..., None]).sum(1).numpy().astype(np.float64)
    bound = np.abs(out64) * 2.0 ** -8 + absum * cfg.k * 2.0 ** -24 + 1e-30
    assert np.all(np.abs(got - out64) <= bound * (1 + 1e-9))
    assert np.all(np.abs(ref32 - out64) <= absum * cfg.k * 2.0 ** -23 + 1e-30)
    ref_bits = torch.from_numpy(ref32.astype(np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert _bf16_ulp_distance(out, ref_bits).max() <= 1


# ---------------------------------------------------------------- Algorithm 1

def test_quaternary_search_matches_searchsorted(orc):
    rng = np.random.default_rng(8)
    for n in [1, 2, 3, 5, 6, 16, 37, 128, 256, 288]:
        counts = rng.integers(0, 50, n).astype(np.int32)
        if n > 4:
            counts[rng.integers(0, n, n // 3)] = 0
        order = rng.permutation(n).astype(np.int32)
        cum = np.cumsum(counts[order].astype(np.int64))
        total = int(cum[-1])
        targets = list(range(0, total, max(1, total // 97))) + [total - 1] if total else []
        for tgt in targets:
            pos, off, iters = orc.quaternary_search(order, counts, tgt)
            ref = int(np.searchsorted(cum, tgt, side="right"))
            assert pos == ref and off == tgt - (int(cum[ref - 1]) if ref else 0)
            assert 0 <= off < counts[order[pos]]
            assert iters <= int(np.ceil(np.log(max(n, 2)) / np.log(4))) + 1
        assert orc.quaternary_search(order, counts, total) is None
        assert orc.quaternary_search(order, counts, -1) is None
    # typical expert counts converge in 4-5 steps, as the paper states
    counts = rng.integers(1, 100, 256).astype(np.int32)
    order = np.arange(256, dtype=np.int32)
    its = {orc.quaternary_search(order, counts, int(t))[2] for t in rng.integers(0, counts.sum(), 200)}
    assert its <= {4, 5}


def test_equal_slices_and_stride_remap(orc):
    for total, workers in [(131072, 148), (7, 3), (0, 4), (5, 8)]:
        b = orc.equal_slices(total, workers)
        sizes = np.diff(b)
        assert b[0] == 0 and b[-1] == total and sizes.max() - sizes.min() <= 1
    for n, rows in [(256, 16), (288, 7), (10, 3), (5, 8)]:
        order = orc.stride_remap(n, rows)
        assert sorted(order.tolist()) == list(range(n))
        cols = -(-n // rows)
        m = np.full(rows * cols, -1)
        m[:n] = np.arange(n)
        ref = m.reshape(rows, cols).T.ravel()
        assert np.array_equal(order, ref[ref >= 0])


def test_hop_distribution_and_the_effect_of_the_remap(orc):
    """Per-worker hop mix: brute force over the expanded token sequence pins the walk; a stride
    remap whose rows are the four distance groups of the experts (Sec. 3.3; the paper does not
    give the matrix shape) brings every worker close to the per-hop bound ceil(V_h / n)."""
    rng = np.random.default_rng(13)
    n, workers = 64, 16                      # 64 experts in 4 boards of 16; board 0 is one hop away
    counts = rng.integers(20, 60, n).astype(np.int32)
    hop_of = (np.arange(n) // 16 >= 1).astype(np.int32)           # 0 = one hop, 1 = two hops
    natural_order = np.arange(n, dtype=np.int32)
    remap_order = orc.stride_remap(n, 4)                          # 0, 16, 32, 48, 1, 17, ...
    for order in (natural_order, remap_order):
        v = orc.hop_distribution(order, counts, hop_of, workers, 2)
        seq = np.repeat(hop_of[order], counts[order])            # hop class of every token sent, in order
        begin = orc.equal_slices(len(seq), workers)
        brute = np.array([[int((seq[begin[w]:begin[w + 1]] == h).sum()) for h in range(2)] for w in range(workers)])
        assert np.array_equal(v, brute)
        assert np.array_equal(v.sum(1), np.diff(begin))          # every token of the slice is counted once
    V = np.array([counts[hop_of == h].sum() for h in range(2)])
    bound = -(-V // workers)
    natural = orc.hop_distribution(natural_order, counts, hop_of, workers, 2)
    remapped = orc.hop_distribution(remap_order, counts, hop_of, workers, 2)
    # natural order: four workers send one-hop tokens only, twelve send two-hop tokens only
    assert natural[:, 0].max() > 3 * bound[0] and (natural[:, 0] == 0).sum() >= 10
    # remapped: every worker has the global mix, within the size of one expert's token count
    assert np.all(remapped[:, 0] > 0) and np.all(remapped[:, 1] > 0)
    assert np.all(remapped <= bound[None, :] + counts.max())
    assert remapped.var(axis=0).sum() < 0.05 * natural.var(axis=0).sum()      # tr(Sigma) shrinks
