"""GPU parity of the readiness-protocol dispatch (Sec. 3.4 of the paper: stop-and-wait,
Token-Flag Fusion, Data-for-Checksum, Sentinel Polling) through the C ABI: every protocol
must leave exactly what the oracle's dispatch leaves, and what it puts on the wire must be
the oracle's encoding of those rows."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu

PROTOCOLS = ["sw", "tff", "dc", "sp"]

CASES = {
    "tiny": W.CONFIGS["tiny"],
    "decode": W.CONFIGS["decode"],
    # 528-byte rows: 44 Token-Flag blocks exactly, a checksum block cut short after 16 bytes
    "ragged": W.Config("ragged", T=37, H=264, E=12, R=3, k=3, seed=4101),
    # 4112-byte rows: the last Token-Flag block is padded; one row per (token, rank)
    "padded_dedup": W.Config("padded_dedup", T=61, H=2056, E=24, R=6, k=4, dedup=1, seed=4102),
    "one_rank": W.Config("one_rank", T=19, H=64, E=4, R=1, k=2, seed=4103),
    "replicas": W.Config("replicas", T=96, H=512, E=36, R=4, k=4, seed=4104, E_logical=32),
    # FP8 rows: a wire row is the e4m3 payload followed by its fp32 scales.  396 bytes: 33 Token-Flag
    # blocks, the 25th Sentinel block cut short after 12 bytes
    "fp8_ragged": W.Config("fp8_ragged", T=96, H=384, E=16, R=4, k=4, payload=1, seed=4105),
    "fp8_dedup": W.Config("fp8_dedup", T=70, H=1024, E=32, R=8, k=4, payload=1, dedup=1, seed=4106),
    # the W8A8 row of the paper's Table 3: hidden 7168, 256 experts, top-8
    "fp8_w8a8": W.Config("fp8_w8a8", T=64, H=7168, E=256, R=32, k=8, payload=1, seed=4107),
    # routing tables no CTA can recount alone (more than 8192 slots): counting and prefix sums are launches
    # of their own in front of the protocol kernel
    "large": W.Config("large", T=1500, H=256, E=32, R=8, k=8, seed=4108),
    "large_fp8_dedup": W.Config("large_fp8_dedup", T=2100, H=256, E=64, R=16, k=8, payload=1, dedup=1, seed=4109),
    "large_replicas": W.Config("large_replicas", T=3000, H=128, E=36, R=4, k=4, seed=4110, E_logical=32),
}


def wire_rows(cfg, recv, r, n):
    """The first n rows of region r as they travel: bf16 rows as they are, FP8 rows as payload bytes
    followed by the bytes of their scales."""
    rows = recv.recv_x[r, :n].reshape(n, -1)
    if cfg.payload:
        rows = np.concatenate([rows, recv.recv_scale[r, :n].reshape(n, -1).view(np.uint8)], axis=1)
    return np.ascontiguousarray(rows)


def wire_checks(buf, proto, cfg, lay, recv, grid):
    v = buf.sync_views
    seq = int(v["seq"].item())
    half = seq & 1
    n_rows = lay.num_rows_per_rank
    times = v["times"].cpu().numpy()[:grid]
    assert (np.diff(times[:, :5], axis=1) >= 0).all(), "per-CTA time stamps must not go backwards"
    assert (times[:, 0] > 0).all()
    if proto == "tff":
        wire = v["tff_wire"].cpu().numpy()
        for r in range(cfg.R):
            sent = wire_rows(cfg, recv, r, int(n_rows[r]))
            for row in range(int(n_rows[r])):
                want = oracle.tff_pack(sent[row], B.UBEP_SYNC_BLOCK_BYTES, B.UBEP_SYNC_FLAG_BYTES, seq)
                assert np.array_equal(wire[r, row], want.reshape(-1)), f"DataBlocks of region {r} row {row}"
                back, missing = oracle.tff_unpack(wire[r, row], sent.shape[1], B.UBEP_SYNC_BLOCK_BYTES,
                                                  B.UBEP_SYNC_FLAG_BYTES, seq)
                assert missing == 0 and np.array_equal(back, sent[row])
    elif proto == "dc":
        sums = v["checksum"].cpu().numpy().view(np.uint64)[half]
        for r in range(cfg.R):
            want = oracle.dc_checksum(recv.recv_x[r, :int(n_rows[r])].reshape(int(n_rows[r]), -1),
                                      B.UBEP_SYNC_DC_BLOCK_BYTES, B.UBEP_SYNC_DC_MARKER_BYTES)
            assert int(sums[r]) == want, f"checksum of region {r}"
        assert (v["counters"].cpu().numpy()[half] == grid).all(), "every sender announces itself to every region"
    elif proto == "sp":
        wire = v["sp_wire"]
        assert bool((wire == 0xFF).all()), "consumed blocks must show the sentinel again"
        row_w = cfg.H + 4 * (cfg.H // 128) if cfg.payload else 2 * cfg.H
        assert wire.shape[2] == -(-row_w // 16) * 16
        assert oracle.sp_pending(wire[0, :2].cpu().numpy(), 16, 16, B.UBEP_SYNC_SENTINEL) == 2 * (wire.shape[2] // 16)
    else:
        assert np.array_equal(v["counters"].cpu().numpy()[2 + half], n_rows), "one count per fenced row"


@pytest.mark.parametrize("proto", PROTOCOLS)
@pytest.mark.parametrize("case", list(CASES))
def test_protocols_match_oracle(case, proto):
    cfg = CASES[case]
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap)
    buf.attach_sync(fill=0x5A)          # attach must initialise whatever the memory held
    x, idx, w, phys, ncopies = Hn.device_inputs(wl)
    if phys is not None:
        buf.set_replicas(phys, ncopies)
    grid = buf.sync_views["times"].shape[0]
    buf.dispatch_sync(proto, x, idx, w)
    Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
    wire_checks(buf, proto, cfg, lay, recv, grid)
    # a second call on the same buffer with other routing and data: nothing of the first may be taken for new
    wl2 = W.with_empty_slots(W.make_workload(dataclasses.replace(cfg, seed=cfg.seed + 50)), 0.15, cfg.seed + 51)
    ids2, lay2, _, recv2 = Hn.oracle_reference(wl2, cap=cap)
    assert int(lay2.num_rows_per_rank.max()) <= cap
    x2, idx2, w2, phys2, ncopies2 = Hn.device_inputs(wl2)
    if phys2 is not None:
        buf.set_replicas(phys2, ncopies2)      # the other seed drew another replica table
    buf.recv_x.fill_(Hn.FILL)
    if cfg.payload:
        buf.recv_scale.view(torch.uint8).fill_(Hn.FILL)
    buf.dispatch_sync(proto, x2, idx2, w2)
    Hn.check_dispatch(buf, wl2, lay2, cap, recv2, check_tails=False, arrival=False)
    if cfg.payload:       # (with tails unchecked the harness leaves the scales out: compare the rows that exist)
        for r in range(cfg.R):
            n = int(lay2.num_rows_per_rank[r])
            Hn._eq(f"recv_scale[{r}]", buf.recv_scale[r, :n].view(torch.int32), recv2.recv_scale[r, :n].view(np.int32))
    wire_checks(buf, proto, cfg, lay2, recv2, grid)
    # combine runs on what the protocol dispatch left
    y_bits = W.make_expert_outputs(cfg, cap)
    out = buf.combine(Hn.to_dev(y_bits, torch.bfloat16), w2)
    want, _ = oracle.combine(y_bits, ids2, wl2.topk_w, lay2.slot_row, cfg.E, cfg.R)
    Hn.check_combine(out, want)
    assert buf.status() == 0


@pytest.mark.parametrize("proto", PROTOCOLS)
@pytest.mark.parametrize("num_ctas", [1, 5, 40])
def test_few_ctas_and_more_regions_than_ctas(proto, num_ctas):
    cfg = W.Config("grid", T=83, H=256, E=32, R=8, k=4, dedup=1, seed=4200 + num_ctas)
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap, num_ctas=num_ctas)
    buf.attach_sync()
    x, idx, w, _, _ = Hn.device_inputs(wl)
    for _ in range(3):
        buf.dispatch_sync(proto, x, idx, w)
    Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
    wire_checks(buf, proto, cfg, lay, recv, num_ctas)


def test_protocols_interleave_with_each_other_and_with_the_main_dispatch():
    cfg = W.CONFIGS["tiny"]
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap)
    buf.attach_sync()
    x, idx, w, _, _ = Hn.device_inputs(wl)
    grid = buf.sync_views["times"].shape[0]
    for proto in ["dc", "main", "sw", "sw", "main", "tff", "sp", "dc", "dc", "main", "sp", "tff", "sw"]:
        buf.recv_x.fill_(Hn.FILL)
        if proto == "main":
            buf.dispatch(x, idx, w)
            Hn.check_dispatch(buf, wl, lay, cap, recv)
        else:
            buf.dispatch_sync(proto, x, idx, w)
            Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
            wire_checks(buf, proto, cfg, lay, recv, grid)


def test_sentinel_scan_counts_the_blocks_polling_could_never_see():
    cfg = W.Config("scan", T=40, H=128, E=8, R=2, k=2, seed=4300)
    wl = W.make_workload(cfg)
    xb = wl.x.copy()
    flat = xb.reshape(-1)
    for blk in (0, 17, 300, 639):              # whole 16-byte blocks of 0xFFFF codes
        flat[blk * 8:(blk + 1) * 8] = 0xFFFF
    flat[8 * 50 + 1:8 * 50 + 9] = 0xFFFF       # eight such codes that straddle two blocks
    _, lay, cap, _ = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap)
    buf.attach_sync()
    want = oracle.sp_pending(xb, 16, 16, B.UBEP_SYNC_SENTINEL)
    assert want == 4
    assert buf.scan_sentinel(Hn.to_dev(xb, torch.bfloat16)) == want
    assert buf.scan_sentinel(Hn.to_dev(wl.x, torch.bfloat16)) == 0
    assert buf.scan_sentinel(Hn.to_dev(wl.x, torch.bfloat16)[:0]) == 0


def test_sentinel_in_the_data_runs_into_the_bounded_wait_and_the_next_call_recovers():
    cfg = W.Config("collide", T=24, H=128, E=8, R=2, k=2, seed=4400)
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    xb = wl.x.copy()
    t = int(np.nonzero((wl.topk_idx >= 0).any(axis=1))[0][0])
    xb[t, 16:24] = 0xFFFF                       # one block of a row that is sent equals the sentinel
    buf = Hn.make_buffer(cfg, cap)
    buf.attach_sync()
    x, idx, w, _, _ = Hn.device_inputs(wl)
    buf.dispatch_sync("sp", Hn.to_dev(xb, torch.bfloat16), idx, w)
    assert buf.status() == B.UBEP_ERR_TIMEOUT   # the kernel gave up and returned; the context is intact
    buf.recv_x.fill_(Hn.FILL)
    buf.dispatch_sync("sp", x, idx, w)
    Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
    wire_checks(buf, "sp", cfg, lay, recv, buf.sync_views["times"].shape[0])
    # A caller that does not ask for the status after the call that gave up: the next Sentinel Polling
    # call must not take that call's leftover blocks for its own -- it reports the condition again
    # and moves nothing; once the status has been read the wire is re-filled and all is well.
    buf.dispatch_sync("sp", Hn.to_dev(xb, torch.bfloat16), idx, w)      # gives up
    buf.recv_x.fill_(Hn.FILL)
    buf.dispatch_sync("sp", x, idx, w)                                   # no status read in between
    torch.cuda.synchronize()
    assert bool((buf.recv_x == Hn.FILL).all()), "a call on a dirty wire must not deliver anything"
    assert buf.status() == B.UBEP_ERR_TIMEOUT
    buf.dispatch_sync("sp", x, idx, w)
    Hn.check_dispatch(buf, wl, lay, cap, recv, arrival=False)
    # the other protocols carry the same bytes without trouble
    for proto in ("tff", "dc", "sw"):
        buf.dispatch_sync(proto, Hn.to_dev(xb, torch.bfloat16), idx, w)
        assert buf.status() == 0
        assert torch.equal(buf.recv_x[0, :int(lay.num_rows_per_rank[0])].cpu(),
                           torch.from_numpy(oracle.dispatch(xb, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R, cap, 0, 0,
                                                            fill=Hn.FILL).recv_x[0, :int(lay.num_rows_per_rank[0])]))


def test_argument_errors():
    cfg = W.CONFIGS["tiny"]
    wl = W.make_workload(cfg)
    _, lay, cap, _ = Hn.oracle_reference(wl)
    buf = Hn.make_buffer(cfg, cap, max_tokens=5000)
    x, idx, w, _, _ = Hn.device_inputs(wl)
    with pytest.raises(B.UbepError) as e:          # no wire buffer yet
        buf.dispatch_sync("tff", x, idx, w)
    assert e.value.code == B.UBEP_ERR_ARG
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.UbepError) as e:
        B.ubep_sync_attach(buf.handle, small)
    assert e.value.code == B.UBEP_ERR_ARENA
    buf.attach_sync()
    with pytest.raises(B.UbepError):
        buf.dispatch_sync(7, x, idx, w)
    big_T = 5001                                    # more tokens than the buffer was made for
    xb = torch.zeros((big_T, cfg.H), dtype=torch.bfloat16, device="cuda")
    ib = torch.zeros((big_T, cfg.k), dtype=torch.int32, device="cuda")
    wb = torch.zeros((big_T, cfg.k), dtype=torch.float32, device="cuda")
    with pytest.raises(B.UbepError) as e:
        B.ubep_dispatch_sync(buf.handle, B.UBEP_SYNC_SW, xb, ib, wb, big_T)
    assert e.value.code == B.UBEP_ERR_ARG
    fp8 = dataclasses.replace(W.CONFIGS["tiny"], payload=1, H=256)
    fbuf = Hn.make_buffer(fp8, cap)
    assert 0 < B.ubep_sync_wire_bytes(fbuf.cfg) < B.ubep_sync_wire_bytes(buf.cfg)   # FP8 rows are shorter on the wire
    # T == 0 leaves zero counts like the main dispatch
    buf.dispatch_sync("dc", x[:0], idx[:0], w[:0])
    assert int(buf.num_rows_per_rank.sum()) == 0 and buf.status() == 0


def test_one_captured_graph_of_all_protocols_replays_with_new_routing():
    """The sequence number that flags and counter halves go by lives on the device, so a captured
    graph of protocol dispatches can be replayed; inputs are rewritten in place between replays."""
    cfg = W.Config("graph", T=160, H=512, E=32, R=8, k=4, seed=4500)
    base = W.make_workload(cfg)
    cap = 256
    bufs = {proto: Hn.make_buffer(cfg, cap) for proto in PROTOCOLS}
    for b in bufs.values():
        b.attach_sync()
    x, idx, w, _, _ = Hn.device_inputs(base)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):                      # warm-up outside capture
        for proto, b in bufs.items():
            b.dispatch_sync(proto, x, idx, w, stream)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for proto, b in bufs.items():
            b.dispatch_sync(proto, x, idx, w, stream)
    for it in range(3):
        wl = W.make_workload(dataclasses.replace(cfg, seed=4600 + it))
        x.copy_(Hn.to_dev(wl.x, torch.bfloat16))
        idx.copy_(Hn.to_dev(wl.topk_idx.astype(np.int32)))
        w.copy_(Hn.to_dev(wl.topk_w))
        for b in bufs.values():
            for name in ("recv_x", "recv_src_idx", "recv_weight"):
                b.views[name].view(torch.uint8).fill_(Hn.FILL)
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        ids, lay, _, recv = Hn.oracle_reference(wl, cap=cap)
        for proto, b in bufs.items():
            Hn.check_dispatch(b, wl, lay, cap, recv, arrival=False)
            wire_checks(b, proto, cfg, lay, recv, b.sync_views["times"].shape[0])
            assert int(b.sync_views["seq"].item()) == 2 + it     # one warm-up call, then one per replay
