"""GPU parity of the path for ranks on different GPUs (ubep_set_peers, ubep_dispatch_sharded,
ubep_wait_arrivals, ubep_combine_sharded), emulated on one GPU: every rank has its own
arena (a separate allocation) and its own buffer handle, the peer table holds the addresses of
all of them, and the ranks' dispatches run one after the other (they never wait for one
another).  Every arena must hold exactly what the oracle puts into that rank's region."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W
from tests import harness as Hn

pytestmark = pytest.mark.gpu

CASES = {
    "tiny": W.CONFIGS["tiny"],
    "dedup": W.Config("dedup", T=96, H=512, E=32, R=8, k=4, dedup=1, seed=5101),
    "ragged": W.Config("ragged", T=37, H=264, E=12, R=3, k=3, seed=5102),
    "fewer_tokens_than_ranks": W.Config("few", T=5, H=128, E=16, R=8, k=2, dedup=1, seed=5103),
    "one_rank": W.Config("one_rank", T=19, H=64, E=4, R=1, k=2, seed=5104),
    "replicas": W.Config("replicas", T=96, H=512, E=36, R=4, k=4, seed=5105, E_logical=32),
    "fp8": W.Config("fp8", T=96, H=384, E=16, R=4, k=4, payload=1, seed=5106),
    "fp8_dedup": W.Config("fp8_dedup", T=70, H=1024, E=32, R=8, k=4, payload=1, dedup=1, seed=5107),
    # routing tables too large to recount in every CTA (T * k > 8192): counts and prefix sums by launches of
    # their own over the whole table, chunks aligned with the ranks' token ranges
    "large": W.Config("large", T=1203, H=512, E=64, R=8, k=8, seed=5108),
    "large_dedup": W.Config("large_dedup", T=2500, H=256, E=48, R=6, k=4, dedup=1, seed=5109),
    "large_fp8_replicas": W.Config("large_fp8", T=1500, H=384, E=36, R=4, k=6, payload=1, seed=5110, E_logical=32),
    "prefill_sized": W.Config("prefill_sized", T=4096, H=1024, E=256, R=8, k=8, seed=5111),
}


def token_range(s, T, R):
    return s * T // R, (s + 1) * T // R


def make_ranks(cfg, cap, wl_phys):
    bufs = [Hn.make_buffer(cfg, cap) for _ in range(cfg.R)]
    ptrs = [b.arena.data_ptr() for b in bufs]
    for r, b in enumerate(bufs):
        if wl_phys is not None:
            b.set_replicas(*wl_phys)
        B.ubep_set_peers(b.handle, r, ptrs)
    return bufs


def dispatch_all(bufs, cfg, x, idx, w, order=None):
    for s in (order if order is not None else range(cfg.R)):
        b0, b1 = token_range(s, cfg.T, cfg.R)
        B.ubep_dispatch_sharded(bufs[s].handle, x[b0:b1].contiguous(), idx, w, cfg.T)


def check_rank(bufs, r, cfg, lay, recv, times=1):
    b = bufs[r]
    B.ubep_wait_arrivals(b.handle)
    assert b.status() == 0
    fill = torch.full_like(b.recv_x[0], Hn.FILL)
    for q in range(cfg.R):          # region r holds the oracle's rows, the other regions of this arena nothing
        want = torch.from_numpy(recv.recv_x[r]).cuda() if q == r else fill
        assert torch.equal(b.recv_x[q], want), f"arena {r} region {q}"
    n = int(lay.num_rows_per_rank[r])
    Hn._eq(f"recv_src_idx[{r}]", b.recv_src_idx[r, :n], recv.recv_src_idx[r, :n])
    if cfg.payload:
        Hn._eq(f"recv_scale[{r}]", b.recv_scale[r, :n].view(torch.int32), recv.recv_scale[r, :n].view(np.int32))
    if cfg.dedup:
        Hn._eq("recv_topk_idx", b.recv_topk_idx[r, :n], recv.recv_topk_idx[r, :n])
        Hn._eq("recv_topk_w", b.recv_topk_w[r, :n].view(torch.int32), recv.recv_topk_w[r, :n].view(np.int32))
        m = int(lay.num_tokens_per_expert[r * cfg.L:(r + 1) * cfg.L].sum())
        assert np.array_equal(b.expert_rows[r, :m].cpu().numpy(), lay.expert_rows[r, :m])
    else:
        Hn._eq("recv_weight", b.recv_weight[r, :n].view(torch.int32), recv.recv_weight[r, :n].view(np.int32))
    # every rank holds the whole set of counts and offsets, and the handles of its own tokens
    Hn._eq("cnt", b.cnt, lay.cnt)
    Hn._eq("src_offset", b.src_offset, lay.src_offset)
    Hn._eq("expert_offset", b.expert_offset, lay.expert_offset)
    Hn._eq("num_tokens_per_expert", b.num_tokens_per_expert, lay.num_tokens_per_expert)
    Hn._eq("num_rows_per_rank", b.num_rows_per_rank, lay.num_rows_per_rank)
    Hn._eq("num_tokens_per_rank", b.num_tokens_per_rank, lay.num_tokens_per_rank)
    b0, b1 = token_range(r, cfg.T, cfg.R)
    Hn._eq("slot_row", b.slot_row[b0:b1], lay.slot_row[b0:b1])
    assert b.shard_arrival.cpu().tolist() == [times * n, times * n]


@pytest.mark.parametrize("case", list(CASES))
def test_sharded_dispatch_and_combine_match_the_oracle(case):
    cfg = CASES[case]
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    x, idx, w, phys, ncopies = Hn.device_inputs(wl)
    bufs = make_ranks(cfg, cap, (phys, ncopies) if phys is not None else None)
    dispatch_all(bufs, cfg, x, idx, w)
    for r in range(cfg.R):
        check_rank(bufs, r, cfg, lay, recv)
    # the same call again, senders in another order: the arrival words keep growing, nothing is reset
    dispatch_all(bufs, cfg, x, idx, w, order=list(reversed(range(cfg.R))))
    for r in range(cfg.R):
        check_rank(bufs, r, cfg, lay, recv, times=2)
    # combine: every rank gathers from the buffers of the ranks that produced the rows
    y_bits = W.make_expert_outputs(cfg, cap)
    ys = []
    for r in range(cfg.R):
        y = torch.full((cfg.R, cap, cfg.H), -7.0, dtype=torch.bfloat16, device="cuda")   # only region r is real
        y[r] = Hn.to_dev(y_bits[r], torch.bfloat16)
        ys.append(y)
    y_ptrs = torch.tensor([y.data_ptr() for y in ys], dtype=torch.int64, device="cuda")
    want, _ = oracle.combine(y_bits, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R)
    for s in range(cfg.R):
        b0, b1 = token_range(s, cfg.T, cfg.R)
        out = torch.zeros((b1 - b0, cfg.H), dtype=torch.bfloat16, device="cuda")
        B.ubep_combine_sharded(bufs[s].handle, y_ptrs, w, cfg.T, out)
        if b1 > b0:
            Hn.check_combine(out, want[b0:b1])
        assert bufs[s].status() == 0


def test_a_receiver_whose_senders_have_not_run_gives_up_and_recovers():
    cfg = W.Config("late", T=64, H=128, E=8, R=2, k=2, seed=5200)
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    x, idx, w, _, _ = Hn.device_inputs(wl)
    bufs = make_ranks(cfg, cap, None)
    dispatch_all(bufs, cfg, x, idx, w, order=[0])        # rank 1 has not sent anything yet
    B.ubep_wait_arrivals(bufs[0].handle)                  # nothing will raise the count: the wait runs out
    assert bufs[0].status() == B.UBEP_ERR_TIMEOUT
    dispatch_all(bufs, cfg, x, idx, w, order=[1])
    for r in range(cfg.R):
        check_rank(bufs, r, cfg, lay, recv)


def test_argument_errors():
    cfg = W.CONFIGS["tiny"]
    wl = W.make_workload(cfg)
    _, lay, cap, _ = Hn.oracle_reference(wl)
    x, idx, w, _, _ = Hn.device_inputs(wl)
    buf = Hn.make_buffer(cfg, cap)
    with pytest.raises(B.UbepError) as e:                 # not in sharded use yet
        B.ubep_dispatch_sharded(buf.handle, x, idx, w, cfg.T)
    assert e.value.code == B.UBEP_ERR_ARG
    ptrs = [buf.arena.data_ptr()] * cfg.R
    with pytest.raises(B.UbepError):
        B.ubep_set_peers(buf.handle, cfg.R, ptrs)         # rank out of range
    with pytest.raises(B.UbepError):
        B.ubep_set_peers(buf.handle, 1, [0] + ptrs[1:])   # a null peer
    other = Hn.make_buffer(cfg, cap)
    with pytest.raises(B.UbepError):                      # the table's own entry must be this buffer's arena
        B.ubep_set_peers(buf.handle, 0, [other.arena.data_ptr()] + ptrs[1:])
    fewer_sources = Hn.make_buffer(dataclasses.replace(cfg, num_src_ranks=2), cap)
    with pytest.raises(B.UbepError):                      # one source rank per GPU
        B.ubep_set_peers(fewer_sources.handle, 0, [fewer_sources.arena.data_ptr()] * cfg.R)


def _driver_worker(rank, world, port, out_path):
    import os
    import sys
    import torch.distributed as dist
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=rank, world_size=world)
    from paper_2607_06202_b200 import sharded
    cfg = W.Config("driver", T=48, H=256, E=8, R=1, k=2, dedup=1, seed=5300)
    wl = W.make_workload(cfg)
    ids, lay, cap, recv = Hn.oracle_reference(wl)
    ep = sharded.ShardedEP(num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T, rows_per_rank_cap=cap,
                           dedup=cfg.dedup)
    x, idx, w, _, _ = Hn.device_inputs(wl)
    region, n = ep.dispatch(x, idx, w, cfg.T)
    n = int(n.item())
    ok = n == int(lay.num_rows_per_rank[0])
    ok = ok and torch.equal(region[:n].view(torch.int16).cpu(), torch.from_numpy(recv.recv_x[0, :n].view(np.int16)))
    ep.y[0, :n] = region[:n]                      # identity experts
    out = ep.combine()
    y_bits = np.zeros((1, cap, cfg.H), np.uint16)
    y_bits[0, :n] = recv.recv_x[0, :n].view(np.uint16)
    want, _ = oracle.combine(y_bits, ids, wl.topk_w, lay.slot_row, cfg.E, cfg.R)
    Hn.check_combine(out, want)
    ok = ok and ep.status() == 0
    with open(out_path, "w") as f:
        f.write("ok" if ok else "mismatch")
    dist.destroy_process_group()


def test_driver_with_one_rank(tmp_path):
    import torch.multiprocessing as mp
    out_path = str(tmp_path / "r0.txt")
    mp.spawn(_driver_worker, args=(1, 29751, out_path), nprocs=1, join=True)
    assert open(out_path).read() == "ok"


def _bench_block_worker(rank, world, port, out_path):
    import contextlib
    import io
    import json
    import os
    import sys
    import torch.distributed as dist
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=rank, world_size=world)
    import bench
    buf = io.StringIO()
    with contextlib.redirect_stdout(buf):
        bench.run_sharded(None, rank, world, 0)
    line = json.loads(buf.getvalue().strip().splitlines()[-1])
    with open(out_path, "w") as f:
        json.dump(line, f)
    dist.destroy_process_group()


def test_the_benchmarks_block_for_ranks_on_different_gpus_with_one_rank(tmp_path):
    """What bench.py prints as its second line under torchrun, run here with a group of one: the
    decode-like shape through ShardedEP, rank 0's region and output against the oracle."""
    import json
    import torch.multiprocessing as mp
    out_path = str(tmp_path / "line.json")
    mp.spawn(_bench_block_worker, args=(1, 29753, out_path), nprocs=1, join=True)
    blk = json.load(open(out_path))["sharded"]
    assert blk["status"] == "ok", blk
    assert blk["parity"] is True and blk["nranks"] == 1
    assert blk["dispatch_us"] > 0 and blk["combine_us"] > 0
