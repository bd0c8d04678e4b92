#!/usr/bin/env python
"""Measurement sweeps beside bench.py (each needs a GPU; the library itself does not use this file).

    python bench_sweeps.py spread [--workload skewed prefill] [--rows 4] [--markdown]
    python bench_sweeps.py sync   [--tokens 128] [--iters 200] [--markdown]
    python bench_sweeps.py roles  [--tokens 512 1024 4096 16384] [--count-warps 0 1 2 4 8] [--markdown]
    python bench_sweeps.py auto   [--tokens 64 128 256 512 1024 2048] [--markdown]
    python bench_sweeps.py budget [--workload decode] [--markdown]

spread: per-CTA latency spread of dispatch under different destination-ordering tables -- the
analogue, on one GPU, of the paper's per-worker token-transmission latencies with and without
expert re-mapping (Sec. 5.4, "Impact of Token Scheduling").
sync: latency of the readiness protocols (stop-and-wait, Token-Flag Fusion, Data-for-Checksum,
Sentinel Polling; Sec. 3.4) over synchronisation granularity and rank count.
roles: FP8 dispatch time over the size of the count group (the paper's core-allocation question:
Sec. 3.2, the cost model of App. A, the group-size heat maps of App. C.3).
auto: the flag-free (LOCAL) against the flag-exchanging (FUSED) schedule over token counts and shape
families, and what AUTO picks.
budget: where the microseconds of one layer go: the dispatch kernel's phases from the library's trace,
taken inside the steady replay of dispatch + combine graphs, beside what a kernel boundary costs by
itself (a chain of empty kernels).
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_06202_b200 import binding as B
from paper_2607_06202_b200 import workload as W

SPREAD_DOC = """Every CTA of the persistent dispatch kernel is one worker with an equal slice of the tokens.
The library's phase trace (ubep_debug_trace) gives, per CTA, when its layout was ready, when its last
copy was issued and when it left.  The tables compared are the identity order, the paper's logical
matrix transposition with `rows` rows (Sec. 3.3) and the reversed order."""

SYNC_DOC = """For every (row bytes, ranks, protocol): kernel = mean time of one ubep_dispatch_sync launch
(CUDA events around `iters` launches); sent / ready = inside the last launch, from the first CTA's
entry to the last sender finishing and to the last receiver having confirmed its region (device
nanosecond timer); wire = bytes put on the wire per payload byte.  Inputs are seeded and synthetic
(Gaussian routing, top-8 of 256 experts)."""

# ------------------------------------------------------------------------------------ spread

READY, ISSUED, STORED, END = 6, 8, 9, 10   # phase slots of the trace (see ubep_debug_trace)


def stride_order(n: int, rows: int) -> np.ndarray:
    """Visiting order of n destinations after the logical matrix transposition of Sec. 3.3: the ids
    fill a matrix of `rows` rows row by row and are read column by column."""
    cols = -(-n // rows)
    grid = np.full(rows * cols, -1, np.int64)
    grid[:n] = np.arange(n)
    order = grid.reshape(rows, cols).T.reshape(-1)
    return order[order >= 0].astype(np.int32)


def spread(cfg: W.Config, order, repeats: int = 5):
    dev = torch.device("cuda", 0)
    wl = W.make_workload(cfg)
    idx = torch.from_numpy(wl.topk_idx.astype(np.int32)).to(dev)
    x = torch.from_numpy(wl.x).view(torch.bfloat16).to(dev)
    w = torch.from_numpy(wl.topk_w.astype(np.float32)).to(dev)
    common = dict(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T,
                  num_src_ranks=cfg.S, payload=cfg.payload, dedup=cfg.dedup)
    probe = B.Buffer(rows_per_rank_cap=1, **common)
    phys = ncopies = None
    if wl.phys is not None:
        phys, ncopies = torch.from_numpy(wl.phys).to(dev), torch.from_numpy(wl.ncopies).to(dev)
        probe.set_replicas(phys, ncopies)
    npr, npe, _ = probe.get_dispatch_layout(idx)
    rows_per_rank = npr if cfg.dedup else npe.view(cfg.R, cfg.L).sum(1)
    cap = W.round_up(max(1, int(rows_per_rank.max().item())), 128)
    probe.close()
    buf = B.Buffer(rows_per_rank_cap=cap, **common)
    if phys is not None:
        buf.set_replicas(phys, ncopies)
    buf.set_dest_order(order)
    B.ubep_debug_trace(buf.handle, True)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    runs = []
    for it in range(repeats + 1):
        flush.fill_(it)                    # cold L2 for every run
        buf.dispatch(x, idx, w)
        torch.cuda.synchronize()
        if it == 0:
            continue                       # first run: warm-up
        tr = buf.trace.cpu().numpy().astype(np.int64)
        t0 = tr[:, 0].min()
        runs.append(np.stack([(tr[:, s] - t0) / 1e3 for s in (READY, ISSUED, STORED, END)], axis=1))
    status = buf.status()
    buf.close()
    if status != 0:
        raise RuntimeError(f"device status {status} ({B.ubep_strerror(status)})")
    return np.median(np.stack(runs), axis=0)   # [CTAs, 4], median over the repeats


def main_spread(argv):
    ap = argparse.ArgumentParser(prog="bench_sweeps.py spread", description=SPREAD_DOC,
                                 formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", nargs="*", default=["skewed", "prefill"], choices=list(W.CONFIGS))
    ap.add_argument("--rows", type=int, default=4, help="rows of the transposition matrix")
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args(argv)
    B.load()
    if args.markdown:
        print("| workload | table | layout ready us (median / max) | sending us: min / median / p95 / max | "
              "max / median | kernel end us (max) |")
        print("|---|---|---|---|---|---|")
    for name in args.workload:
        cfg = W.CONFIGS[name]
        tables = {"identity": None, f"transposed ({args.rows} rows)": stride_order(cfg.R, args.rows),
                  "reversed": np.arange(cfg.R - 1, -1, -1, dtype=np.int32)}
        for label, order in tables.items():
            t = spread(cfg, order)
            send = t[:, 3] - t[:, 0]          # layout ready (movers released) -> CTA done, all its copies complete
            line = (name, label, np.median(t[:, 0]), t[:, 0].max(), send.min(), np.median(send),
                    np.percentile(send, 95), send.max(), send.max() / np.median(send), t[:, 3].max())
            if args.markdown:
                print("| %s | %s | %.1f / %.1f | %.1f / %.1f / %.1f / %.1f | %.2f | %.1f |" % line)
            else:
                print("%s %-22s ready %.1f/%.1f  sending min %.1f med %.1f p95 %.1f max %.1f  max/med %.2f  end %.1f"
                      % line)



# -------------------------------------------------------------------------------------- sync

PROTOCOLS = ["sw", "tff", "dc", "sp"]


def wire_ratio(proto: str, row_bytes: int) -> float:
    if proto == "tff":
        payload = B.UBEP_SYNC_BLOCK_BYTES - B.UBEP_SYNC_FLAG_BYTES
        return B.UBEP_SYNC_BLOCK_BYTES * -(-row_bytes // payload) / row_bytes
    return 1.0


def measure(cfg: W.Config, iters: int, warmup: int = 20):
    dev = torch.device("cuda", 0)
    wl = W.make_workload(cfg)
    idx = torch.from_numpy(wl.topk_idx.astype(np.int32)).to(dev)
    x = torch.from_numpy(wl.x).view(torch.bfloat16).to(dev)
    w = torch.from_numpy(wl.topk_w.astype(np.float32)).to(dev)
    probe = B.Buffer(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T,
                     rows_per_rank_cap=1, dedup=cfg.dedup, payload=cfg.payload)
    npr, npe, _ = probe.get_dispatch_layout(idx)
    rows_per_rank = npr if cfg.dedup else npe.view(cfg.R, cfg.L).sum(1)
    cap = W.round_up(max(1, int(rows_per_rank.max().item())), 16)
    n_rows = int(rows_per_rank.sum().item())
    probe.close()
    buf = B.Buffer(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T,
                   rows_per_rank_cap=cap, dedup=cfg.dedup, payload=cfg.payload)
    views = buf.attach_sync()
    out = {}
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for proto in PROTOCOLS + ["main"]:
        def call():
            if proto == "main":
                buf.dispatch(x, idx, w)
            else:
                buf.dispatch_sync(proto, x, idx, w)
        for _ in range(warmup):
            call()
        torch.cuda.synchronize()
        start.record()
        for _ in range(iters):
            call()
        stop.record()
        torch.cuda.synchronize()
        status = buf.status()
        if status != 0:
            raise RuntimeError(f"{proto}: device status {status} ({B.ubep_strerror(status)})")
        rec = {"kernel_us": start.elapsed_time(stop) * 1e3 / iters}
        if proto != "main":
            t = views["times"].cpu().numpy()
            t_first = int(t[:, 0].min())
            rec["layout_us"] = (int(t[:, 1].max()) - t_first) / 1e3
            rec["sent_us"] = (int(t[:, 2].max()) - t_first) / 1e3
            rec["ready_us"] = (int(t[:, 3].max()) - t_first) / 1e3
            rec["wire_ratio"] = wire_ratio(proto, cfg.H + 4 * (cfg.H // 128) if cfg.payload else 2 * cfg.H)
        out[proto] = rec
    buf.close()
    return out, n_rows


def main_sync(argv):
    ap = argparse.ArgumentParser(prog="bench_sweeps.py sync", description=SYNC_DOC,
                                 formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--tokens", type=int, default=128)
    ap.add_argument("--iters", type=int, default=200)
    ap.add_argument("--hidden", type=int, nargs="*", default=[256, 1024, 4096, 7168])
    ap.add_argument("--ranks", type=int, nargs="*", default=[8, 32, 128])
    ap.add_argument("--payload", type=int, default=0, choices=[0, 1], help="1 = FP8 rows (payload + scales on the wire)")
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args(argv)
    B.load()
    rows = []
    for R in args.ranks:
        for H in args.hidden:
            cfg = W.Config(f"sync_T{args.tokens}_H{H}_R{R}", T=args.tokens, H=H, E=256, R=R, k=8, payload=args.payload,
                           seed=7000 + R + H)
            res, n_rows = measure(cfg, args.iters)
            row_bytes = H + 4 * (H // 128) if args.payload else 2 * H
            rows.append({"tokens": args.tokens, "row_bytes": row_bytes, "ranks": R, "rows": n_rows, **res})
    if not args.markdown:
        for r in rows:
            print(json.dumps(r))
        return
    print("| row bytes | ranks | rows | protocol | kernel us | layout us | sent us | ready us | wire bytes / payload byte |")
    print("|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        for proto in PROTOCOLS + ["main"]:
            m = r[proto]
            if proto == "main":
                print(f"| {r['row_bytes']} | {r['ranks']} | {r['rows']} | main path | {m['kernel_us']:.2f} | | | | 1.000 |")
            else:
                print(f"| {r['row_bytes']} | {r['ranks']} | {r['rows']} | {proto.upper()} | {m['kernel_us']:.2f} | "
                      f"{m['layout_us']:.2f} | {m['sent_us']:.2f} | {m['ready_us']:.2f} | {m['wire_ratio']:.3f} |")


# ------------------------------------------------------------------------- roles / auto

def dispatch_us(cfg: W.Config, pipeline: int = 0, count_warps: int = -1, min_timed_s: float = 0.08):
    """Median time of one ubep_dispatch on rotating buffer sets (cold L2), timed like bench.py does:
    graphs of dispatches only, blocks between CUDA events.  Returns (us, what AUTO would run it as)."""
    import bench as BM

    class A:
        quant_warps = 0
        prefetch_rows = 0
        no_graph = False
    A.pipeline, A.count_warps = pipeline, count_warps
    b = BM.Bench(cfg, A, 0, 1)
    steps = 2 * b.nsets
    blocks = b.time_blocks(b.make_block(b.dispatch, steps), steps, 1, min_timed_s=min_timed_s)
    us = BM.summarize_blocks(blocks, steps)["median_us"]
    status = b.sets[0]["buf"].status()
    b.close()
    if status != 0:
        raise RuntimeError(f"device status {status} ({B.ubep_strerror(status)})")
    return us


def predicted_count_share(E: int, k: int, tokens_per_cta: float) -> float:
    """The paper's cost model (App. A): the share of workers that should count grows with the number
    of experts and shrinks with top-k times the tokens a worker sends, n_count ~ N_exp / (K_top * B_sz)."""
    return E / (k * max(tokens_per_cta, 1e-9))


def main_roles(argv):
    ap = argparse.ArgumentParser(prog="bench_sweeps.py roles")
    ap.add_argument("--tokens", type=int, nargs="*", default=[512, 1024, 4096, 16384])
    ap.add_argument("--count-warps", type=int, nargs="*", default=[0, 1, 2, 4, 8])
    ap.add_argument("--shapes", nargs="*", default=["256,8", "128,8", "288,8", "256,4"], help="E,k pairs")
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args(argv)
    B.load()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    head = ["E", "k", "T", "tokens / CTA", "E / (k * tokens per CTA)"] + [f"n_count={n}" for n in args.count_warps] + ["best"]
    if args.markdown:
        print("| " + " | ".join(head) + " |")
        print("|" + "---|" * len(head))
    for shape in args.shapes:
        E, k = (int(v) for v in shape.split(","))
        R = 72 if E == 288 else 32
        for T in args.tokens:
            cfg = W.Config(f"roles_E{E}_k{k}_T{T}", T=T, H=7168, E=E, R=R, k=k, payload=1, seed=9000 + T + E + k)
            # FUSED asked for explicitly: the count group exists in the schedules with an exchange
            times = [dispatch_us(cfg, B.UBEP_PIPELINE_FUSED, n) for n in args.count_warps]
            best = args.count_warps[int(np.argmin(times))]
            row = [E, k, T, f"{T / sms:.1f}", f"{predicted_count_share(E, k, T / sms):.2f}"] + [f"{t:.1f}" for t in times] + [best]
            print(("| " + " | ".join(str(v) for v in row) + " |") if args.markdown else " ".join(str(v) for v in row), flush=True)


def main_auto(argv):
    ap = argparse.ArgumentParser(prog="bench_sweeps.py auto")
    ap.add_argument("--tokens", type=int, nargs="*", default=[64, 128, 256, 512, 768, 1024, 1536, 2048])
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args(argv)
    B.load()
    families = [("H=7168 E=256 R=32", dict(H=7168, E=256, R=32)), ("H=4096 E=128 R=16", dict(H=4096, E=128, R=16)),
                ("H=7168 E=288 R=72", dict(H=7168, E=288, R=72))]
    head = ["family", "rows", "dedup", "T", "FUSED us", "LOCAL us", "AUTO us", "AUTO / better"]
    if args.markdown:
        print("| " + " | ".join(head) + " |")
        print("|" + "---|" * len(head))
    for label, shp in families:
        for payload in (0, 1):
            for dedup in (0, 1):
                for T in args.tokens:
                    cfg = W.Config(f"auto_T{T}", T=T, k=8, payload=payload, dedup=dedup, seed=9100 + T, **shp)
                    fused = dispatch_us(cfg, B.UBEP_PIPELINE_FUSED)
                    try:
                        local = dispatch_us(cfg, B.UBEP_PIPELINE_LOCAL)
                    except B.UbepError:
                        local = float("nan")      # the table does not fit in shared memory
                    auto = dispatch_us(cfg, B.UBEP_PIPELINE_AUTO)
                    better = np.nanmin([fused, local])
                    row = [label, "fp8" if payload else "bf16", dedup, T, f"{fused:.1f}", f"{local:.1f}", f"{auto:.1f}",
                           f"{auto / better:.2f}"]
                    print(("| " + " | ".join(str(v) for v in row) + " |") if args.markdown else " ".join(str(v) for v in row),
                          flush=True)


# ----------------------------------------------------------------------------------- budget

PHASES = [(0, "CTA starts (predecessor complete)"), (1, "routing table staged, bitmaps built"), (5, "rows assigned"),
          (6, "movers released"), (7, "mover warp's first row in shared memory, its copies issued"), (8, "last copy issued"),
          (9, "copies complete"), (3, "expert-level outputs written (duty group)"), (10, "CTA ends")]


def main_budget(argv):
    import bench as BM
    ap = argparse.ArgumentParser(prog="bench_sweeps.py budget")
    ap.add_argument("--workload", default="decode")
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args(argv)
    B.load()

    class A:
        pipeline = 0
        quant_warps = 0
        count_warps = -1
        prefetch_rows = 0
        no_graph = False
    cfg = W.CONFIGS[args.workload]
    b = BM.Bench(cfg, A, 0, 1)
    steps = 4 * b.nsets
    # (1) the layer and its kernels, as bench.py times them
    layer = BM.summarize_blocks(b.time_blocks(b.make_block(b.step, steps), steps, 2, min_timed_s=0.1), steps)
    disp = BM.summarize_blocks(b.time_blocks(b.make_block(b.dispatch, steps), steps, 1, min_timed_s=0.05), steps)
    comb = BM.summarize_blocks(b.time_blocks(b.make_block(b.combine, steps), steps, 1, min_timed_s=0.05), steps)
    # (2) what a kernel boundary costs: chains of empty kernels, ordinary and programmatic launches
    h = b.sets[0]["buf"].handle
    empty = {}
    for label, ahead in (("ordinary launch", False), ("programmatic stream serialization", True)):
        def one(_s, ahead=ahead):
            B.ubep_debug_empty_launch(h, ahead, b.stream)
        blocks = b.time_blocks(b.make_block(one, 200), 200, 1, min_timed_s=0.05)
        empty[label] = BM.summarize_blocks(blocks, 200)
    # (3) the dispatch kernel's phases inside the steady replay of dispatch + combine
    for s in b.sets:
        B.ubep_debug_trace(s["buf"].handle, True)
    blk = b.make_block(b.step, steps)
    for _ in range(3):
        blk()
    torch.cuda.synchronize()
    acc = []
    for _ in range(6):
        blk()
        torch.cuda.synchronize()
        acc += [s["buf"].trace.cpu().numpy().astype(np.int64).copy() for s in b.sets]
    rows = []
    for slot, label in PHASES:
        per = []
        for tr in acc:
            t0 = tr[:, 0].min()
            ok = (tr[:, slot] >= t0) & (tr[:, slot] < t0 + 10 ** 7)
            col = (tr[ok, slot] - t0) / 1e3
            if len(col):
                per.append((col.min(), np.median(col), col.max()))
        if per:
            rows.append((label,) + tuple(np.median(np.array(per), 0)))
    b.close()
    p = print
    p(f"workload {args.workload}: layer {layer['median_us']:.2f} us (min {layer['min_us']:.2f}); dispatch alone "
      f"{disp['median_us']:.2f}, combine alone {comb['median_us']:.2f} (each: per kernel in a chain of its own kind)")
    for label, e in empty.items():
        p(f"empty kernel, {label}: {e['median_us']:.2f} us per launch in a chain (min {e['min_us']:.2f})")
    if args.markdown:
        p("\n| phase of the dispatch kernel (us after the first CTA's start) | earliest CTA | median CTA | last CTA |")
        p("|---|---|---|---|")
    for label, lo, med, hi in rows:
        p((f"| {label} | {lo:.2f} | {med:.2f} | {hi:.2f} |") if args.markdown else f"{label:60s} {lo:7.2f} {med:7.2f} {hi:7.2f}")


SWEEPS = {"spread": main_spread, "sync": main_sync, "roles": main_roles, "auto": main_auto, "budget": main_budget}


def main():
    if len(sys.argv) < 2 or sys.argv[1] not in SWEEPS:
        print(__doc__)
        sys.exit(2)
    SWEEPS[sys.argv[1]](sys.argv[2:])


if __name__ == "__main__":
    main()
