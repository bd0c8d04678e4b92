"""Latency of the readiness protocols (stop-and-wait, Token-Flag Fusion, Data-for-Checksum,
Sentinel Polling; Sec. 3.4 of the paper) over synchronisation granularity and rank count --
the analogue of the paper's dispatch-latency comparison of the Data-as-Flag variants.

    python -m paper_2607_06202_b200.sync_sweep [--tokens 128] [--iters 200] [--markdown]

For every (row bytes, ranks, protocol) it reports
  * kernel: mean time of one ubep_dispatch_sync launch (CUDA events around `iters` launches),
  * sent / ready: inside the last launch, from the first CTA's entry to the last sender
    finishing and to the last receiver having confirmed its region (device nanosecond timer),
  * wire: bytes put on the wire per payload byte.
Inputs are seeded and synthetic (Gaussian routing, top-8 of 256 experts).  Needs a GPU.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B
from . import workload as W

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
                     rows_per_rank_cap=1, dedup=cfg.dedup)
    npr, npe, _ = probe.get_dispatch_layout(idx)
    rows_per_rank = npr if cfg.dedup else npe.view(cfg.R, cfg.L).sum(1)
    cap = W.round_up(max(1, int(rows_per_rank.max().item())), 16)
    n_rows = int(rows_per_rank.sum().item())
    probe.close()
    buf = B.Buffer(num_ranks=cfg.R, num_experts=cfg.E, hidden=cfg.H, topk=cfg.k, max_tokens=cfg.T,
                   rows_per_rank_cap=cap, dedup=cfg.dedup)
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
            rec["wire_ratio"] = wire_ratio(proto, 2 * cfg.H)
        out[proto] = rec
    buf.close()
    return out, n_rows


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--tokens", type=int, default=128)
    ap.add_argument("--iters", type=int, default=200)
    ap.add_argument("--hidden", type=int, nargs="*", default=[256, 1024, 4096, 7168])
    ap.add_argument("--ranks", type=int, nargs="*", default=[8, 32, 128])
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args()
    B.load()
    rows = []
    for R in args.ranks:
        for H in args.hidden:
            cfg = W.Config(f"sync_T{args.tokens}_H{H}_R{R}", T=args.tokens, H=H, E=256, R=R, k=8, seed=7000 + R + H)
            res, n_rows = measure(cfg, args.iters)
            rows.append({"tokens": args.tokens, "row_bytes": 2 * H, "ranks": R, "rows": n_rows, **res})
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


if __name__ == "__main__":
    main()
