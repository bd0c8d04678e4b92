"""Per-CTA latency spread of dispatch under different destination-ordering tables -- the
analogue, on one GPU, of the paper's per-worker token-transmission latencies with and without
expert re-mapping (Sec. 5.4, "Impact of Token Scheduling").

    python -m paper_2607_06202_b200.cta_spread [--workload skewed] [--rows 4] [--markdown]

Every CTA of the persistent dispatch kernel is one worker with an equal slice of the tokens.  The
library's phase trace (ubep_debug_trace) gives, per CTA, when its layout was ready, when its last
copy was issued and when it left.  The tables compared are the identity order, the paper's logical
matrix transposition with `rows` rows (Sec. 3.3) and the reversed order.  Needs a GPU.
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import binding as B
from . import workload as W

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


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--workload", nargs="*", default=["skewed", "prefill"], choices=list(W.CONFIGS))
    ap.add_argument("--rows", type=int, default=4, help="rows of the transposition matrix")
    ap.add_argument("--markdown", action="store_true")
    args = ap.parse_args()
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


if __name__ == "__main__":
    main()
