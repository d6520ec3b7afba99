"""Synthetic re-creation of the paper's buffer-management ablations (Section 6.5): decode
throughput and GPU hit ratio of one workload as the per-set HBM budget goes from nothing
("Base": every selected page crosses the host link), to the mandatory pages only
("+Mandatory": room for one step's selection, i.e. only last step's pages can hit), to
multiples of it ("+Buffering": the bucketed LRU keeps older pages).

    python -m paper_2604_26837_b200.ablation [--workload c2] [--batch 2] [--steps 96] [--evict-exact]

Prints one line per budget; with --evict-exact every budget is run twice, once with the paper's
eviction (every page up to the threshold timestamp) and once with the exact-demand variant,
to show what the over-eviction costs in hit ratio.  Marshalling and timing only; every stage runs in the library.
"""
from __future__ import annotations

import argparse
import json

import torch

import workloads as W

from .driver import SpinRun


def run_budget(w: W.Workload, slots: int, steps: int, prime: int, device="cuda:0", evict_exact: int = 0) -> dict:
    run = SpinRun(W.scaled(w, steps=steps + prime + 2), device, slots_per_set=slots, evict_exact=evict_exact)
    stream = torch.cuda.Stream(device)
    B, L = w.batch, w.num_layers
    with torch.cuda.stream(stream):
        for r in range(B):
            for l in range(L):
                k, v, tp, cen = run.gen_prefill(r, l)
                run.prefill(r, l, k, v, tp, cen, stream)
        qs = {(r, l): W.QueryStream(w, r, l, device) for r in range(B) for l in range(L)}
        out = torch.zeros(B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        ins = []
        for s in range(prime + steps):
            for l in range(L):
                kn, vn = run.gen_step_tokens(l, s)
                q = torch.stack([qs[(r, l)].next() for r in range(B)]).contiguous()
                ins.append((l, kn, vn, q))
        per_step = L
        for i in range(prime * per_step):
            run.step(*ins[i], out, stream)
        torch.cuda.synchronize(device)
        st0 = run.spin.stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(prime * per_step, (prime + steps) * per_step):
            run.step(*ins[i], out, stream)
        e1.record(stream)
    torch.cuda.synchronize(device)
    st1 = run.spin.stats()
    ms = e0.elapsed_time(e1)
    sel = st1["selected_pages"] - st0["selected_pages"]
    hit = st1["hit_pages"] - st0["hit_pages"]
    res = dict(slots=slots, tokens_per_s=B * steps / (ms * 1e-3), ms_per_step=ms / steps,
               hit_ratio=hit / max(sel, 1), evicted_pages_per_step=(st1["evicted_pages"] - st0["evicted_pages"]) / steps,
               bypass_pages=st1["bypass_pages"] - st0["bypass_pages"],
               pcie_mb_per_step=(st1["pcie_bytes"] - st0["pcie_bytes"]) / steps / 1e6,
               error_bits=st1["error_bits"])
    run.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--batch", type=int, default=2)
    ap.add_argument("--steps", type=int, default=96)
    ap.add_argument("--prime", type=int, default=32)
    ap.add_argument("--evict-exact", action="store_true")
    args = ap.parse_args()
    w = W.scaled(W.CONFIGS[args.workload], batch=args.batch)
    mandatory = w.topk * max(1, w.max_partition_pages // 2 if w.partition_kind == W.PART_CLUSTER_CENTROID else 1)
    if w.partition_kind == W.PART_TOKEN_DOT:
        mandatory = 512
    rows = []
    for mult, label in ((0, "Base (no GPU buffer)"), (1, "+Mandatory (1x)"), (2, "+Buffering 2x"), (3, "+Buffering 3x"),
                        (4, "+Buffering 4x"), (5, "+Buffering 5x"), (6, "+Buffering 6x"), (8, "+Buffering 8x")):
        r = run_budget(w, mandatory * mult, args.steps, args.prime)
        r["label"], r["x_mandatory"] = label, mult
        if args.evict_exact:
            e = run_budget(w, mandatory * mult, args.steps, args.prime, evict_exact=1)
            r["exact"] = {k: e[k] for k in ("hit_ratio", "evicted_pages_per_step", "tokens_per_s", "error_bits")}
        rows.append(r)
        print(json.dumps(r), flush=True)
    base = rows[1]["tokens_per_s"]
    print("\n| budget | slots/set | hit ratio | host-link MB/step | ms/step | tokens/s | vs +Mandatory |")
    print("|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['label']} | {r['slots']} | {r['hit_ratio']:.3f} | {r['pcie_mb_per_step']:.2f} | "
              f"{r['ms_per_step']:.3f} | {r['tokens_per_s']:.0f} | {r['tokens_per_s'] / base:.2f}x |")
    if args.evict_exact:
        print("\n| budget | hit ratio (paper's eviction) | evicted pages/step | hit ratio (exact demand) | evicted pages/step | tokens/s exact / paper's |")
        print("|---|---|---|---|---|---|")
        for r in rows:
            e = r["exact"]
            print(f"| {r['label']} | {r['hit_ratio']:.3f} | {r['evicted_pages_per_step']:.1f} | {e['hit_ratio']:.3f} | "
                  f"{e['evicted_pages_per_step']:.1f} | {e['tokens_per_s'] / r['tokens_per_s']:.2f}x |")


if __name__ == "__main__":
    main()
