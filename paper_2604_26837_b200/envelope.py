"""The ideal sparse-serving envelope of Section 3.1 for a recorded run: Eq. 1-3 evaluated with
the miss ratio of an offline-optimal (Belady, farthest next use) cache of the same size, next to
what the bucketed LRU achieved and to the measured step time.

    python -m paper_2604_26837_b200.envelope [--workload c2] [--batch 8] [--steps 96]

Host-side analysis only: the library runs the steps, its debug dump gives each set's selected
partitions per step, and the replay below never touches the device.
"""
from __future__ import annotations

import argparse
import json
from typing import Dict, List, Sequence

PAGE_BYTES = 8192


def belady_miss_pages(trace: Sequence[Sequence[int]], pages_of: Dict[int, int], capacity: int) -> int:
    """Missed pages of an offline-optimal cache of `capacity` pages for one set.

    trace[t] = partitions selected at step t (all needed at once).  A partition is cached whole
    or not at all.  On a miss the victims are the resident partitions, not selected at this step,
    whose next use lies farthest in the future (never used again first); a selected partition
    is always cached while room can be made for it (its pages are this step's mandatory pages).  With one page per
    partition this is Belady's MIN and optimal; with partitions of different sizes it is the
    usual greedy envelope.  What does not fit even after evicting everything else is bypassed
    (fetched, not cached), as the library does."""
    T = len(trace)
    next_use: List[Dict[int, int]] = [dict() for _ in range(T)]      # next_use[t][p] = next step > t using p
    seen: Dict[int, int] = {}
    for t in range(T - 1, -1, -1):
        for p in trace[t]:
            next_use[t][p] = seen.get(p, T + 1)
        for p in trace[t]:
            seen[p] = t
    resident: Dict[int, int] = {}                                   # partition -> step of its next use
    used = 0
    misses = 0
    for t in range(T):
        sel = set(trace[t])
        for p in sel:
            if p in resident:
                resident[p] = next_use[t][p]
        for p in sorted(sel, key=lambda x: next_use[t][x]):           # soonest reuse first
            if p in resident:
                continue
            n = pages_of.get(p, 1)
            misses += n
            while used + n > capacity:
                victims = [v for v in resident if v not in sel]
                if not victims:
                    break
                v = max(victims, key=lambda x: (resident[x], x))
                used -= pages_of.get(v, 1)
                del resident[v]
            if used + n <= capacity:
                resident[p] = next_use[t][p]
                used += n
    return misses


def eq3_tpot(summary_bytes: float, kv_topk_bytes: float, rho: float, bw_hbm: float, bw_pcie: float) -> float:
    """Eq. 3 with T_MLP = 0: (QK_score + KV_topk) / BW_HBM + rho * KV_topk / BW_PCIe, seconds."""
    return (summary_bytes + kv_topk_bytes) / bw_hbm + rho * kv_topk_bytes / bw_pcie


def main():
    import torch
    import workloads as W
    from .driver import SpinRun
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--steps", type=int, default=96)
    ap.add_argument("--hbm-gbs", type=float, default=6547.8)
    ap.add_argument("--pcie-gbs", type=float, default=55.4)
    args = ap.parse_args()
    w = W.CONFIGS[args.workload]
    if args.batch:
        w = W.scaled(w, batch=args.batch)
    w = W.scaled(w, steps=args.steps)
    dev = "cuda:0"
    run = SpinRun(w, dev)
    for r in range(w.batch):
        k, v, tp, cen = run.gen_prefill(r, 0)
        run.prefill(r, 0, k, v, tp, cen)
    qs = [W.QueryStream(w, r, 0, dev) for r in range(w.batch)]
    out = torch.zeros(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    traces: Dict[tuple, List[List[int]]] = {(r, h): [] for r in range(w.batch) for h in range(w.num_kv_heads)}
    pages_of: Dict[tuple, Dict[int, int]] = {key: {} for key in traces}
    cap_pages = w.topk * max(1, w.max_partition_pages) + args.steps // 16 + 4
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ms = []
    for step in range(args.steps):
        kn, vn = run.gen_step_tokens(0, step)
        q = torch.stack([s.next() for s in qs]).contiguous()
        ev0.record()
        run.step(0, kn, vn, q, out)
        ev1.record()
        torch.cuda.synchronize()
        step_ms.append(ev0.elapsed_time(ev1))
        for (r, h) in traces:
            d = run.spin.debug_dump(run.reqs[r], 0, h, w.topk, cap_pages, run.budgets[r], 1 << 15)
            parts = [int(p) for p in d["parts"]]
            traces[(r, h)].append(parts)
            for p in parts:
                pages_of[(r, h)][p] = max(1, -(-int(d["part_tokens"][p]) // 16))
    st = run.spin.stats()
    sel_pages = st["selected_pages"]
    lru_miss = st["miss_pages"]
    bel_miss = sum(belady_miss_pages(traces[key], pages_of[key], run.budgets[key[0]]) for key in traces)
    steps = args.steps
    summ = st["candidates_scored"] * (512 if w.partition_kind == 0 else 256) / steps
    kv = (st["selected_pages"] + st["tail_pages"]) * PAGE_BYTES / steps
    warm = step_ms[steps // 4:]
    res = dict(workload=w.name, batch=w.batch, steps=steps, slots_per_set=run.budgets[0],
               rho_bucketed_lru=lru_miss / sel_pages, rho_belady=bel_miss / sel_pages,
               eq3_us_with_belady=1e6 * eq3_tpot(summ, kv, bel_miss / sel_pages, args.hbm_gbs * 1e9, args.pcie_gbs * 1e9),
               eq3_us_with_bucketed_lru=1e6 * eq3_tpot(summ, kv, lru_miss / sel_pages, args.hbm_gbs * 1e9, args.pcie_gbs * 1e9),
               measured_us_per_step_warm=1e3 * sum(warm) / len(warm),
               note="cold start included in both miss ratios; measured time is per synchronised step")
    print(json.dumps(res))
    run.close()


if __name__ == "__main__":
    main()
