"""How long a prefill's Offload (Section 4.1: pages written to pinned host memory) keeps the
caller's stream busy, written through versus asynchronous (`spin_config.offload_stage_bytes`).

    python -m paper_2604_26837_b200.offload_overlap [--workload c2] [--batch 2] [--stage-mb 256]

Per layer the caller's stream runs `spin_append_kv` for every request and then a stand-in for
the next layer's compute (a bf16 GEMM).  Reported: the time of the caller's stream for all
layers, and the time until the last page has reached host memory.  Marshalling and timing
only; the pages move in the library.
"""
from __future__ import annotations

import argparse
import json

import torch

import workloads as W

from .driver import SpinRun


def run(w: W.Workload, stage_bytes: int, gemm_n: int, device="cuda:0") -> dict:
    r = SpinRun(w, device, offload_stage_bytes=stage_bytes)
    stream = torch.cuda.Stream(device)
    a = torch.randn(gemm_n, gemm_n, device=device, dtype=torch.bfloat16)
    kv = [[r.gen_prefill(q, l) for l in range(w.num_layers)] for q in range(w.batch)]
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for l in range(w.num_layers):
            for q in range(w.batch):
                k, v, tp, cen = kv[q][l]
                r.prefill(q, l, k, v, tp, cen, stream)
            a = (a @ a).clamp_(-1, 1)                 # the next layer's compute
        e1.record(stream)
    e1.synchronize()
    caller_ms = e0.elapsed_time(e1)
    import time
    t0 = time.perf_counter()
    torch.cuda.synchronize(device)                    # the library's stream drains
    drain_ms = (time.perf_counter() - t0) * 1e3
    bytes_ = sum(k.numel() * 4 for row in kv for (k, _, _, _) in row)
    err = r.spin.stats()["error_bits"]
    r.close()
    return dict(stage_mb=stage_bytes / 2**20, caller_stream_ms=caller_ms, drain_after_ms=drain_ms,
                offloaded_mb=bytes_ / 1e6, error_bits=err)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--batch", type=int, default=2)
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--stage-mb", type=int, default=256)
    ap.add_argument("--gemm", type=int, default=8192)
    args = ap.parse_args()
    w = W.scaled(W.CONFIGS[args.workload], batch=args.batch, num_layers=args.layers, steps=4)
    for stage in (0, args.stage_mb << 20):
        run(w, stage, args.gemm)                      # warm-up (allocator, clocks)
        print(json.dumps(run(w, stage, args.gemm)), flush=True)


if __name__ == "__main__":
    main()
