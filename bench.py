#!/usr/bin/env python
"""Benchmark of the sparse decode step (append one token + Select/Retrieve/Attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

A "step" is one pass of the whole hot path over one batch of synthetic input: for every layer
of the workload, one appended token per request and one decode call.  The default workload
is the Llama-3-8B-shaped single layer (batch 8, 32768-token contexts, page min/max
partitions, 128 pages per set and step, 25% HBM budget).  With N > 1 every rank runs an
independent replica on its own GPU (sets are independent: no collective on the data path).

Prints ONE JSON line (rank 0).  `value` is decode tokens/s with inputs resident in HBM, timed
with CUDA events on the launching stream; `e2e` is the same metric through the C ABI with
HOST buffers (q, new k/v copied in, output copied out, every step).  The L2 is flushed
between timed steps (untimed), as it would be by the other layers of a real model.
"""
from __future__ import annotations

import argparse
import datetime
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

PAGE_BYTES = 8192
# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu captures
# (profiles/), keyed by workload then kernel; None = not captured for this workload.
NCU_TRAFFIC = {"c2": {"fetch": None, "score": 71.1e6, "attn_split": 65.7e6}}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), source="measured (MEASURED_PEAKS.json)")
    return dict(hbm_gbs=6650.0, source="fallback (profiling recipe)")


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 100 ms while the bench runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.path = tempfile.mktemp(prefix="spin_clocks_", suffix=".csv")
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0: datetime.datetime, t1: datetime.datetime):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        for line in open(self.path):
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                rows.append((ts, float(parts[1]), float(parts[2]), parts[5:9]))
            except Exception:
                continue
        try:
            os.unlink(self.path)
        except OSError:
            pass
        if not rows:
            return None
        inside = [r for r in rows if t0 <= r[0] <= t1] or rows[-3:]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in inside for i in range(4) if r[3][i].lower().startswith("active")})
        return dict(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                    reasons=reasons, samples=len(inside))


def pcie_link(gpu_id: str):
    """Generation and width of the GPU's host link as nvidia-smi reports them now (or None)."""
    try:
        out = subprocess.run(["nvidia-smi", "-i", gpu_id, "--query-gpu=pcie.link.gen.current,pcie.link.width.current",
                              "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
        gen, width = [int(x.strip()) for x in out.strip().splitlines()[0].split(",")]
        return dict(gen=gen, width=width)
    except Exception:
        return None


def measure_pcie_gbs(torch, device, stream) -> float:
    """Peak of the host link as one large pinned host->device copy (best of 5)."""
    n = 256 << 20
    src = torch.empty(n, dtype=torch.uint8).pin_memory()
    dst = torch.empty(n, dtype=torch.uint8, device=device)
    best = 0.0
    with torch.cuda.stream(stream):
        for _ in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dst.copy_(src, non_blocking=True)
            e1.record(stream)
            e1.synchronize()
            best = max(best, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    return best


def oracle_run(w, budget_s: float, steps_cap: int, warmup: int, sample_requests: int = 1):
    """Time the CPU oracle, as it stands, on `sample_requests` requests of the workload."""
    import numpy as np
    import workloads as W
    from oracle import spin_oracle as O
    try:
        from threadpoolctl import threadpool_limits
        limiter = threadpool_limits(1)
    except Exception:
        limiter = None
    orc = O.SpinOracle(O.OracleConfig(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                      w.page_tokens, w.partition_kind, w.topk, w.lru_buckets))
    reqs = []
    for r in range(sample_requests):
        req = orc.request_open(w.slots_per_set if w.slots_per_set else min(w.topk * 2, 512))
        reqs.append(req)
        for l in range(w.num_layers):
            k, v = W.kv_tokens(w, r, l, 0, w.request_context(r))
            if w.partition_kind == W.PART_CLUSTER_CENTROID:
                orc.append_kv(req, l, W.to_bits(k), W.to_bits(v),
                              W.cluster_assignment(w, r, l, w.request_context(r)).numpy(),
                              W.to_bits(W.centroids(w, r, l)))
            else:
                orc.append_kv(req, l, W.to_bits(k), W.to_bits(v))
    qs = {(r, l): W.QueryStream(w, r, l) for r in range(sample_requests) for l in range(w.num_layers)}
    times = []
    step = 0
    t_start = time.perf_counter()
    while True:
        ins = []
        for l in range(w.num_layers):
            kv = [W.kv_tokens(w, r, l, w.request_context(r) + step, 1) for r in range(sample_requests)]
            q = np.stack([W.to_bits(qs[(r, l)].next()) for r in range(sample_requests)])
            ins.append((l, [(W.to_bits(k), W.to_bits(v)) for k, v in kv], q))
        t0 = time.perf_counter()
        for l, kv, q in ins:
            for r, (kb, vb) in enumerate(kv):
                orc.append_kv(reqs[r], l, kb, vb)
            orc.decode_step(l, reqs, q)
        dt = time.perf_counter() - t0
        if step >= warmup:
            times.append(dt)
        step += 1
        if len(times) >= steps_cap or (len(times) >= 2 and time.perf_counter() - t_start > budget_s):
            break
    if limiter is not None:
        limiter.restore_original_limits()
    total = sum(times)
    return dict(value=sample_requests * len(times) / total, steps=len(times), ms_per_step=1e3 * total / len(times),
                cores=1, sample=f"{sample_requests} of {w.batch} requests x {len(times)} decode steps "
                                f"(all {w.num_kv_heads} kv heads, {w.num_layers} layer(s)), numpy, 1 thread")


def rank_workload(base, rank: int, total_steps: int):
    """The replica a rank runs: same shapes, its own seed (sets are independent, so N ranks are N
    independent replicas with no collective on the data path)."""
    import workloads as W
    return W.scaled(base, seed=base.seed + 1000 * rank, steps=total_steps)


def allreduce_max(values, device="cpu"):
    """Max over ranks of a list of floats (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_value(units_per_rank: int, world: int, max_elapsed_ms: float) -> float:
    """Whole-job throughput: the units all ranks processed over the slowest rank's time."""
    return units_per_rank * world / (max_elapsed_ms * 1e-3)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="spin", choices=["spin", "reference"])
    ap.add_argument("--prime", type=int, default=24, help="untimed decode steps that warm the KV cache (setup)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--resident-scoring", type=int, default=0, help="spin_config.resident_scoring: 0 automatic, 1 always, -1 never")
    ap.add_argument("--context", type=int, default=0, help="override the context length (smaller captures)")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--layers", type=int, default=0, help="override the layer count (scaled runs of the 32-layer config)")
    ap.add_argument("--fetch-mode", type=int, default=0, help="0 fused into attention, 1 separate copy kernel")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    import workloads as W
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    base = W.CONFIGS[args.workload]
    if args.context:
        base = W.scaled(base, context=args.context)
    if args.batch:
        base = W.scaled(base, batch=args.batch)
    if args.layers:
        base = W.scaled(base, num_layers=args.layers)
    # a workload without a fixed budget states a total: 60 GB of KV over its 32 layers and 64
    # requests; a scaled run keeps the per-layer, per-request share
    cache_pages_per_layer = None
    if base.slots_per_set == 0:
        cache_pages_per_layer = int(60e9 / 32 / PAGE_BYTES * base.batch / 64)
    metric, unit = "decode_tokens_per_s", "tokens/s"
    cfg_desc = dict(workload=f"{base.name}: batch {base.batch} x {base.num_layers} layer(s), "
                             f"{base.num_q_heads}q/{base.num_kv_heads}kv heads, context {base.context}, "
                             f"kind {base.partition_kind}, top-k {base.topk}, "
                             f"{base.slots_per_set if base.slots_per_set else 'dynamic'} slots/set, "
                             f"{base.lru_buckets} buckets, drift {base.drift}",
                    global_batch=base.batch * world, context=base.context, parallelism=f"replicas x{world}")

    if args.impl == "reference":
        if rank != 0:
            return
        r = oracle_run(base, budget_s=120.0, steps_cap=args.steps, warmup=args.warmup)
        print(json.dumps(dict(
            impl="reference", metric=metric, value=r["value"], unit=unit, n_gpus=args.gpus, steps=r["steps"],
            warmup=args.warmup, ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak",
            vs_baseline=None, dtype="f64", data="synthetic", config=cfg_desc,
            cpu_baseline=dict(value=r["value"], unit=unit, cores=r["cores"], kind="oracle", sample=r["sample"]),
            e2e=dict(value=r["value"], unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))
        return

    import torch
    from paper_2604_26837_b200 import build as spin_build
    if rank == 0:
        spin_build.build()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    from paper_2604_26837_b200.driver import SpinRun

    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    K, Wm, P = args.steps, args.warmup, args.prime
    prof_steps = min(K, 64)
    e2e_steps = 0 if args.no_e2e else K
    total_steps = P + Wm + K + K + prof_steps + (Wm + e2e_steps)
    w = rank_workload(base, rank, total_steps)
    run = SpinRun(w, device, fetch_mode=args.fetch_mode, cache_pages_per_layer=cache_pages_per_layer,
                  resident_scoring=args.resident_scoring)
    stream = torch.cuda.Stream(device)
    B, L = w.batch, w.num_layers

    def barrier():
        torch.cuda.synchronize(device)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(device)

    with torch.cuda.stream(stream):
        for r in range(B):
            for l in range(L):
                k, v, tp, cen = run.gen_prefill(r, l)
                run.prefill(r, l, k, v, tp, cen, stream)
                del k, v
        # inputs of every decode step, resident in HBM before any timed region
        qstreams = {(r, l): W.QueryStream(w, r, l, device) for r in range(B) for l in range(L)}
        q_all = torch.empty(total_steps, L, B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        k_all = torch.empty(total_steps, L, B, w.num_kv_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        v_all = torch.empty_like(k_all)
        for s in range(total_steps):
            for l in range(L):
                k_all[s, l], v_all[s, l] = run.gen_step_tokens(l, s)
                for r in range(B):
                    q_all[s, l, r] = qstreams[(r, l)].next()
        out = torch.zeros(B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        flush = torch.empty(64 << 20, dtype=torch.int32, device=device)        # 256 MiB
    torch.cuda.synchronize(device)
    pcie_gbs = measure_pcie_gbs(torch, device, stream)
    cur = [0]

    def flush_l2_fn():
        # write 256 MiB (> 126 MB L2), then read it back so that the L2 is left full of CLEAN
        # lines, as it is after the weights of a model's other layers have streamed through;
        # a write-only flush would leave dirty lines whose write-back taxes the timed kernels
        flush.zero_()
        flush.max()

    def one_step(s):
        for l in range(L):
            run.step(l, k_all[s, l], v_all[s, l], q_all[s, l], out, stream)

    def timed_steps(n, flush_l2=True):
        evs = []
        with torch.cuda.stream(stream):
            for _ in range(n):
                if flush_l2:
                    flush_l2_fn()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                one_step(cur[0])
                e1.record(stream)
                cur[0] += 1
                evs.append((e0, e1))
        torch.cuda.synchronize(device)
        return [a.elapsed_time(b) for a, b in evs]

    props = torch.cuda.get_device_properties(device)
    sampler = ClockSampler(f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(local_rank))
    cold_steps = timed_steps(P + Wm)                       # cache priming + warm-up: reported apart (cold start)
    st0 = run.spin.stats()
    barrier()
    t_begin = datetime.datetime.now()
    per_step = timed_steps(K)
    barrier()
    t_end = datetime.datetime.now()
    st1 = run.spin.stats()
    elapsed_ms = sum(per_step)
    # back-to-back variant without the L2 flush (one pair of events around all K steps)
    with torch.cuda.stream(stream):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(K):
            one_step(cur[0])
            cur[0] += 1
        e1.record(stream)
    torch.cuda.synchronize(device)
    noflush_ms = e0.elapsed_time(e1) / K
    clocks = sampler.stop(t_begin, t_end)
    link = pcie_link(f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(local_rank))

    # per-kernel durations, measured live with CUDA events recorded between the launches
    stp0 = run.spin.stats()
    run.spin.profile(True)
    timed_steps(prof_steps)
    prof = run.spin.profile_read()
    run.spin.profile(False)
    stp1 = run.spin.stats()

    # end to end: host buffers in, host buffer out, every step
    e2e = None
    if e2e_steps:
        qh = q_all[cur[0]:cur[0] + Wm + e2e_steps].cpu().pin_memory()
        kh = k_all[cur[0]:cur[0] + Wm + e2e_steps].cpu().pin_memory()
        vh = v_all[cur[0]:cur[0] + Wm + e2e_steps].cpu().pin_memory()
        oh = torch.zeros(B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16).pin_memory()
        e2e_times = []
        oh_bits = oh.view(torch.int16).numpy()           # the pinned output buffer as the host reads it
        checksum = 0
        # the step's host buffers as the caller would hold them (views made outside the timed region)
        host_in = [[(kh[i, l], vh[i, l], qh[i, l]) for l in range(L)] for i in range(Wm + e2e_steps)]
        with torch.cuda.stream(stream):
            for i in range(Wm + e2e_steps):
                flush_l2_fn()
                stream.synchronize()
                t0 = time.perf_counter()
                for l in range(L):
                    kk, vv, qq = host_in[i][l]
                    run.step(l, kk, vv, qq, oh, stream)
                stream.synchronize()                       # the result is read on the host
                checksum += int(oh_bits[0, 0, 0]) + int(oh_bits[-1, -1, -1])
                if i >= Wm:
                    e2e_times.append(time.perf_counter() - t0)
        e2e_ms = 1e3 * sum(e2e_times)
        h2d = L * (qh[0, 0].numel() + kh[0, 0].numel() + vh[0, 0].numel()) * 2
        d2h = L * oh.numel() * 2
    final = run.spin.stats()

    if world > 1:
        elapsed_ms, e2e_max, noflush_ms = allreduce_max([elapsed_ms, e2e_ms if e2e_steps else 0.0, noflush_ms], device)
        if e2e_steps:
            e2e_ms = e2e_max
    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    value = aggregate_value(B * K, world, elapsed_ms)
    d = {k: st1[k] - st0[k] for k in st0 if k not in ("error_bits", "debug_words")}
    hbm_step = d["hbm_bytes"] / K
    pcie_step = d["pcie_bytes"] / K
    t_hbm = hbm_step / (peaks["hbm_gbs"] * 1e9)
    t_pcie = pcie_step / (pcie_gbs * 1e9)
    t_step = elapsed_ms * 1e-3 / K
    dp = {k: stp1[k] - stp0[k] for k in stp0 if k not in ("error_bits", "debug_words")}
    kern = {}
    miss_b = dp["miss_pages"] * PAGE_BYTES
    admit_b = (dp["miss_pages"] - dp["bypass_pages"]) * PAGE_BYTES
    kv_b = (dp["selected_pages"] + dp["tail_pages"]) * PAGE_BYTES
    fused = args.fetch_mode == 0
    # algorithmic bytes per kernel over the profiled steps: (HBM bytes, host-link bytes)
    bytes_of = dict(score=(dp["candidates_scored"] * (512 if w.partition_kind == 0 else 256), 0),
                    fetch=(admit_b, admit_b),
                    attn_split=((kv_b - miss_b + admit_b, miss_b) if fused else (kv_b - (miss_b - admit_b), miss_b - admit_b)))
    tot_ms = sum(ms for _, ms in prof.values()) or 1.0
    for name, (n, ms) in prof.items():
        if not n:
            continue
        kern[name] = dict(launches=n, avg_us=1e3 * ms / n, share=ms / tot_ms)
        if name in bytes_of:
            hb, pb = bytes_of[name]
            t_h, t_p = hb / (peaks["hbm_gbs"] * 1e9), pb / (pcie_gbs * 1e9)
            kern[name].update(hbm_gbs=hb / (ms * 1e-3) / 1e9, pcie_gbs=pb / (ms * 1e-3) / 1e9,
                              bound="pcie" if t_p > t_h else "hbm", roof_frac=max(t_h, t_p) / (ms * 1e-3))
    top = max((k_ for k_ in ("fetch", "score", "attn_split") if k_ in kern), key=lambda k_: kern[k_]["share"])
    bound = kern[top]["bound"]
    peak = pcie_gbs if bound == "pcie" else peaks["hbm_gbs"]
    achieved = kern[top]["pcie_gbs"] if bound == "pcie" else kern[top]["hbm_gbs"]
    traffic = (NCU_TRAFFIC.get(args.workload) or {}).get(top) if not (args.context or args.batch or args.layers) else None
    names = dict(fetch="k_fetch", score="k_score", attn_split="k_attn (attention + page fetch)" if fused else "k_attn")
    roofline = dict(kernel=names[top], bound=bound, achieved=achieved, peak=peak, unit="GB/s",
                    frac=kern[top]["roof_frac"], traffic=traffic,
                    peak_source=("pinned H2D copy measured in this run" if bound == "pcie" else peaks["source"]),
                    avg_launch_us=kern[top]["avg_us"],
                    hbm_bytes_per_launch=bytes_of[top][0] / kern[top]["launches"],
                    pcie_bytes_per_launch=bytes_of[top][1] / kern[top]["launches"])
    line = dict(
        metric=metric, value=value, unit=unit, n_gpus=world, steps=K, warmup=Wm, ms_per_step=elapsed_ms / K,
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16 in, f32 accumulate", data="synthetic",
        config=dict(cfg_desc, primed_steps=P, l2="flushed between timed steps (256 MiB written then read back, untimed)",
                    note="single-layer config: tokens/s is per-layer-step throughput"),
        p50_tpot_ms=statistics.median(per_step), ms_per_step_noflush=noflush_ms,
        gpu_launches=int(d["kernel_launches"]), clocks=clocks,
        step_roofline=dict(hbm_bytes_per_step=hbm_step, pcie_bytes_per_step=pcie_step,
                           hbm_gbs_peak=peaks["hbm_gbs"], hbm_peak_source=peaks["source"], pcie_gbs_peak=pcie_gbs,
                           t_hbm_us=1e6 * t_hbm, t_pcie_us=1e6 * t_pcie, t_step_us=1e6 * t_step,
                           bound="pcie" if t_pcie > t_hbm else "hbm", frac=max(t_hbm, t_pcie) / t_step,
                           frac_vs_nominal_8tbs=max(hbm_step / 8e12, t_pcie) / t_step, pcie_link=link,
                           miss_ratio=d["miss_pages"] / max(d["selected_pages"], 1)),
        roofline=roofline, kernels=kern, error_bits=final["error_bits"])
    n_cold = min(8, len(cold_steps))
    if n_cold:
        # the first steps after prefill start from an empty GPU cache (every selected page misses)
        line["cold_start"] = dict(steps=n_cold, first_step_ms=cold_steps[0],
                                  mean_ms_per_step=sum(cold_steps[:n_cold]) / n_cold)
    if e2e_steps:
        line["e2e"] = dict(value=B * e2e_steps * world / (e2e_ms * 1e-3), unit=unit, h2d_bytes_per_step=h2d,
                           d2h_bytes_per_step=d2h, ms_per_step=e2e_ms / e2e_steps)
    run.close()
    del run
    if world == 1 and not args.no_cpu_baseline:
        r = oracle_run(base, budget_s=20.0, steps_cap=64, warmup=1)
        line["cpu_baseline"] = dict(value=r["value"], unit=unit, cores=r["cores"], kind="oracle", sample=r["sample"])
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
