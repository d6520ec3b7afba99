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


def measure_pcie_gbs(torch, device, stream) -> dict:
    """Peak of the host link, host to device: the better of a large pinned copy-engine transfer
    (best of 10) and of SM-issued reads of pinned memory by a grid that fills the GPU (the
    library's link probe, best of 6).  The host is shared with other jobs, so single
    measurements wander by 10-20%; the best one is the link's peak."""
    import paper_2604_26837_b200 as P
    n = 256 << 20
    src = torch.empty(n, dtype=torch.uint8).pin_memory()
    dst = torch.empty(n, dtype=torch.uint8, device=device)
    dma = 0.0
    with torch.cuda.stream(stream):
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            dst.copy_(src, non_blocking=True)
            e1.record(stream)
            e1.synchronize()
            dma = max(dma, n / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    del src, dst
    # a small context just for its pinned host tier (256 MiB of pages)
    cfg = P.make_config(device=device.index or 0, num_layers=1, num_q_heads=4, num_kv_heads=1, max_requests=1,
                        max_context_tokens=4096, partition_kind=0, topk=16, gpu_cache_pages=64, host_pages=32768)
    ctx = P.Spin(cfg, device)
    sm = 0.0
    with torch.cuda.stream(stream):
        for _ in range(7):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            ctx.debug_link_probe(32768, stream)
            e1.record(stream)
            e1.synchronize()
            sm = max(sm, 32768 * 8192 / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    ctx.close()
    return dict(gbs=max(dma, sm), copy_engine_gbs=dma, sm_read_gbs=sm,
                source="best of a 256 MiB pinned copy-engine transfer and of SM-issued reads of pinned memory, measured in this run")


def oracle_run(w, budget_s: float, steps_cap: int, warmup: int, sample_requests: int = 1, first_request: int = 0):
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
    ids = list(range(first_request, first_request + sample_requests))       # requests of the workload that are run
    for r in ids:
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
    qs = {(r, l): W.QueryStream(w, r, l) for r in ids for l in range(w.num_layers)}
    times = []
    step = 0
    t_start = time.perf_counter()
    while True:
        ins = []
        for l in range(w.num_layers):
            kv = [W.kv_tokens(w, r, l, w.request_context(r) + step, 1) for r in ids]
            q = np.stack([W.to_bits(qs[(r, l)].next()) for r in ids])
            ins.append((l, [(W.to_bits(k), W.to_bits(v)) for k, v in kv], q))
        t0 = time.perf_counter()
        for l, kv, q in ins:
            for i_, (kb, vb) in enumerate(kv):
                orc.append_kv(reqs[i_], l, kb, vb)
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


def workload_bytes(w, d):
    """Algorithmic bytes of the counted set-steps `d` (differences of spin_stats): HBM = summaries
    scanned + selected KV read once + the tail pages + missed pages written into their slots;
    host link = missed pages.  Token-granular selection reads the selected token ROWS (512 B of
    K and V each) of the selected pages, not whole pages."""
    summ = d["candidates_scored"] * (512 if w.partition_kind == 0 else 256)
    admit = (d["miss_pages"] - d["bypass_pages"]) * PAGE_BYTES
    if w.partition_kind == 1:
        cand_per_set = (w.context // w.page_tokens) * w.page_tokens
        kv = d["set_steps"] * min(w.topk, cand_per_set) * 512 + d["tail_pages"] * PAGE_BYTES
    else:
        kv = (d["selected_pages"] + d["tail_pages"]) * PAGE_BYTES
    return dict(hbm=summ + kv + admit, pcie=d["miss_pages"] * PAGE_BYTES, summaries=summ, kv=kv, admit=admit)


def measure(base, args, K, Wm, rank, world, device, do_e2e, pcie_gbs, peaks, cache_pages_per_layer):
    """Prefill, prime the cache to its steady state, warm up, time K steps of one workload.
    Returns the record of this rank (times in ms; stats differences over the timed window)."""
    import torch
    import workloads as W
    from paper_2604_26837_b200.driver import SpinRun
    prime_cap = args.prime_cap
    prof_steps = min(K, 32)
    e2e_steps = K if do_e2e else 0
    total_steps = prime_cap + Wm + K + K + prof_steps + (Wm + e2e_steps)
    w = rank_workload(base, rank, total_steps)
    run = SpinRun(w, device, fetch_mode=args.fetch_mode, cache_pages_per_layer=cache_pages_per_layer,
                  resident_scoring=args.resident_scoring)
    stream = torch.cuda.Stream(device)
    B, L = w.batch, w.num_layers
    t_setup = time.perf_counter()
    with torch.cuda.stream(stream):
        for r in range(B):
            for l in range(L):
                k, v, tp, cen = run.gen_prefill(r, l)
                run.prefill(r, l, k, v, tp, cen, stream)
                del k, v
        qstreams = {(r, l): W.QueryStream(w, r, l, device) for r in range(B) for l in range(L)}
        out = torch.zeros(B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        flush = torch.empty(64 << 20, dtype=torch.int32, device=device)        # 256 MiB
    torch.cuda.synchronize(device)
    cur = [0]

    def gen_inputs(n):
        """Inputs of the next n decode steps, resident in HBM before any timed region."""
        q_ = torch.empty(n, L, B, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        k_ = torch.empty(n, L, B, w.num_kv_heads, w.head_dim, dtype=torch.bfloat16, device=device)
        v_ = torch.empty_like(k_)
        with torch.cuda.stream(stream):
            for i in range(n):
                for l in range(L):
                    k_[i, l], v_[i, l] = run.gen_step_tokens(l, cur[0] + i)
                    for r in range(B):
                        q_[i, l, r] = qstreams[(r, l)].next()
        torch.cuda.synchronize(device)
        return q_, k_, v_

    def flush_l2_fn():
        # write 256 MiB (> 126 MB L2), then read it back so that the L2 is left full of CLEAN
        # lines, as it is after the weights of a model's other layers have streamed through;
        # a write-only flush would leave dirty lines whose write-back taxes the timed kernels
        flush.zero_()
        flush.max()

    def timed_steps(n, flush_l2=True):
        q_, k_, v_ = gen_inputs(n)
        evs = []
        with torch.cuda.stream(stream):
            for i in range(n):
                if flush_l2:
                    flush_l2_fn()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for l in range(L):
                    run.step(l, k_[i, l], v_[i, l], q_[i, l], out, stream)
                e1.record(stream)
                evs.append((e0, e1))
        torch.cuda.synchronize(device)
        cur[0] += n
        return [a.elapsed_time(b) for a, b in evs]

    # cold start, then priming until the cache is in its steady state: the slots are full and
    # every step evicts (Section 5.3 step 3 has work to do), or the cap is reached
    cold_steps = timed_steps(8)
    primed, evicting_chunks = 8, 0
    while primed < prime_cap and evicting_chunks < 2:
        s0 = run.spin.stats()
        timed_steps(8, flush_l2=False)
        s1 = run.spin.stats()
        primed += 8
        evicting_chunks = evicting_chunks + 1 if s1["evicted_pages"] > s0["evicted_pages"] else 0
    timed_steps(Wm)
    st0 = run.spin.stats()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.synchronize(device)
        dist.barrier()
    t_begin = datetime.datetime.now()
    per_step = timed_steps(K)
    if world > 1:
        torch.cuda.synchronize(device)
        dist.barrier()
    t_end = datetime.datetime.now()
    st1 = run.spin.stats()
    # back-to-back variant without the L2 flush (one pair of events around all K steps)
    q_, k_, v_ = gen_inputs(K)
    with torch.cuda.stream(stream):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(K):
            for l in range(L):
                run.step(l, k_[i, l], v_[i, l], q_[i, l], out, stream)
        e1.record(stream)
    torch.cuda.synchronize(device)
    cur[0] += K
    noflush_ms = e0.elapsed_time(e1) / K
    # per-kernel durations, measured live with CUDA events recorded between the launches
    stp0 = run.spin.stats()
    run.spin.profile(True)
    timed_steps(prof_steps)
    prof = run.spin.profile_read()
    run.spin.profile(False)
    stp1 = run.spin.stats()
    rec = dict(w=w, per_step=per_step, noflush_ms=noflush_ms, cold_steps=cold_steps, primed=primed,
               t_begin=t_begin, t_end=t_end, prof=prof, B=B, L=L)
    skip = ("error_bits", "debug_words", "status")
    rec["d"] = {k: st1[k] - st0[k] for k in st0 if k not in skip}
    rec["dp"] = {k: stp1[k] - stp0[k] for k in stp0 if k not in skip}
    # end to end: host buffers in, host buffer out, every step
    if e2e_steps:
        q_, k_, v_ = gen_inputs(Wm + e2e_steps)
        qh, kh, vh = q_.cpu().pin_memory(), k_.cpu().pin_memory(), v_.cpu().pin_memory()
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
        rec["e2e_ms"] = 1e3 * sum(e2e_times)
        rec["h2d"] = L * (qh[0, 0].numel() + kh[0, 0].numel() + vh[0, 0].numel()) * 2
        rec["d2h"] = L * oh.numel() * 2
    # the design's latency floor: two chained launches and one flag hand-over, timed like a step
    floor = []
    with torch.cuda.stream(stream):
        for _ in range(24):
            flush_l2_fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            run.spin.debug_launch_floor(stream)
            e1.record(stream)
            floor.append((e0, e1))
    torch.cuda.synchronize(device)
    rec["floor_us"] = 1e3 * statistics.median(a.elapsed_time(b) for a, b in floor[4:])
    rec["final"] = run.spin.stats()
    rec["setup_s"] = time.perf_counter() - t_setup
    run.close()
    del run
    torch.cuda.empty_cache()
    return rec


def summarise(rec, args, K, world, elapsed_ms, pcie_gbs, peaks, fused, full_size):
    """The figures of one workload: throughput, step roofline, per-kernel table, dominant kernel."""
    w, d, dp, prof, B = rec["w"], rec["d"], rec["dp"], rec["prof"], rec["B"]
    per_step = rec["per_step"]
    by = workload_bytes(w, d)
    hbm_step, pcie_step = by["hbm"] / K, by["pcie"] / K
    t_hbm = hbm_step / (peaks["hbm_gbs"] * 1e9)
    t_pcie = pcie_step / (pcie_gbs * 1e9)
    t_step = elapsed_ms * 1e-3 / K
    byp = workload_bytes(w, dp)
    miss_b, admit_b = byp["pcie"], byp["admit"]
    # algorithmic bytes per kernel over the profiled steps: (HBM bytes, host-link bytes)
    bytes_of = dict(score=(byp["summaries"], 0), fetch=(admit_b, admit_b),
                    attn_split=((byp["kv"] - miss_b + admit_b, miss_b) if fused else (byp["kv"] - (miss_b - admit_b), miss_b - admit_b)))
    kern = {}
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
    traffic = (NCU_TRAFFIC.get(w.name) or {}).get(top) if full_size else None
    names = dict(fetch="k_fetch", score="k_score", attn_split="k_attn (attention + page fetch)" if fused else "k_attn")
    roofline = dict(kernel=names[top], bound=bound, achieved=achieved, peak=peak, unit="GB/s",
                    frac=kern[top]["roof_frac"], traffic=traffic,
                    peak_source=("host link peak measured in this run (see step_roofline.pcie_peak)" if bound == "pcie" else peaks["source"]),
                    avg_launch_us=kern[top]["avg_us"],
                    hbm_bytes_per_launch=bytes_of[top][0] / kern[top]["launches"],
                    pcie_bytes_per_launch=bytes_of[top][1] / kern[top]["launches"])
    step_roofline = dict(hbm_bytes_per_step=hbm_step, pcie_bytes_per_step=pcie_step,
                         hbm_gbs_peak=peaks["hbm_gbs"], hbm_peak_source=peaks["source"], pcie_gbs_peak=pcie_gbs,
                         t_hbm_us=1e6 * t_hbm, t_pcie_us=1e6 * t_pcie, t_step_us=1e6 * t_step,
                         bound="pcie" if t_pcie > t_hbm else "hbm", frac=max(t_hbm, t_pcie) / t_step,
                         frac_vs_nominal_8tbs=max(hbm_step / 8e12, t_pcie) / t_step,
                         miss_ratio=d["miss_pages"] / max(d["selected_pages"], 1))
    sets = d["set_steps"] / K
    return dict(value=aggregate_value(B * K, world, elapsed_ms), ms_per_step=elapsed_ms / K,
                p50_tpot_ms=statistics.median(per_step), ms_per_step_noflush=rec["noflush_ms"],
                step_roofline=step_roofline, roofline=roofline, kernels=kern,
                miss_ratio=step_roofline["miss_ratio"], evicted_pages_per_step=d["evicted_pages"] / K,
                missed_pages_per_step=d["miss_pages"] / K, sets_per_step=sets, primed_steps=rec["primed"],
                gpu_launches=int(d["kernel_launches"]), error_bits=rec["final"]["error_bits"],
                setup_s=round(rec["setup_s"], 1),
                latency_floor=dict(us=rec["floor_us"], step_over_floor=(elapsed_ms / K * 1e3) / max(rec["floor_us"], 1e-9),
                                   what="two empty kernels chained by programmatic dependent launch with one flag "
                                        "hand-over, same stream, CUDA events, L2 flushed: what a step costs before it touches KV"))


def workload_desc(base, world):
    return dict(workload=f"{base.name}: batch {base.batch} x {base.num_layers} layer(s), "
                         f"{base.num_q_heads}q/{base.num_kv_heads}kv heads, context {base.context}, "
                         f"kind {base.partition_kind}, top-k {base.topk}, "
                         f"{base.slots_per_set if base.slots_per_set else 'dynamic'} slots/set, "
                         f"{base.lru_buckets} buckets, drift {base.drift}",
                global_batch=base.batch * world, context=base.context, parallelism=f"replicas x{world}")


def _oracle_worker(args):
    name, kw, budget_s, steps_cap, r = args
    import workloads as W
    base = W.scaled(W.CONFIGS[name], **kw)
    return oracle_run(base, budget_s, steps_cap, 1, sample_requests=1, first_request=r)


def oracle_all_cores(base_name, kw, budget_s, steps_cap):
    """The oracle on every host core at once: one process per request (requests are independent),
    each a single numpy thread; throughput = requests x steps over the slowest process's time."""
    import multiprocessing as mp
    import workloads as W
    base = W.scaled(W.CONFIGS[base_name], **kw)
    n = min(os.cpu_count() or 1, base.batch)
    ctx = mp.get_context("spawn")
    t0 = time.perf_counter()
    with ctx.Pool(n) as pool:
        res = pool.map(_oracle_worker, [(base_name, kw, budget_s, steps_cap, r) for r in range(n)])
    wall = time.perf_counter() - t0
    steps = min(r["steps"] for r in res)
    slowest = max(r["ms_per_step"] for r in res)
    return dict(value=n / (slowest * 1e-3), unit="tokens/s", cores=n, nproc=os.cpu_count(), kind="oracle",
                sample=f"{n} of {base.batch} requests in {n} processes (one numpy thread each) x {steps} decode steps; "
                       f"rate = requests over the slowest process's mean step time", wall_s=round(wall, 1))


def parse_cpulist(text):
    """'0-3,8,10-11' -> [0, 1, 2, 3, 8, 10, 11]"""
    cpus = []
    for part in text.strip().split(","):
        if not part:
            continue
        lo, _, hi = part.partition("-")
        cpus.extend(range(int(lo), int(hi or lo) + 1))
    return cpus


def bind_near_gpu(props, sysfs="/sys/bus/pci/devices"):
    """Pin this process to the CPUs local to its GPU (the PCI device's local_cpulist), so that the
    pinned host tier it allocates next is first touched, and hence placed, on the GPU's NUMA node:
    with several replicas each pulling tens of GB/s over its own link, host-memory placement
    decides the scaling curve.  A no-op where the file is missing or lists every CPU (a
    single-node host).  Returns what it did, for the JSON line."""
    try:
        bus = "%04x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
        with open(os.path.join(sysfs, bus, "local_cpulist")) as f:
            local = set(parse_cpulist(f.read()))
        allowed = os.sched_getaffinity(0)
        target = local & allowed
        if not target or target == allowed:
            return dict(bound=False, local_cpus=len(local), why="single node or no locality information")
        os.sched_setaffinity(0, target)
        return dict(bound=True, local_cpus=len(target))
    except (OSError, AttributeError, ValueError) as e:
        return dict(bound=False, why=type(e).__name__)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--impl", default="spin", choices=["spin", "reference"])
    ap.add_argument("--prime-cap", type=int, default=160,
                    help="at most this many untimed decode steps to bring the KV cache to its steady state (setup)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="only the headline workload, not the other configurations")
    ap.add_argument("--per-config-steps", type=int, default=32)
    ap.add_argument("--resident-scoring", type=int, default=0,
                    help="spin_config.resident_scoring: 0 automatic, 1 queue-fed resident grid, -1 one CTA per item, 2 streaming")
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
    overrides = {}
    if args.context:
        overrides["context"] = args.context
    if args.batch:
        overrides["batch"] = args.batch
    if args.layers:
        overrides["num_layers"] = args.layers
    base = W.scaled(W.CONFIGS[args.workload], **overrides)

    def cache_budget(b):
        # a workload without a fixed budget states a total: 60 GB of KV over its 32 layers and 64
        # requests; a scaled run keeps the per-layer, per-request share
        return int(60e9 / 32 / PAGE_BYTES * b.batch / 64) if b.slots_per_set == 0 else None
    metric, unit = "decode_tokens_per_s", "tokens/s"
    cfg_desc = workload_desc(base, world)

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

    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    numa = bind_near_gpu(torch.cuda.get_device_properties(device))     # before any pinned allocation
    K, Wm = args.steps, args.warmup
    peaks = load_peaks()
    link_peak = measure_pcie_gbs(torch, device, torch.cuda.Stream(device))
    pcie_gbs = link_peak["gbs"]
    props = torch.cuda.get_device_properties(device)
    gpu_id = f"GPU-{props.uuid}" if hasattr(props, "uuid") else str(local_rank)
    fused = args.fetch_mode == 0
    full_size = not overrides

    sampler = ClockSampler(gpu_id)
    rec = measure(base, args, K, Wm, rank, world, device, not args.no_e2e, pcie_gbs, peaks, cache_budget(base))
    clocks = sampler.stop(rec["t_begin"], rec["t_end"])
    link = pcie_link(gpu_id)
    elapsed_ms = sum(rec["per_step"])
    e2e_ms = rec.get("e2e_ms", 0.0)
    noflush_ms = rec["noflush_ms"]
    if world > 1:
        elapsed_ms, e2e_ms, noflush_ms = allreduce_max([elapsed_ms, e2e_ms, noflush_ms], device)
        rec["noflush_ms"] = noflush_ms
    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    head = summarise(rec, args, K, world, elapsed_ms, pcie_gbs, peaks, fused, full_size)
    head["step_roofline"]["pcie_link"] = link
    head["step_roofline"]["pcie_peak"] = link_peak
    line = dict(
        metric=metric, value=head["value"], unit=unit, n_gpus=world, steps=K, warmup=Wm, ms_per_step=head["ms_per_step"],
        higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16 in, f32 accumulate", data="synthetic",
        config=dict(cfg_desc, primed_steps=head["primed_steps"],
                    prime="untimed decode steps until the slots are full and every step evicts (cap --prime-cap)",
                    l2="flushed between timed steps (256 MiB written then read back, untimed)",
                    note="single-layer config: tokens/s is per-layer-step throughput"),
        p50_tpot_ms=head["p50_tpot_ms"], ms_per_step_noflush=head["ms_per_step_noflush"],
        gpu_launches=head["gpu_launches"], clocks=clocks, numa=numa, step_roofline=head["step_roofline"],
        roofline=head["roofline"], kernels=head["kernels"], miss_ratio=head["miss_ratio"],
        evicted_pages_per_step=head["evicted_pages_per_step"], missed_pages_per_step=head["missed_pages_per_step"],
        latency_floor=head["latency_floor"], error_bits=head["error_bits"])
    cold_steps = rec["cold_steps"]
    n_cold = min(8, len(cold_steps))
    if n_cold:
        # the first steps after prefill start from an empty GPU cache (every selected page misses)
        line["cold_start"] = dict(steps=n_cold, first_step_ms=cold_steps[0],
                                  mean_ms_per_step=sum(cold_steps[:n_cold]) / n_cold)
    if "e2e_ms" in rec:
        line["e2e"] = dict(value=rec["B"] * K * world / (e2e_ms * 1e-3), unit=unit, h2d_bytes_per_step=rec["h2d"],
                           d2h_bytes_per_step=rec["d2h"], ms_per_step=e2e_ms / K)

    # the other benchmark configurations, each at its full size (the mixed-length one scaled to
    # this box and labelled), fewer timed steps: which of them meet the roofline target
    if world == 1 and not args.no_per_config and full_size and args.workload == "c2":
        per = {}
        others = [("c1", {}, "as worded"), ("c3", {}, "as worded"), ("c4", {}, "as worded"),
                  ("c5_scaled", dict(batch=16, num_layers=1),
                   "SCALED to this box: 16 of the 64 requests, 1 of the 32 layers, the same per-request and "
                   "per-layer share of the 60 GB budget (the configuration as worded needs ~1.1 TB of pinned host memory)")]
        Kp = args.per_config_steps
        for name, kw, label in others:
            b2 = W.scaled(W.CONFIGS[name.split("_")[0]], **kw)
            smp = ClockSampler(gpu_id)
            r2 = measure(b2, args, Kp, Wm, 0, 1, device, False, pcie_gbs, peaks, cache_budget(b2))
            ck = smp.stop(r2["t_begin"], r2["t_end"])
            s2 = summarise(r2, args, Kp, 1, sum(r2["per_step"]), pcie_gbs, peaks, fused, not kw)
            s2.update(config=workload_desc(b2, 1)["workload"], size=label, steps=Kp, clocks=ck,
                      meets_0p60=bool(s2["step_roofline"]["frac"] >= 0.60))
            s2.pop("kernels")
            per[name] = s2
        line["per_config"] = per
        line["target"] = dict(step_roofline_frac=0.60,
                              met={**{"c2": bool(head["step_roofline"]["frac"] >= 0.60)},
                                   **{k_: v_["meets_0p60"] for k_, v_ in per.items()}})
    if world == 1 and not args.no_cpu_baseline:
        r = oracle_run(base, budget_s=15.0, steps_cap=64, warmup=1)
        line["cpu_baseline"] = dict(value=r["value"], unit=unit, cores=r["cores"], kind="oracle", sample=r["sample"])
        line["cpu_baseline_all_cores"] = oracle_all_cores(args.workload, overrides, 15.0, 64)
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
