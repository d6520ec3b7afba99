"""Parity of the CUDA library against the CPU oracle, step by step, through the C ABI.

Integer results (selections, partitions, hit/miss/bypass classes, evictions, page lists,
GPU page table contents, residency bits, counters) and fp32 scores are compared bit for bit;
attention outputs within max-abs 2e-2 and mean-abs 2e-3 (bf16 K/V, fp32 accumulation).
"""
import math

import numpy as np
import pytest
import torch

import workloads as W
from oracle import spin_oracle as O

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3
REL_L2 = 2e-2          # relative L2 error of the outputs of a whole run (bf16 outputs: ~3e-3)


def _wl(kind, **kw):
    base = dict(name="t", seed=77, batch=2, num_layers=2, num_q_heads=8, num_kv_heads=2,
                head_dim=128, page_tokens=16, context=16 * 40 + 5, partition_kind=kind, topk=6,
                slots_per_set=16, lru_buckets=4, steps=24, drift=0.25, kv_recipe="normal")
    base.update(kw)
    return W.Workload(**base)


def run_parity(w, sm_scale=0.0, slots=None, segment_entries=0, check_bytes=True, tol_scale=1.0,
               one_call=False, fetch_mode=0, host_tables_only=0, host_io=None, cache_pages_per_layer=None,
               oracle_reqs=None, budget_schedule=None, spare_cache_pages=0, evict_exact=0,
               offload_stage_bytes=0, resident_scoring=0, reindex_every=0):
    """oracle_reqs: the requests mirrored in the oracle (default all).  Sets are independent, so the
    oracle run on a sample of the batch's requests must agree with those requests of the full batch."""
    from paper_2604_26837_b200.driver import SpinRun
    dev = "cuda:0"
    run = SpinRun(w, dev, trace=True, sm_scale=sm_scale, slots_per_set=slots,
                  segment_entries=segment_entries, fetch_mode=fetch_mode, host_tables_only=host_tables_only,
                  cache_pages_per_layer=cache_pages_per_layer, spare_cache_pages=spare_cache_pages,
                  evict_exact=evict_exact, offload_stage_bytes=offload_stage_bytes,
                  resident_scoring=resident_scoring)
    S = run.slots
    orc = O.SpinOracle(O.OracleConfig(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim,
                                      w.page_tokens, w.partition_kind, w.topk, w.lru_buckets, sm_scale,
                                      bool(evict_exact)))
    sample = list(range(w.batch)) if oracle_reqs is None else list(oracle_reqs)
    oreq = {r: orc.request_open(run.budgets[r]) for r in sample}
    for r in range(w.batch):
        for l in range(w.num_layers):
            k, v, tp, cen = run.gen_prefill(r, l)
            run.prefill(r, l, k, v, tp, cen)
            if r not in oreq:
                continue
            if tp is not None:
                orc.append_kv(oreq[r], l, W.to_bits(k), W.to_bits(v), tp.cpu().numpy(), W.to_bits(cen))
            else:
                orc.append_kv(oreq[r], l, W.to_bits(k), W.to_bits(v))
    qs = {(r, l): W.QueryStream(w, r, l, dev) for r in range(w.batch) for l in range(w.num_layers)}
    out = torch.zeros(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16, device=dev)
    if host_io:                          # q / k / v / out handed over as HOST buffers
        out = torch.zeros(w.batch, w.num_q_heads, w.head_dim, dtype=torch.bfloat16)
        out = out.pin_memory() if host_io == "pinned" else out

    def to_io(x):
        if not host_io:
            return x
        x = x.cpu()
        return x.pin_memory() if host_io == "pinned" else x
    cap_sel = w.topk
    cap_pages = w.topk * max(1, w.max_partition_pages) + (w.steps + 16) // 16 + 2
    worst_abs, worst_mean, rel_num, rel_den = 0.0, 0.0, 0.0, 0.0
    folded = 0
    tied_at_k = 0                    # set-steps whose k-th and (k+1)-th best scores are equal
    for step in range(w.steps):
        for r, new_slots in (budget_schedule or {}).get(step, {}).items():     # buffer elasticity between steps
            run.set_budget(r, new_slots)
            if r in oreq:
                orc.set_budget(oreq[r], new_slots)
        if reindex_every and step and step % reindex_every == 0:                # Index during decode (clusters)
            for r in range(w.batch):
                for l in range(w.num_layers):
                    run.reindex(r, l)
                    if r in oreq:
                        folded += sum(len(x) for x in orc.reindex(oreq[r], l))
        for l in range(w.num_layers):
            kn, vn = run.gen_step_tokens(l, step)
            kb, vb = W.to_bits(kn), W.to_bits(vn)
            for r in sample:
                orc.append_kv(oreq[r], l, kb[r:r + 1], vb[r:r + 1])
            q = torch.stack([qs[(r, l)].next() for r in range(w.batch)]).contiguous()
            kio, vio, qio = to_io(kn), to_io(vn), to_io(q)
            if one_call:                      # spin_decode_step_append: append + decode in one call
                run.step(l, kio, vio, qio, out)
            else:
                run.append(l, kio, vio)
                run.decode(l, qio, out)
            ref = orc.decode_step(l, [oreq[r] for r in sample], W.to_bits(q)[sample])
            torch.cuda.synchronize()
            got = out.float().cpu().numpy().astype(np.float64)[sample]
            err = np.abs(got - ref)
            worst_abs, worst_mean = max(worst_abs, err.max()), max(worst_mean, err.mean())
            rel_num += float((err ** 2).sum())
            rel_den += float((ref ** 2).sum())
            for r in sample:
                for h in range(w.num_kv_heads):
                    tr = orc.last_trace[(oreq[r], l, h)]
                    st = orc.set(oreq[r], l, h)
                    ncand = len(tr.scores)
                    S = run.budgets[r]
                    d = run.spin.debug_dump(run.reqs[r], l, h, cap_sel, cap_pages, S,
                                            st.n_partitions() + 1, ncand + 1)
                    where = f"step {step} layer {l} req {r} head {h}"
                    assert np.array_equal(d["scores"].view(np.uint32), tr.scores.view(np.uint32)), where
                    assert list(d["selected"]) == list(tr.selected), where
                    if ncand > w.topk:
                        ranked = np.sort(tr.scores)[::-1]
                        tied_at_k += int(ranked[w.topk - 1] == ranked[w.topk])
                    assert list(d["parts"]) == list(tr.partitions), where
                    cls = {0: [], 1: [], 2: []}
                    for p, s_ in zip(d["parts"], d["part_state"]):
                        cls[int(s_)].append(int(p))
                    assert cls[0] == tr.hits, where
                    assert sorted(cls[1] + cls[2]) == tr.misses and cls[2] == tr.bypass, where
                    pages = list(zip(d["page_partition"].tolist(), d["page_idx"].tolist(),
                                     d["page_mask"].tolist(), d["page_slot"].tolist()))
                    assert pages == tr.pages, where
                    assert list(d["slot_partition"]) == list(tr.slot_part), where
                    assert list(d["slot_page_idx"]) == list(tr.slot_pidx), where
                    assert list(d["slot_ts"]) == list(tr.slot_ts), where
                    ev = [(s_, int(p), int(i)) for s_, (p, i) in
                          enumerate(zip(d["slot_evicted_partition"], d["slot_evicted_page_idx"])) if p >= 0]
                    assert ev == tr.evicted, where
                    assert list(d["part_resident"]) == list(tr.resident), where
                    assert list(d["part_tokens"]) == st.part_tokens, where
                    assert d["n_tokens"] == st.n_tokens and d["step"] == st.t, where
                    if check_bytes and (step % 5 == 0 or step == w.steps - 1):
                        # Retrieve step 4: every cached slot holds exactly the host page's bytes
                        for s_ in np.nonzero(tr.slot_part >= 0)[0][:: max(1, S // 6)]:
                            p, i = int(tr.slot_part[s_]), int(tr.slot_pidx[s_])
                            gpu = run.spin.debug_read_page(run.reqs[r], l, h, slot=int(s_))
                            host = run.spin.debug_read_page(run.reqs[r], l, h, partition=p, page_idx=i)
                            page = st.cpu_page_table[st.part_offset[p] + i]
                            valid = min(16, st.part_tokens[p] - 16 * i)
                            assert np.array_equal(gpu, host), where
                            assert np.array_equal(gpu[0][:valid], st.page_k[page][:valid]), where
                            assert np.array_equal(gpu[1][:valid], st.page_v[page][:valid]), where
    stats = run.spin.stats()
    assert stats["error_bits"] == 0, (stats["error_bits"], stats["first_error_site"], stats["debug_words"])
    # every set of the batch (not only the mirrored requests) must have counted its appends and steps
    for r in range(w.batch):
        for l in range(w.num_layers):
            for h in range(w.num_kv_heads):
                dd = run.spin.debug_dump(run.reqs[r], l, h, cap_sel, cap_pages, run.budgets[r], 1 << 15)
                assert dd["n_tokens"] == run.ctx[r] + w.steps and dd["step"] == w.steps, (r, l, h, dd["n_tokens"], dd["step"])
    if len(sample) == w.batch:
        for key in ("selected_partitions", "selected_pages", "tail_pages", "hit_pages", "miss_pages",
                    "evicted_pages", "bypass_pages"):
            assert stats[key] == orc.counters[key], key
        assert stats["set_steps"] == orc.counters["steps"]
        assert stats["pcie_bytes"] == orc.step_bytes()["pcie"]
    # properties that hold at any size
    assert stats["set_steps"] == w.batch * w.num_layers * w.num_kv_heads * w.steps
    assert stats["selected_pages"] == stats["hit_pages"] + stats["miss_pages"]
    assert stats["bypass_pages"] <= stats["miss_pages"] and stats["pcie_bytes"] == stats["miss_pages"] * 8192
    assert worst_abs <= MAX_ABS * tol_scale and worst_mean <= MEAN_ABS * tol_scale, (worst_abs, worst_mean)
    # the absolute tolerance says little when the softmax is nearly uniform (outputs of a few
    # hundredths): the relative L2 error over all compared outputs must be small as well
    rel_l2 = math.sqrt(rel_num / max(rel_den, 1e-30))
    assert rel_l2 < REL_L2 * tol_scale, rel_l2
    run.close()
    return dict(folded=folded, max_abs=worst_abs, mean_abs=worst_mean, rel_l2=rel_l2, stats=stats, tied_at_k=tied_at_k)


@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_page_minmax_small(sm_scale):
    r = run_parity(_wl(W.PART_PAGE_MINMAX), sm_scale=sm_scale)
    assert r["rel_l2"] < 2e-2


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_TOKEN_DOT, W.PART_CLUSTER_CENTROID])
def test_append_and_decode_in_one_call(kind):
    # 40 steps cross two page boundaries: both the side-stream append and the serialised one run
    extra = dict(kv_recipe="mixture", num_clusters=23, max_partition_pages=8) if kind == W.PART_CLUSTER_CENTROID else {}
    run_parity(_wl(kind, steps=40, topk=12 if kind == W.PART_TOKEN_DOT else 6, **extra), one_call=True)


@pytest.mark.parametrize("fetch_mode", [0, 1])
def test_host_tables_read_over_the_link_as_in_the_paper(fetch_mode):
    # no HBM mirror: Partition Offset / CPU page table are read from pinned host memory
    run_parity(_wl(W.PART_PAGE_MINMAX, steps=30, topk=10, slots_per_set=7), host_tables_only=1,
               fetch_mode=fetch_mode, one_call=True)
    run_parity(_wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=23, max_partition_pages=8,
                   steps=20), host_tables_only=1, fetch_mode=fetch_mode)


@pytest.mark.parametrize("host_io", ["pinned", "pageable"])
@pytest.mark.parametrize("one_call", [True, False])
def test_host_buffers_in_and_out(host_io, one_call):
    run_parity(_wl(W.PART_PAGE_MINMAX, steps=20), host_io=host_io, one_call=one_call, check_bytes=False)


def test_separate_fetch_kernel_mode():
    run_parity(_wl(W.PART_PAGE_MINMAX, steps=30), fetch_mode=1)
    run_parity(_wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=23, max_partition_pages=8,
                   steps=20), fetch_mode=1, one_call=True)


@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_page_minmax_outlier_keys_gqa4_many_buckets(sm_scale):
    w = _wl(W.PART_PAGE_MINMAX, num_q_heads=8, num_kv_heads=2, kv_recipe="outlier", outlier_channels=4,
            lru_buckets=64, steps=80, topk=8, slots_per_set=24, drift=0.1, context=16 * 70 + 15)
    run_parity(w, sm_scale=sm_scale)


def test_page_minmax_step_counter_passes_bucket_count_and_segments_are_crossed():
    # 16-entry segments: tables span several second-level segments; n=3 buckets: demotion active
    w = _wl(W.PART_PAGE_MINMAX, lru_buckets=3, steps=40, topk=12, slots_per_set=40, context=16 * 100 + 1,
            batch=3, num_layers=1)
    run_parity(w, segment_entries=16)


def test_page_minmax_overflowing_budget_bypasses():
    w = _wl(W.PART_PAGE_MINMAX, topk=10, slots_per_set=7, steps=12)
    r = run_parity(w)
    assert r["stats"]["bypass_pages"] > 0


def test_page_minmax_single_bucket_and_gqa1_gqa8():
    run_parity(_wl(W.PART_PAGE_MINMAX, lru_buckets=1, steps=10, num_q_heads=2, num_kv_heads=2))
    run_parity(_wl(W.PART_PAGE_MINMAX, steps=6, num_q_heads=16, num_kv_heads=2))


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_TOKEN_DOT, W.PART_CLUSTER_CENTROID, W.PART_PAGE_MEAN])
def test_gqa_group_of_two(kind):
    # two query heads per kv head: the score reduction trades one head between lane pairs
    extra = dict(kv_recipe="mixture", num_clusters=19, max_partition_pages=8) if kind == W.PART_CLUSTER_CENTROID else {}
    run_parity(_wl(kind, num_q_heads=4, num_kv_heads=2, steps=10, topk=6 if kind != W.PART_TOKEN_DOT else 50, **extra))


def test_more_slots_than_the_shared_memory_path_holds():
    # > 1024 slots per set: the cache manager works on the page table in global memory
    w = _wl(W.PART_PAGE_MINMAX, context=16 * 1300 + 3, slots_per_set=1100, topk=40, steps=36, batch=1,
            num_layers=1, lru_buckets=8, drift=0.4)
    run_parity(w, check_bytes=False, one_call=True)


def test_mixed_context_lengths_and_per_request_budgets():
    # the mixed-batch configuration in small: contexts drawn per request, query drift drawn per
    # request, budgets split from a per-layer total in proportion to sequence length
    w = _wl(W.PART_PAGE_MINMAX, batch=5, num_layers=1, context=16 * 90, ctx_range=(40, 16 * 90),
            drift_choices=(0.01, 0.1, 0.5), topk=10, steps=30, lru_buckets=8)
    r = run_parity(w, cache_pages_per_layer=2 * 5 * 12, one_call=True)
    assert r["stats"]["evicted_pages"] > 0


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_CLUSTER_CENTROID])
def test_budget_shrinks_and_grows_between_steps(kind):
    # request 0: 20 -> 9 slots (mid-segment cut with 16-entry segments) -> 33 -> 0 -> 12; request 1: 20 -> 26 -> 5
    extra = dict(kv_recipe="mixture", num_clusters=29, max_partition_pages=8) if kind == W.PART_CLUSTER_CENTROID else {}
    w = _wl(kind, steps=34, topk=7, slots_per_set=20, lru_buckets=4, **extra)
    sched = {6: {0: 9}, 11: {0: 33, 1: 26}, 19: {0: 0}, 23: {0: 12, 1: 5}}
    r = run_parity(w, segment_entries=16, budget_schedule=sched, spare_cache_pages=2 * 2 * 40, one_call=True)
    assert r["stats"]["bypass_pages"] > 0 and r["stats"]["evicted_pages"] > 0


@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_page_mean_landmarks(sm_scale):
    # mean-pooled page summaries (Table 1, ShadowKV's Index) scored by q . mean
    w = _wl(W.PART_PAGE_MEAN, steps=36, topk=7, slots_per_set=18, lru_buckets=8, kv_recipe="page_centre")
    run_parity(w, sm_scale=sm_scale, one_call=True)


def test_empty_and_short_contexts():
    # fewer candidates than top-k, and a context shorter than one page (no candidate at all)
    run_parity(_wl(W.PART_PAGE_MINMAX, context=16 * 3 + 2, topk=8, steps=20))
    run_parity(_wl(W.PART_PAGE_MINMAX, context=3, topk=4, steps=30, batch=1, num_layers=1))


@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_token_dot(sm_scale):
    w = _wl(W.PART_TOKEN_DOT, topk=40, slots_per_set=30, kv_recipe="page_centre", steps=20,
            num_q_heads=4, num_kv_heads=1, context=16 * 60 + 9)
    run_parity(w, sm_scale=sm_scale)


def test_token_dot_overflow_and_ties():
    # i.i.d. keys spread the chosen tokens over more pages than the budget holds
    w = _wl(W.PART_TOKEN_DOT, topk=64, slots_per_set=20, steps=10, context=16 * 50)
    r = run_parity(w)
    assert r["stats"]["bypass_pages"] > 0


@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_cluster_centroid(sm_scale):
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=37, topk=5, slots_per_set=30,
            context=16 * 50 + 3, steps=40, max_partition_pages=8, lru_buckets=8)
    run_parity(w, sm_scale=sm_scale)


def test_cluster_centroid_tight_budget_with_empty_clusters():
    # 300 clusters over 400 tokens: many empty and single-token clusters; budget overflows
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=300, topk=20, slots_per_set=12,
            context=400, steps=20, max_partition_pages=4, batch=1)
    run_parity(w)


def test_exact_demand_eviction_variant():
    # the variant that evicts only what the misses need (not the paper's rule): both cache
    # managers (shared-memory copy; page table in global memory), single- and multi-page partitions
    w = _wl(W.PART_PAGE_MINMAX, steps=40, lru_buckets=4, drift=0.4)
    r = run_parity(w, evict_exact=1)
    ref = run_parity(w)
    assert 0 < r["stats"]["evicted_pages"] < ref["stats"]["evicted_pages"]
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=37, topk=5, slots_per_set=30,
            context=16 * 50 + 3, steps=40, max_partition_pages=8, lru_buckets=3)
    run_parity(w, evict_exact=1)
    w = _wl(W.PART_PAGE_MINMAX, context=16 * 1300 + 3, slots_per_set=1100, topk=40, steps=36, batch=1,
            num_layers=1, lru_buckets=4, drift=0.4)
    run_parity(w, check_bytes=False, one_call=True, evict_exact=1)


def test_token_dot_more_keys_than_one_cta_holds():
    # > 16384 candidate keys per set: scoring, then one thread-block cluster per set for the
    # top-k (ragged slices: 20800 keys over 4 CTAs), which starts on the set's scored flag and
    # whose first CTA goes on as the cache manager; and the same with more slots than the
    # shared-memory cache manager takes, so that the cluster only selects and k_cache follows
    w = _wl(W.PART_TOKEN_DOT, context=16 * 1300 + 5, topk=300, slots_per_set=120, steps=20, batch=2,
            num_layers=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8, drift=0.3, kv_recipe="page_centre", centre_sd=0.5)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["stats"]["evicted_pages"] > 0
    w = _wl(W.PART_TOKEN_DOT, context=16 * 1300 + 5, topk=300, slots_per_set=1100, steps=6, batch=1,
            num_layers=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8, drift=0.3, kv_recipe="page_centre", centre_sd=0.5)
    run_parity(w, check_bytes=False, one_call=True)


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_TOKEN_DOT])
def test_asynchronous_offload_of_prefill_pages(kind):
    # prefill pages go through a staging ring (4 slots x 3 pages x 2 kv heads here, so a
    # 40-page prefill wraps the ring several times) and reach host memory on the library's own
    # stream; the first decode step waits for them; results and host bytes as without it
    w = _wl(kind, topk=6 if kind == W.PART_PAGE_MINMAX else 64, steps=12)
    r = run_parity(w, offload_stage_bytes=4 * 3 * 2 * 8192, check_bytes=True)
    assert r["stats"]["miss_pages"] > 0


def test_asynchronous_offload_of_a_cluster_prefill():
    # cluster granularity: the prefill's rows are packed into the clusters' pages in the staging
    # ring (4 slots x 3 pages x 2 kv heads: ~90 pages per head wrap it many times), with heads
    # that own different numbers of pages; host bytes, traces and outputs as written through
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=37, topk=5, slots_per_set=30,
            context=16 * 50 + 3, steps=16, max_partition_pages=8, lru_buckets=8)
    r = run_parity(w, offload_stage_bytes=4 * 3 * 2 * 8192, check_bytes=True, one_call=True)
    assert r["stats"]["miss_pages"] > 0
    # and with Index during decode folding tail pages into clusters whose pages came through the ring
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=23, topk=5, slots_per_set=40,
            context=16 * 30 + 7, steps=44, max_partition_pages=12, lru_buckets=8, batch=2, num_layers=1)
    r = run_parity(w, offload_stage_bytes=4 * 4 * 2 * 8192, reindex_every=20)
    assert r["folded"] == 2 * 2 * 32


def test_token_dot_more_keys_resident_scoring_grid():
    # the queue-fed resident scoring grid in front of the cluster top-k: several items per CTA,
    # ragged last segments, tail items
    w = _wl(W.PART_TOKEN_DOT, context=16 * 1300 + 5, topk=300, slots_per_set=120, steps=20, batch=2,
            num_layers=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8, drift=0.3, kv_recipe="page_centre", centre_sd=0.5)
    r = run_parity(w, check_bytes=False, one_call=True, resident_scoring=1)
    assert r["stats"]["evicted_pages"] > 0


def test_page_minmax_more_pages_than_one_cta_holds():
    # > 16384 candidate PAGES per set (a 264K-token context): the thread-block cluster selects
    # whole partitions here (no token masks), its first CTA manages the cache
    w = _wl(W.PART_PAGE_MINMAX, context=16 * 16500 + 3, topk=64, slots_per_set=100, steps=6, batch=1,
            num_layers=1, num_q_heads=2, num_kv_heads=1, lru_buckets=8, drift=0.3)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["stats"]["miss_pages"] > 0


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_CLUSTER_CENTROID, W.PART_TOKEN_DOT])
def test_resident_scoring_grid(kind):
    # the queue-fed form of the scoring kernel (automatic only for long scoring phases), forced
    # on: mixed lengths (requests own different numbers of work items), an empty request,
    # steps that complete a page (stand-alone append first) and steps that do not
    if kind == W.PART_CLUSTER_CENTROID:
        w = _wl(kind, kv_recipe="mixture", num_clusters=37, topk=5, slots_per_set=30,
                context=16 * 50 + 3, steps=24, max_partition_pages=8, lru_buckets=8)
    else:
        w = _wl(kind, batch=5, num_layers=1, context=16 * 300, ctx_range=(0, 16 * 300),
                drift_choices=(0.01, 0.1, 0.5), topk=10 if kind == W.PART_PAGE_MINMAX else 100, steps=36, lru_buckets=8)
    r = run_parity(w, one_call=True, resident_scoring=1, check_bytes=kind != W.PART_CLUSTER_CENTROID)
    assert r["stats"]["miss_pages"] > 0


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_CLUSTER_CENTROID, W.PART_TOKEN_DOT, W.PART_PAGE_MEAN])
def test_streaming_scoring_kernel(kind):
    # the streaming form of scoring (ring of TMA stages, a selection CTA per set, scores handed
    # over word by word): mixed lengths with an empty request, ragged last stages, steps that
    # complete a page, query groups of 4, 2 and 1; scores must stay bit-exact
    if kind == W.PART_CLUSTER_CENTROID:
        w = _wl(kind, kv_recipe="mixture", num_clusters=37, topk=5, slots_per_set=30,
                context=16 * 50 + 3, steps=24, max_partition_pages=8, lru_buckets=8)
    else:
        w = _wl(kind, batch=5, num_layers=1, context=16 * 300, ctx_range=(0, 16 * 300),
                drift_choices=(0.01, 0.1, 0.5), topk=10 if kind != W.PART_TOKEN_DOT else 100, steps=36, lru_buckets=8)
    r = run_parity(w, one_call=True, resident_scoring=2, check_bytes=kind == W.PART_PAGE_MINMAX)
    assert r["stats"]["miss_pages"] > 0
    for hq in (4, 2):
        run_parity(_wl(kind if kind != W.PART_CLUSTER_CENTROID else W.PART_PAGE_MINMAX, num_q_heads=hq, num_kv_heads=2,
                       steps=12, context=16 * 70 + 9), one_call=True, resident_scoring=2, check_bytes=False)


def test_streaming_scoring_kernel_with_the_cluster_top_k_and_ties():
    # > 16384 candidate keys per set: streaming scoring, then the thread-block cluster per set that
    # takes the scores out of the hand-over buffer; tied scores across the slices
    w = _wl(W.PART_TOKEN_DOT, context=16 * 1300 + 5, topk=300, slots_per_set=120, steps=10, batch=2,
            num_layers=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8, drift=0.3, kv_recipe="tied", tie_period=1000)
    r = run_parity(w, check_bytes=False, one_call=True, resident_scoring=2)
    assert r["tied_at_k"] == 2 * 2 * 10


def test_cluster_tail_is_folded_into_the_clusters_during_decode():
    # Index during decode: every 20 steps the full tail pages join the clusters of their best
    # centroids (new cluster pages, stale residency dropped, layout rewritten, tail rotated);
    # selections, cache traces, page lists, host bytes and outputs stay equal to the oracle's
    w = _wl(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=23, topk=5, slots_per_set=40,
            context=16 * 30 + 7, steps=70, max_partition_pages=12, lru_buckets=8, batch=2, num_layers=2)
    r = run_parity(w, reindex_every=20)
    assert r["stats"]["miss_pages"] > 0 and r["folded"] == 2 * 2 * 2 * 48


def test_tiny_configuration_full_size():
    # the first benchmark configuration as stated: 4096-token context, top-16, 64 slots, 8 buckets
    r = run_parity(W.CONFIGS["c1"], check_bytes=False, one_call=True)
    assert r["stats"]["set_steps"] == 32 and r["stats"]["evicted_pages"] > 0
