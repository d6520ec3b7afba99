"""spin_paged_attention_static: the allocation-free attention entry point.

Some users of this library run where they may not allocate GPU memory at all (inside another
component's fixed memory budget, or on a path where the allocator must not be touched), so
they cannot build a context.  For them the library carries its split-K scratch as a built-in
array.  This test drives the entry point through the C ABI with page lists taken from a
normal decode step and checks, on two calls in a row (the second reuses the array with the
first call's leftovers in it), that the output matches spin_decode_step's; further cases
(full and empty lists, one page, chunk boundaries, groups of 1 and 8, hundreds of chunks)
compare it with the CPU oracle's fp64 attention over the same rows.  Only well-formed inputs
are used.
"""
import numpy as np
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS, MEAN_ABS = 2e-2, 2e-3


def test_static_attention_matches_decode_step_twice_in_a_row():
    import paper_2604_26837_b200 as P
    from paper_2604_26837_b200.driver import SpinRun
    dev = "cuda:0"
    w = W.Workload(name="na", seed=5, batch=2, num_layers=1, num_q_heads=8, num_kv_heads=2, head_dim=128,
                   page_tokens=16, context=16 * 37 + 6, partition_kind=W.PART_PAGE_MINMAX, topk=20,
                   slots_per_set=32, lru_buckets=8, steps=5, drift=0.2, kv_recipe="normal")
    run = SpinRun(w, dev, trace=True)
    G, H, T, d = w.group, w.num_kv_heads, 16, 128
    ks, vs = [], []
    for r in range(w.batch):
        k, v, _, _ = run.gen_prefill(r, 0)
        run.prefill(r, 0, k, v)
        ks.append(k)
        vs.append(v)
    qs = [W.QueryStream(w, r, 0, dev) for r in range(w.batch)]
    out = torch.zeros(w.batch, w.num_q_heads, d, dtype=torch.bfloat16, device=dev)
    for step in range(w.steps):
        kn, vn = run.gen_step_tokens(0, step)
        run.append(0, kn, vn)
        for r in range(w.batch):
            ks[r] = torch.cat([ks[r], kn[r:r + 1]])
            vs[r] = torch.cat([vs[r], vn[r:r + 1]])
        q = torch.stack([s.next() for s in qs]).contiguous()
        run.decode(0, q, out)
    torch.cuda.synchronize()
    ref = out.float().cpu().numpy()

    # page pool of all four sets, laid out as the library's pages: 16 K rows, then 16 V rows
    n_tok = ks[0].shape[0]
    pages_per_set = (n_tok + T - 1) // T
    pool = torch.zeros(w.batch * H * pages_per_set, 2, T, d, dtype=torch.bfloat16, device=dev)
    for r in range(w.batch):
        for h in range(H):
            base = (r * H + h) * pages_per_set
            kk = torch.zeros(pages_per_set * T, d, dtype=torch.bfloat16, device=dev)
            vv = torch.zeros_like(kk)
            kk[:n_tok], vv[:n_tok] = ks[r][:, h], vs[r][:, h]
            pool[base:base + pages_per_set, 0] = kk.view(pages_per_set, T, d)
            pool[base:base + pages_per_set, 1] = vv.view(pages_per_set, T, d)
    stride = w.topk + 3
    n_sets = w.batch * H
    ids = np.zeros((n_sets, stride), dtype=np.int32)
    masks = np.zeros((n_sets, stride), dtype=np.uint32)
    counts = np.zeros(n_sets, dtype=np.int32)
    for r in range(w.batch):
        for h in range(H):
            dmp = run.spin.debug_dump(run.reqs[r], 0, h, w.topk, stride, run.slots, pages_per_set + 1)
            s = r * H + h
            n = len(dmp["page_partition"])
            counts[s] = n
            for i in range(n):
                part = int(dmp["page_partition"][i])
                page = part if part >= 0 else pages_per_set - 1          # the tail is the newest page
                ids[s, i] = s * pages_per_set + page
                masks[s, i] = dmp["page_mask"][i]
    ids_d, masks_d, counts_d = (torch.from_numpy(x).to(dev) for x in (ids, masks, counts))
    q_sets = q.view(w.batch, H, G, d).reshape(n_sets, G, d).contiguous()
    before = torch.cuda.memory_allocated()
    for call in range(2):
        got = torch.full((n_sets, G, d), float("nan"), dtype=torch.bfloat16, device=dev)
        rc = P.spin_paged_attention_static(q_sets, pool, ids_d, masks_d, counts_d, n_sets, stride, G, 0.0,
                                           got, torch.cuda.current_stream())
        assert rc == 0
        torch.cuda.synchronize()
        g = got.float().cpu().numpy().reshape(w.batch, w.num_q_heads, d)
        err = np.abs(g - ref)
        assert np.isfinite(g).all(), f"call {call}"
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (call, err.max(), err.mean())
        del got
    assert torch.cuda.memory_allocated() == before
    # a request beyond the built-in scratch is refused, nothing runs
    rc = P.spin_paged_attention_static(q_sets, pool, ids_d, masks_d, counts_d, 1 << 20, stride, G, 0.0,
                                       q_sets, torch.cuda.current_stream())
    assert rc == 1
    run.close()


def _static_case(group, counts, stride, seed, n_pool_pages=None, sm_scale=0.0):
    """Random pool, lists and masks -> (library output, fp64 reference) for one call."""
    import paper_2604_26837_b200 as P
    from oracle import spin_oracle as O
    dev, T, d = "cuda:0", 16, 128
    n_sets = len(counts)
    g = torch.Generator(device="cpu").manual_seed(seed)
    n_pool = n_pool_pages or (sum(counts) + 3)
    pool = torch.randn(n_pool, 2, T, d, generator=g).to(torch.bfloat16)
    q = torch.randn(n_sets, group, d, generator=g).to(torch.bfloat16)
    rng = np.random.default_rng(seed)
    ids = np.full((n_sets, stride), -1, dtype=np.int32)              # unused entries are never read
    masks = np.zeros((n_sets, stride), dtype=np.uint32)
    perm = rng.permutation(n_pool)
    at = 0
    for s, n in enumerate(counts):
        ids[s, :n] = perm[at:at + n]
        at += n
        masks[s, :n] = rng.integers(0, 1 << 16, size=n, dtype=np.uint32)
        if n > 2:
            masks[s, 1] = 0                                          # a listed page with no token attended
            masks[s, 0] = 0xFFFF
    scale = sm_scale if sm_scale else 1.0 / np.sqrt(d)
    ref = np.zeros((n_sets, group, d))
    pool_bits = W.to_bits(pool)
    for s, n in enumerate(counts):
        rows_k, rows_v = [], []
        for i in range(n):
            keep = [r for r in range(T) if (int(masks[s, i]) >> r) & 1]
            rows_k.append(pool_bits[ids[s, i], 0, keep])
            rows_v.append(pool_bits[ids[s, i], 1, keep])
        K = O.bf16_to_f32(np.concatenate(rows_k)) if rows_k else np.zeros((0, d), np.float32)
        V = O.bf16_to_f32(np.concatenate(rows_v)) if rows_v else np.zeros((0, d), np.float32)
        ref[s] = O.attention_fp64(O.bf16_to_f32(W.to_bits(q[s])), K, V, scale)
    args = [x.to(dev) for x in (q, pool, torch.from_numpy(ids), torch.from_numpy(masks),
                                torch.from_numpy(np.asarray(counts, dtype=np.int32)))]
    outs = []
    for call in range(2):
        got = torch.full((n_sets, group, d), float("nan"), dtype=torch.bfloat16, device=dev)
        rc = P.spin_paged_attention_static(args[0], args[1], args[2], args[3], args[4], n_sets, stride, group,
                                           sm_scale, got, torch.cuda.current_stream())
        assert rc == 0
        torch.cuda.synchronize()
        outs.append(got.float().cpu().numpy().astype(np.float64))
    return outs, ref


@pytest.mark.parametrize("group", [1, 8])
def test_static_attention_boundary_lists_against_the_fp64_reference(group):
    # a full list (n_pages == list_stride, three chunks of 8, 8 and 3 pages), an empty set, one
    # page, exactly one chunk, one page more than a chunk; query groups of 1 and of 8
    outs, ref = _static_case(group, [19, 0, 1, 8, 9], 19, seed=40 + group, sm_scale=1.0)
    for call, got in enumerate(outs):
        assert np.isfinite(got).all(), call
        err = np.abs(got - ref)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (call, err.max(), err.mean())
        assert np.array_equal(got[1], np.zeros_like(got[1]))         # the empty set: zero output
        rel = np.sqrt((err ** 2).sum() / (ref ** 2).sum())
        assert rel < 2e-2, rel


def test_static_attention_many_chunks_merge_in_tiles():
    # 4800 pages in one set (600 chunks: the merge works through them in tiles), query group 8
    outs, ref = _static_case(8, [4800], 4800, seed=7)
    for got in outs:
        err = np.abs(got - ref)
        assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (err.max(), err.mean())
        assert np.sqrt((err ** 2).sum() / (ref ** 2).sum()) < 2e-2
