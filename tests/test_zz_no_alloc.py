"""spin_paged_attention_static: the allocation-free attention entry point.

Some users of this library run where they may not allocate GPU memory at all (inside another
component's fixed memory budget, or on a path where the allocator must not be touched), so
they cannot build a context.  For them the library carries its split-K scratch as a built-in
array.  This test drives the entry point through the C ABI with page lists taken from a
normal decode step and checks, on two calls in a row (the second reuses the array with the
first call's leftovers in it), that the output matches spin_decode_step's.
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
