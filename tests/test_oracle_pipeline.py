"""Pins for the oracle's attention and for the whole decode step.  CPU only."""
import dataclasses
import math
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import spin_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def dense_attention_loops(q, K, V, scale):
    """Textbook attention, one scalar at a time (independent of the oracle's matmuls)."""
    G, d = len(q), len(q[0])
    out = [[0.0] * d for _ in range(G)]
    for g in range(G):
        logit = [scale * sum(q[g][c] * K[i][c] for c in range(d)) for i in range(len(K))]
        m = max(logit)
        w = [math.exp(x - m) for x in logit]
        z = sum(w)
        for c in range(d):
            out[g][c] = sum(w[i] * V[i][c] for i in range(len(K))) / z
    return np.array(out)


def test_attention_equals_scalar_loops():
    rng = np.random.default_rng(0)
    q, K, V = rng.standard_normal((2, 16)), rng.standard_normal((37, 16)), rng.standard_normal((37, 16))
    got = O.attention_fp64(q, K, V, 0.7)
    ref = dense_attention_loops(q.tolist(), K.tolist(), V.tolist(), 0.7)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)


def test_attention_special_cases():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((4, 128))
    K = rng.standard_normal((9, 128))
    V = rng.standard_normal((9, 128))
    assert np.allclose(O.attention_fp64(q, K[:1], V[:1], 1.0), np.repeat(V[:1], 4, axis=0))
    same = np.repeat(V[:1], 9, axis=0)
    assert np.allclose(O.attention_fp64(q, K, same, 1.0), np.repeat(V[:1], 4, axis=0))
    assert np.array_equal(O.attention_fp64(q, K[:0], V[:0], 1.0), np.zeros((4, 128)))
    # a dominant key takes (almost) all the weight
    K2 = K.copy()
    K2[3] = 50.0 * q[0] / np.linalg.norm(q[0])
    assert np.allclose(O.attention_fp64(q[:1], K2, V, 1.0), V[3:4], atol=1e-6)


def _tiny(kind, **kw):
    base = dict(name="t", seed=11, batch=2, num_layers=2, num_q_heads=4, num_kv_heads=2,
                head_dim=128, page_tokens=16, context=16 * 9 + 5, partition_kind=kind, topk=4,
                slots_per_set=6, lru_buckets=4, steps=12, drift=0.3, kv_recipe="normal")
    base.update(kw)
    return W.Workload(**base)


def _run(w, sm_scale=0.0, topk=None, slots=None, collect=None):
    cfg = O.OracleConfig(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, w.page_tokens,
                         w.partition_kind, w.topk if topk is None else topk, w.lru_buckets, sm_scale)
    orc = O.SpinOracle(cfg)
    reqs, allk, allv = [], {}, {}
    for r in range(w.batch):
        req = orc.request_open(w.slots_per_set if slots is None else slots)
        reqs.append(req)
        for l in range(w.num_layers):
            k, v = W.kv_tokens(w, r, l, 0, w.context)
            allk[(r, l)], allv[(r, l)] = [W.to_bits(k)], [W.to_bits(v)]
            if w.partition_kind == W.PART_CLUSTER_CENTROID:
                tp = W.cluster_assignment(w, r, l, w.context).numpy()
                orc.append_kv(req, l, W.to_bits(k), W.to_bits(v), tp, W.to_bits(W.centroids(w, r, l)))
            else:
                orc.append_kv(req, l, W.to_bits(k), W.to_bits(v))
    qs = {(r, l): W.QueryStream(w, r, l) for r in range(w.batch) for l in range(w.num_layers)}
    outs = []
    for step in range(w.steps):
        for l in range(w.num_layers):
            for r in range(w.batch):
                k, v = W.kv_tokens(w, r, l, w.context + step, 1)
                allk[(r, l)].append(W.to_bits(k)); allv[(r, l)].append(W.to_bits(v))
                orc.append_kv(reqs[r], l, W.to_bits(k), W.to_bits(v))
            q = np.stack([W.to_bits(qs[(r, l)].next()) for r in range(w.batch)])
            out = orc.decode_step(l, reqs, q)
            outs.append((step, l, q, out))
            if collect is not None:
                collect(step, l, orc)
    return orc, reqs, allk, allv, outs


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_TOKEN_DOT, W.PART_CLUSTER_CENTROID])
@pytest.mark.parametrize("sm_scale", [0.0, 1.0])
def test_selecting_everything_equals_dense_attention(kind, sm_scale):
    w = _tiny(kind, steps=3, batch=1, num_layers=1, context=16 * 4 + 7,
              kv_recipe="mixture" if kind == W.PART_CLUSTER_CENTROID else "normal", num_clusters=5)
    orc, reqs, allk, allv, outs = _run(w, sm_scale=sm_scale, topk=10 ** 6, slots=4)
    scale = sm_scale if sm_scale else 1.0 / math.sqrt(128)
    G = w.group
    for step, l, q, out in outs:
        n = w.context + step + 1
        K = O.bf16_to_f32(np.concatenate(allk[(0, l)])[:n]).astype(np.float64)
        V = O.bf16_to_f32(np.concatenate(allv[(0, l)])[:n]).astype(np.float64)
        qf = O.bf16_to_f32(q[0]).astype(np.float64)
        for h in range(w.num_kv_heads):
            ref = dense_attention_loops(qf[h * G:(h + 1) * G].tolist(), K[:, h].tolist(),
                                        V[:, h].tolist(), scale)
            assert np.allclose(out[0, h * G:(h + 1) * G], ref, rtol=1e-9, atol=1e-11)


def test_page_mode_structure_and_tail():
    w = _tiny(W.PART_PAGE_MINMAX)
    seen = []

    def collect(step, l, orc):
        for (r, ll, h), tr in orc.last_trace.items():
            if ll != l:
                continue
            st = orc.set(r, l, h)
            n = w.context + step + 1
            assert st.n_tokens == n
            # newest page (full or not) is the tail and never a candidate
            assert st.n_partitions() == (n - 1) // 16
            tail = [p for p in tr.pages if p[3] == -2]
            assert len(tail) == 1 and tail[0][2] == (1 << ((n - 1) % 16 + 1)) - 1
            assert len(tr.selected) == min(w.topk, st.n_partitions())
            assert list(tr.selected) == sorted(set(tr.selected)) and tr.selected.max() < st.n_partitions()
            # identity mapping partition <-> page, all 16 tokens valid
            for (p, i, mask, slot) in tr.pages[:-1]:
                assert i == 0 and mask == 0xFFFF
                assert st.part_offset[p] == p and st.cpu_page_table[p] == p
            seen.append(len(tr.bypass))
    _run(w, collect=collect)
    assert seen


def test_token_mode_masks_and_pages():
    w = _tiny(W.PART_TOKEN_DOT, topk=20, slots_per_set=8)

    def collect(step, l, orc):
        for (r, ll, h), tr in orc.last_trace.items():
            if ll != l:
                continue
            toks = [int(x) for x in tr.selected]
            assert len(toks) == 20 and toks == sorted(set(toks))
            assert list(tr.partitions) == sorted({t // 16 for t in toks})
            got = {(p, r_) for (p, i, mask, slot) in tr.pages if slot != -2
                   for r_ in range(16) if (mask >> r_) & 1}
            assert got == {(t // 16, t % 16) for t in toks}
    _run(w, collect=collect)


def test_cluster_mode_packing_invariants():
    w = _tiny(W.PART_CLUSTER_CENTROID, kv_recipe="mixture", num_clusters=7, topk=3,
              slots_per_set=9, context=16 * 12 + 3, steps=20)
    orc, reqs, allk, allv, outs = _run(w)
    for r in range(w.batch):
        for l in range(w.num_layers):
            tp = W.cluster_assignment(w, r, l, w.context).numpy()
            kb = allk[(r, l)][0]
            for h in range(w.num_kv_heads):
                st = orc.set(reqs[r], l, h)
                assert sum(st.part_tokens) == w.context                     # every token once
                n_cluster_pages = sum(-(-m // 16) for m in st.part_tokens)
                assert st.part_offset == list(np.cumsum([0] + [-(-m // 16) for m in st.part_tokens[:-1]]))
                assert len(st.tail_pages) == -(-w.steps // 16) and st.n_pages == n_cluster_pages + len(st.tail_pages)
                for c in range(w.num_clusters):                              # order kept inside a cluster
                    idx = np.nonzero(tp[:, h] == c)[0]
                    assert st.part_tokens[c] == len(idx)
                    for j, tok in enumerate(idx):
                        page = st.cpu_page_table[st.part_offset[c] + j // 16]
                        assert np.array_equal(st.page_k[page, j % 16], kb[tok, h])
                tr = orc.last_trace[(reqs[r], l, h)]
                assert [p for p in tr.pages if p[3] == -2][-1][2] == (1 << ((w.steps - 1) % 16 + 1)) - 1


def test_counters_and_eq2_bytes():
    w = _tiny(W.PART_PAGE_MINMAX)
    orc, *_ = _run(w)
    c = orc.counters
    sets = w.batch * w.num_layers * w.num_kv_heads
    assert c["steps"] == sets * w.steps
    assert c["selected_pages"] == c["hit_pages"] + c["miss_pages"]
    # Eq. 2: KV_topk = 2 * d * e * (selected tokens) per set and step
    assert orc.step_bytes()["kv_read"] == (c["selected_pages"] + c["tail_pages"]) * 2 * 128 * 2 * 16


def _c1_trace_lines():
    w = W.CONFIGS["c1"]
    lines = []

    def collect(step, l, orc):
        tr = orc.last_trace[(0, 0, 0)]
        ev = ",".join(f"{s}:{p}" for s, p, _ in tr.evicted)
        lines.append(f"{step} sel={','.join(map(str, tr.selected))} miss={','.join(map(str, tr.misses))} "
                     f"evict={ev}")
    orc, reqs, _, _, outs = _run(w, collect=collect)
    return lines, outs


def test_c1_regression_against_stored_oracle_trace():
    # Stored by tests/golden/make_c1_golden.py (oracle only).  Guards the oracle against
    # silent drift; it is not an independent pin.
    lines, outs = _c1_trace_lines()
    stored = [x.rstrip("\n") for x in open(os.path.join(GOLD, "c1_oracle_trace.txt")) if not x.startswith("#")]
    assert lines == stored


# ---- Index during decode (cluster granularity): full tail pages fold into the clusters -------

def _bits(x):
    """fp32 -> bf16 bit patterns (round to nearest even)."""
    return (O.f32_to_bf16_f32(np.asarray(x, dtype=np.float32)).view(np.uint32) >> 16).astype(np.uint16)


def _clustered_set(rng, n_tokens, C, d=128, slots=12, topk=4):
    cfg = O.OracleConfig(1, 2, 1, d, 16, O.PART_CLUSTER_CENTROID, topk, 4)
    st = O.OracleSet(cfg, slots)
    cen = rng.standard_normal((C, d)).astype(np.float32) * 2.0
    assign = rng.integers(0, C, size=n_tokens)
    k = cen[assign] + 0.2 * rng.standard_normal((n_tokens, d)).astype(np.float32)
    v = rng.standard_normal((n_tokens, d)).astype(np.float32)
    st.append_clustered(_bits(k), _bits(v), assign, _bits(cen))
    return cfg, st, cen


def _all_rows(st):
    rows = []
    for c in range(st.n_partitions()):
        for i in range(st.partition_pages(c)):
            page = st.cpu_page_table[st.part_offset[c] + i]
            valid = min(st.T, st.part_tokens[c] - i * st.T)
            rows += [(st.page_k[page, r].tobytes(), st.page_v[page, r].tobytes()) for r in range(valid)]
    for j, page in enumerate(st.tail_pages):
        valid = st.tail_len if j == len(st.tail_pages) - 1 else st.T
        rows += [(st.page_k[page, r].tobytes(), st.page_v[page, r].tobytes()) for r in range(valid)]
    return rows


def test_reindex_moves_every_tail_token_to_its_best_centroid_and_keeps_all_rows():
    rng = np.random.default_rng(21)
    C = 9
    cfg, st, cen = _clustered_set(rng, 150, C)
    cen_bf = O.bf16_to_f32(_bits(cen)).astype(np.float64)
    new_assign = rng.integers(0, C, size=40)
    nk = cen[new_assign] + 0.2 * rng.standard_normal((40, 128)).astype(np.float32)
    nv = rng.standard_normal((40, 128)).astype(np.float32)
    kb, vb = _bits(nk), _bits(nv)
    st.append_tokens(kb, vb)                       # 2 full tail pages + 8 tokens
    before = sorted(_all_rows(st))
    counts = list(st.part_tokens)
    taken = st.reindex()
    assert sorted(_all_rows(st)) == before                     # nothing lost, nothing doubled
    assert len(taken) == 32 and len(st.tail_pages) == 1 and st.tail_len == 8
    # well separated centroids: the winner is the plain float64 argmax, which is the generating cluster
    best = np.argmax(O.bf16_to_f32(kb[:32]).astype(np.float64) @ cen_bf.T, axis=1)
    assert [c for _, c in taken] == [int(x) for x in best] == [int(x) for x in new_assign[:32]]
    # arrival order at the end of each cluster
    for t, c in taken:
        pos = counts[c]
        page = st.cpu_page_table[st.part_offset[c] + pos // 16]
        assert st.page_k[page, pos % 16].tobytes() == kb[t].tobytes()
        counts[c] += 1
    assert counts == st.part_tokens
    assert st.reindex() == []                                  # nothing full is left in the tail


def test_reindex_leaves_dense_attention_unchanged_and_drops_stale_residency():
    rng = np.random.default_rng(22)
    C = 6
    cfg, st, cen = _clustered_set(rng, 90, C, slots=40, topk=C)    # top-k = every cluster: dense attention
    q = _bits(rng.standard_normal((2, 128)).astype(np.float32))
    st.append_tokens(_bits(rng.standard_normal((33, 128)).astype(np.float32)),
                     _bits(rng.standard_normal((33, 128)).astype(np.float32)))
    out0, tr0 = st.decode(q)
    assert all(st.part_resident[c] for c in range(C) if st.part_tokens[c])
    taken = st.reindex()
    touched = {c for _, c in taken}
    assert touched and all(st.part_resident[c] == 0 for c in touched)
    assert not (set(int(p) for p in st.slot_part if p >= 0) & touched)
    out1, tr1 = st.decode(q)
    np.testing.assert_allclose(out1, out0, rtol=0, atol=1e-12)  # same tokens attended, other order
    assert set(tr1.misses) == touched                            # exactly the stale clusters are fetched again


def test_reindex_with_a_full_newest_page_empties_the_tail_and_equal_scores_go_to_the_lower_cluster():
    rng = np.random.default_rng(23)
    cfg = O.OracleConfig(1, 1, 1, 128, 16, O.PART_CLUSTER_CENTROID, 2, 4)
    st = O.OracleSet(cfg, 8)
    cen = rng.standard_normal((3, 128)).astype(np.float32)
    cen[2] = cen[1]                                              # clusters 1 and 2 share a centroid
    k = rng.standard_normal((20, 128)).astype(np.float32)
    st.append_clustered(_bits(k), _bits(k), rng.integers(0, 3, size=20), _bits(cen))
    nk = np.repeat(cen[1:2] * 3.0, 16, axis=0)
    st.append_tokens(_bits(nk), _bits(nk))   # exactly one full page
    taken = st.reindex()
    assert [c for _, c in taken] == [1] * 16 and st.tail_pages == [] and st.tail_len == 0
    st.append_tokens(_bits(nk[:3]), _bits(nk[:3]))
    assert len(st.tail_pages) == 1 and st.tail_len == 3


# ---- Index of a full tail page: the summaries the set builds from its own pages -------------
# (Table 1, Index column; Section 4.1 "Index").  The checks below rebuild every summary from the
# keys that were handed to append_tokens, never from the set's page store, so a summary taken
# from the wrong page, the wrong rows or the wrong channel order fails them.

def _distinct_keys(rng, n_tokens, d=128):
    """bf16-exact keys, every token's row recognisable: small integers plus a per-token offset."""
    base = rng.integers(-40, 41, size=(n_tokens, d)).astype(np.float32)
    base += (np.arange(n_tokens, dtype=np.float32) % 7)[:, None]
    return base                                                  # |x| <= 46: exact in bf16


def _set_through_append(kind, keys, chunks, topk=3, slots=4, G=2):
    cfg = O.OracleConfig(1, G, 1, 128, 16, kind, topk, 4)
    st = O.OracleSet(cfg, slots)
    kb = _bits(keys)
    vb = _bits(np.zeros_like(keys))
    i = 0
    for m in chunks:                                             # ragged appends: prefill, then decode tokens
        st.append_tokens(kb[i:i + m], vb[i:i + m])
        i += m
    assert i == keys.shape[0]
    return st


def test_minmax_summaries_are_the_per_channel_extremes_of_their_own_page():
    rng = np.random.default_rng(21)
    n = 16 * 6 + 9
    keys = _distinct_keys(rng, n)
    st = _set_through_append(O.PART_PAGE_MINMAX, keys, [16 * 2 + 3, 1, 1, 12, 16 * 3 + 1, 1, 1, 1, 1, 1, 2])
    P = st.n_partitions()
    assert P == 6 and st.tail_len == 9                           # the newest page is the tail, never a candidate
    for p in range(P):
        page = keys[16 * p:16 * p + 16]
        assert np.array_equal(st.sum_min[p], page.min(axis=0)), p
        assert np.array_equal(st.sum_max[p], page.max(axis=0)), p
        assert st.part_tokens[p] == 16 and st.part_offset[p] == p


def test_minmax_bound_holds_for_every_key_of_the_page_through_the_whole_step():
    rng = np.random.default_rng(22)
    G, n = 4, 16 * 8 + 5
    keys = O.f32_to_bf16_f32(rng.standard_normal((n, 128)).astype(np.float32) * 3.0)
    st = _set_through_append(O.PART_PAGE_MINMAX, keys, [n - 20] + [1] * 20, G=G)
    for step in range(3):
        q = O.f32_to_bf16_f32(rng.standard_normal((G, 128)).astype(np.float32))
        _, tr = st.decode(_bits(q), want_output=False)
        P = len(tr.scores)
        assert P == 8
        exact = (q.astype(np.float64) @ keys.astype(np.float64).T).sum(axis=0)      # sum_g q_g . k, per token
        for p in range(P):
            # the page's score bounds the summed dot product of each of ITS OWN keys ...
            assert exact[16 * p:16 * p + 16].max() <= float(tr.scores[p]) * (1 + 1e-5) + 1e-4, (step, p)


def test_minmax_score_is_attained_by_a_page_of_identical_keys():
    # one page of 16 copies of the same row: min = max = that row, so the bound is the dot product
    rng = np.random.default_rng(23)
    G = 2
    row = O.f32_to_bf16_f32(rng.standard_normal(128).astype(np.float32))
    other = O.f32_to_bf16_f32(rng.standard_normal((16, 128)).astype(np.float32))
    keys = np.concatenate([np.repeat(row[None], 16, axis=0), other, other[:3]])
    st = _set_through_append(O.PART_PAGE_MINMAX, keys, [keys.shape[0]], G=G)
    q = O.f32_to_bf16_f32(rng.standard_normal((G, 128)).astype(np.float32))
    _, tr = st.decode(_bits(q), want_output=False)
    want = float((q.astype(np.float64) @ row.astype(np.float64)).sum())
    assert abs(float(tr.scores[0]) - want) <= 1e-5 * max(1.0, abs(want))
    assert float(tr.scores[1]) >= float((q.astype(np.float64) @ other.astype(np.float64).T).sum(axis=0).max()) - 1e-4


def test_token_summaries_are_the_tokens_own_key_rows_and_scores_their_dot_products():
    rng = np.random.default_rng(24)
    G, n = 2, 16 * 5 + 2
    keys = _distinct_keys(rng, n)
    st = _set_through_append(O.PART_TOKEN_DOT, keys, [16 * 3 + 15, 1, 1, 16, 1], topk=9, G=G)
    P = st.n_partitions()
    assert P == 5
    assert np.array_equal(st.sum_vec[:P * 16], keys[:P * 16])    # row i of the summaries is token i's key
    q = O.f32_to_bf16_f32(rng.standard_normal((G, 128)).astype(np.float32))
    _, tr = st.decode(_bits(q), want_output=False)
    want = (q.astype(np.float64) @ keys[:P * 16].astype(np.float64).T).sum(axis=0)
    assert len(tr.scores) == P * 16
    assert np.allclose(tr.scores.astype(np.float64), want, rtol=1e-5, atol=1e-3)
    # and the selection is the brute-force top-9 of those dot products (distinct by construction)
    order = sorted(range(P * 16), key=lambda i: (-float(tr.scores[i]), i))[:9]
    assert list(tr.selected) == sorted(order)
