"""CPU oracle for the sparse decode step over a hierarchical paged KV cache.

THIS IS TEST INFRASTRUCTURE, not a product path.  It is a plain, slow, obviously correct
restatement of what one decode step computes, written from the paper's description; the
CUDA library shares no code with it and never calls it.  Only tests, the smoke check and
the benchmark's CPU-baseline leg may import it.

What follows which passage of the paper ("Spin", arXiv 2604.26837):

* data model (partitions over fixed-size head-wise pages, four mapping tables)
                                   -- Section 5.2 "Partition Abstraction"
* Select = score against per-partition summaries, then top-k
                                   -- Table 1 (Select column), Section 4.1 "Select"
* Retrieve lookup path, steps 1-4  -- Section 5.2, last paragraph
* bucketed LRU, steps 1-4          -- Section 5.3 "Bucketed LRU Replacement"
* Attention over the selected KV   -- Section 4.1 "Attention" (standard softmax attention)
* byte model of a step             -- Section 3.1, Eq. 1-3

Where the paper is silent the reading taken here is stated next to the code; every such
reading is also listed in the design notes of the repository.

Precision: summaries and scores are fp32 with ONE fixed summation tree (so that selections
can be compared bit for bit); attention is fp64.

Pins (tests marked "not gpu"): dense attention by an independent triple loop when top-k
covers everything; a brute-force last-use LRU simulator; the closed form of a page's
timestamp; a hand-derived worked example of the four LRU steps; page size 1 making the
min/max bound equal the dot product bit for bit; the bound invariant q.k <= score(page);
brute-force stable sort for top-k with ties; the summaries a set builds at page fill rebuilt
from the appended keys (per-channel extremes of the page's own 16 keys, a token's own key
row) and the scores of a whole step checked against fp64 dot products of those keys; the
order in which a group's heads are added, on values where the order changes the fp32 sum.  Nothing in the paper prints a worked numeric
example, so absolute hit ratios and outputs are "parity unpinned" beyond those pins.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

PART_PAGE_MINMAX = 0
PART_TOKEN_DOT = 1
PART_CLUSTER_CENTROID = 2
PART_PAGE_MEAN = 3

F32 = np.float32


def f32_to_bf16_f32(x: np.ndarray) -> np.ndarray:
    """Round fp32 to the nearest bf16 (ties to even) and widen back to fp32 (finite inputs)."""
    b = np.asarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> 16) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to fp32."""
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


# --------------------------------------------------------------------------------------
# Select: scoring (Table 1: score(roped_q, k_sums); Section 4.1 "Select")
# --------------------------------------------------------------------------------------

def canonical_sum(terms: np.ndarray) -> np.ndarray:
    """Sum fp32 terms over the last axis in the one summation order both sides use.

    The paper does not fix an order.  Reading: the channels are cut into blocks of 8
    consecutive channels; each block is summed left to right; the block sums are then
    combined by a balanced tree over adjacent pairs ((b0+b1), (b2+b3), ... then pairs of
    those).  Every addition is a single fp32 rounding.
    """
    terms = np.asarray(terms, dtype=F32)
    d = terms.shape[-1]
    nb = d // 8
    assert d % 8 == 0 and nb & (nb - 1) == 0, "head_dim must be 8 * 2^j"
    t = terms.reshape(terms.shape[:-1] + (nb, 8))
    s = t[..., 0]
    for i in range(1, 8):
        s = (s + t[..., i]).astype(F32)
    while s.shape[-1] > 1:
        s = (s[..., 0::2] + s[..., 1::2]).astype(F32)
    return s[..., 0]


def _group_total(per_head: np.ndarray) -> np.ndarray:
    """Set score from the per-query-head scores [G][P]: ((s0 + s1) + s2) + ...

    The paper does not say how a kv head's group of query heads is aggregated.  Reading:
    the sum, in ascending head order.  A final "+ 0.0" turns -0.0 into +0.0 so that equal
    scores have equal bits.
    """
    tot = per_head[0].astype(F32)
    for g in range(1, per_head.shape[0]):
        tot = (tot + per_head[g]).astype(F32)
    return (tot + F32(0.0)).astype(F32)


def score_minmax(q: np.ndarray, smin: np.ndarray, smax: np.ndarray) -> np.ndarray:
    """Upper-bound score of each page: sum_c max(q_c*min_c, q_c*max_c), per head, summed.

    q: fp32 [G][d]; smin/smax: fp32 [P][d] (values that are exact bf16) -> fp32 [P].
    A product of two bf16 values is exact in fp32, so only the additions round.
    """
    per_head = np.empty((q.shape[0], smin.shape[0]), dtype=F32)
    for g in range(q.shape[0]):
        terms = np.maximum(q[g][None, :] * smin, q[g][None, :] * smax).astype(F32)
        per_head[g] = canonical_sum(terms)
    return _group_total(per_head)


def score_dot(q: np.ndarray, summ: np.ndarray) -> np.ndarray:
    """Score of each token / cluster: q . summary (key row or centroid), per head, summed."""
    per_head = np.empty((q.shape[0], summ.shape[0]), dtype=F32)
    for g in range(q.shape[0]):
        per_head[g] = canonical_sum((q[g][None, :] * summ).astype(F32))
    return _group_total(per_head)


# --------------------------------------------------------------------------------------
# Select: top-k (Table 1: "-> topk")
# --------------------------------------------------------------------------------------

def topk_select(scores: np.ndarray, k: int) -> np.ndarray:
    """The min(k, n) best candidates: higher score first, equal scores -> lower index.

    Returns the chosen indices in ascending order (int64).
    """
    n = scores.shape[0]
    kk = min(int(k), n)
    if kk <= 0:
        return np.zeros(0, dtype=np.int64)
    order = np.argsort(-scores.astype(F32), kind="stable")
    return np.sort(order[:kk]).astype(np.int64)


# --------------------------------------------------------------------------------------
# Bucketed LRU (Section 5.3, steps 1-4)
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class LruResult:
    hits: List[int]                       # selected partitions that were resident
    misses: List[int]                     # selected partitions that were not (incl. bypassed)
    bypass: List[int]                     # missed partitions that could not be cached
    evicted: List[Tuple[int, int, int]]   # (slot, partition, page_idx) in slot order
    admitted: List[Tuple[int, int, int]]  # (slot, partition, page_idx) in admission order
    demand: int
    threshold: int                        # x of step 3 (-2 when no eviction scan ran)


def bucketed_lru_step(slot_part: np.ndarray, slot_pidx: np.ndarray, slot_ts: np.ndarray,
                      resident: np.ndarray, n_pages_of: np.ndarray,
                      selected: Sequence[int], t: int, n: int, exact: bool = False) -> LruResult:
    """One replacement round of one set; mutates the slot arrays and `resident` in place.

    slot_part/slot_pidx/slot_ts: int arrays [S]; an empty slot has partition -1 and
    timestamp -1.  resident: per partition 0/1.  n_pages_of: per partition page count.
    selected: partition ids in ascending order.  t: this request's decode-step counter
    (0 for its first step).  n: number of timestamp values (buckets).

    Step 1  classify the selected partitions by the residency flag; demand = pages of misses.
    Step 2  top = min(t, n-1); pages of hit partitions <- top; once t > n-1 every other
            occupied page <- ts-1.  Reading: floored at 0, the stated range being [0, n-1].
    Step 3  if demand > 0: histogram of the updated timestamps (empty slots in bucket -1),
            smallest x whose cumulative count reaches the demand, every occupied page with
            ts <= x is evicted (so more than `demand` pages may go) and its partition
            becomes non-resident.  Reading: pages hit in this step are left out of the
            histogram and are never victims; for n >= 2 they sit alone in bucket `top`,
            so this equals the paper's rule whenever the other slots can meet the demand.
            If even x = n-1 does not meet the demand, x = n-1 (everything else goes).
            Variant `exact` (not the paper's rule; it measures what the over-eviction costs):
            pages with ts < x go as before, but of bucket x only the first
            `demand - #(pool pages with ts < x)` pages in ascending slot order are taken;
            a partition that loses a page this way goes whole (cached whole or not at all).
    Step 4  admission.  Reading (the paper does not say which freed page goes to which
            miss): free slots in ascending slot order, missed pages in ascending
            (partition, page_idx) order, i-th page to i-th free slot, timestamp `top`.
            Reading for an over-full set (the paper's scheduler rules this out): a
            partition is cached whole or not at all; one whose pages no longer fit is
            "bypassed" -- attended from host memory, left non-resident -- and later,
            smaller partitions may still be admitted.
    """
    S = slot_part.shape[0]
    sel = [int(p) for p in selected]
    hits = [p for p in sel if resident[p]]
    misses = [p for p in sel if not resident[p]]
    demand = int(sum(int(n_pages_of[p]) for p in misses))

    top = min(int(t), n - 1)
    occupied = slot_part >= 0
    hit_slot = occupied & np.isin(slot_part, np.asarray(hits, dtype=slot_part.dtype))
    slot_ts[hit_slot] = top
    if t > n - 1:
        other = occupied & ~hit_slot
        slot_ts[other] = np.maximum(0, slot_ts[other] - 1)

    evicted: List[Tuple[int, int, int]] = []
    threshold = -2
    if demand > 0:
        pool = ~hit_slot                       # empties (ts -1) and non-hit pages
        threshold = n - 1
        for x in range(-1, n):
            if int(np.count_nonzero(pool & (slot_ts <= x))) >= demand:
                threshold = x
                break
        victim = occupied & pool & (slot_ts <= threshold)
        if exact and threshold >= 0:
            need = demand - int(np.count_nonzero(pool & (slot_ts < threshold)))
            bucket = np.nonzero(occupied & pool & (slot_ts == threshold))[0]      # ascending slots
            taken = np.unique(slot_part[bucket[:max(need, 0)]])
            victim = occupied & pool & ((slot_ts < threshold) | np.isin(slot_part, taken))
        for s in np.nonzero(victim)[0]:
            evicted.append((int(s), int(slot_part[s]), int(slot_pidx[s])))
            resident[slot_part[s]] = 0
            slot_part[s] = -1
            slot_pidx[s] = 0
            slot_ts[s] = -1

    free = [int(s) for s in np.nonzero(slot_part < 0)[0]]
    used = 0
    admitted: List[Tuple[int, int, int]] = []
    bypass: List[int] = []
    for p in misses:
        npg = int(n_pages_of[p])
        if npg <= len(free) - used:
            for i in range(npg):
                s = free[used + i]
                slot_part[s] = p
                slot_pidx[s] = i
                slot_ts[s] = top
                admitted.append((s, p, i))
            used += npg
            resident[p] = 1
        else:
            bypass.append(p)
    assert S == slot_part.shape[0]
    return LruResult(hits, misses, bypass, evicted, admitted, demand, threshold)


# --------------------------------------------------------------------------------------
# Attention (Section 4.1 "Attention": standard softmax attention over the selected tokens)
# --------------------------------------------------------------------------------------

def attention_fp64(q: np.ndarray, K: np.ndarray, V: np.ndarray, sm_scale: float) -> np.ndarray:
    """softmax(sm_scale * q K^T) V for every query head; everything in fp64.

    q: [G][d], K/V: [n_tok][d] -> [G][d].  With no tokens the output is zero.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    if K.shape[0] == 0:
        return np.zeros_like(q)
    logits = sm_scale * (q @ K.T)                       # [G][n_tok]
    logits -= logits.max(axis=1, keepdims=True)
    w = np.exp(logits)
    return (w @ V) / w.sum(axis=1, keepdims=True)


# --------------------------------------------------------------------------------------
# The set: one (request, layer, kv head)
# --------------------------------------------------------------------------------------

@dataclasses.dataclass
class StepTrace:
    """Everything of one set's decode step that is compared bit for bit."""
    selected: np.ndarray        # chosen candidate ids, ascending (tokens in token mode)
    partitions: np.ndarray      # partitions handed to the cache manager, ascending
    hits: List[int]
    misses: List[int]
    bypass: List[int]
    evicted: List[Tuple[int, int, int]]
    # page list in attention order: (partition, page_idx, token mask, slot); slot is the
    # set-local GPU page table index, -1 for a bypassed page, -2 for a local tail page
    pages: List[Tuple[int, int, int, int]]
    slot_part: np.ndarray
    slot_pidx: np.ndarray
    slot_ts: np.ndarray
    resident: np.ndarray
    scores: np.ndarray


@dataclasses.dataclass
class OracleConfig:
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int = 128
    page_tokens: int = 16
    partition_kind: int = PART_PAGE_MINMAX
    topk: int = 16
    lru_buckets: int = 64
    sm_scale: float = 0.0          # 0 -> 1/sqrt(head_dim) (the paper gives no scale)
    evict_exact: bool = False      # evict only what the demand needs (variant, see bucketed_lru_step)


class OracleSet:
    """State of one (request, layer, kv head): host pages, tables, summaries, GPU slots."""

    def __init__(self, cfg: OracleConfig, slots: int):
        self.cfg = cfg
        self.T, self.d = cfg.page_tokens, cfg.head_dim
        self.kind = cfg.partition_kind
        # host tier: every page of the set, complete (eviction needs no write-back)
        self.cap = 64
        self.page_k = np.zeros((self.cap, self.T, self.d), dtype=np.uint16)
        self.page_v = np.zeros((self.cap, self.T, self.d), dtype=np.uint16)
        self.n_pages = 0
        self.n_tokens = 0
        # Meta-partition table: token count + residency; Partition Offset table; CPU page
        # table (flat list of the set's host pages; here the logical page number itself)
        self.part_tokens: List[int] = []
        self.part_resident: List[int] = []
        self.part_offset: List[int] = []
        self.cpu_page_table: List[int] = []
        # summaries kept on the GPU tier
        self.sum_min = np.zeros((0, self.d), dtype=F32)
        self.sum_max = np.zeros((0, self.d), dtype=F32)
        self.sum_vec = np.zeros((0, self.d), dtype=F32)     # token keys or centroids
        self._sum_rows = 0
        # local tail: pages that are always attended and never candidates
        self.tail_pages: List[int] = []
        self.tail_len = 0                                   # tokens in the last tail page
        # GPU page table: S slots of (partition, page_idx, timestamp)
        self.slot_part = np.full(slots, -1, dtype=np.int64)
        self.slot_pidx = np.zeros(slots, dtype=np.int64)
        self.slot_ts = np.full(slots, -1, dtype=np.int64)
        self.t = 0
        self.clustered = False

    # ---- host pages ------------------------------------------------------------------
    def _new_page(self) -> int:
        if self.n_pages == self.cap:
            self.cap *= 2
            for name in ("page_k", "page_v"):
                old = getattr(self, name)
                new = np.zeros((self.cap, self.T, self.d), dtype=np.uint16)
                new[: old.shape[0]] = old
                setattr(self, name, new)
        self.n_pages += 1
        self.cpu_page_table.append(self.n_pages - 1)
        return self.n_pages - 1

    def _grow_rows(self, name: str, rows: int):
        arr = getattr(self, name)
        if rows > arr.shape[0]:
            new = np.zeros((max(rows, 2 * arr.shape[0], 256), self.d), dtype=F32)
            new[: arr.shape[0]] = arr
            setattr(self, name, new)

    # ---- Index + Offload -------------------------------------------------------------
    def _index_tail_page(self):
        """The full tail page becomes partition #P (page and token granularity).

        Reading (the paper has Index run again from time to time during decode and gives no
        period): a page becomes a candidate when the first token of the next page arrives, so
        the newest page -- full or not -- is always the local tail.
        """
        page = self.tail_pages.pop()
        assert self.tail_len == self.T and not self.tail_pages
        p = len(self.part_tokens)
        self.part_tokens.append(self.T)
        self.part_resident.append(0)
        self.part_offset.append(page)
        keys = bf16_to_f32(self.page_k[page])                     # [T][d]
        if self.kind == PART_PAGE_MINMAX:
            self._grow_rows("sum_min", p + 1)
            self._grow_rows("sum_max", p + 1)
            self.sum_min[p] = keys.min(axis=0)
            self.sum_max[p] = keys.max(axis=0)
        elif self.kind == PART_PAGE_MEAN:
            # landmark = mean of the page's keys (Table 1, ShadowKV's Index).  Reading (the paper
            # gives no precision): keys added in token order in fp32, times 1/T, rounded to bf16
            self._grow_rows("sum_vec", p + 1)
            acc = keys[0].astype(F32)
            for r in range(1, self.T):
                acc = (acc + keys[r]).astype(F32)
            self.sum_vec[p] = f32_to_bf16_f32((acc * F32(1.0 / self.T)).astype(F32))
        else:                                                     # token granularity
            self._grow_rows("sum_vec", (p + 1) * self.T)
            self.sum_vec[p * self.T:(p + 1) * self.T] = keys
        self.tail_len = 0

    def append_tokens(self, k_bits: np.ndarray, v_bits: np.ndarray):
        """Append tokens in order (page / token granularity, or decode tokens of a
        clustered set, which only ever extend the always-attended tail)."""
        n, i = int(k_bits.shape[0]), 0
        while i < n:
            if not self.tail_pages or self.tail_len == self.T:
                if self.tail_pages and not self.clustered:
                    self._index_tail_page()
                self.tail_pages.append(self._new_page())
                self.tail_len = 0
            page = self.tail_pages[-1]
            m = min(self.T - self.tail_len, n - i)          # rows that still fit this page
            self.page_k[page, self.tail_len:self.tail_len + m] = k_bits[i:i + m]
            self.page_v[page, self.tail_len:self.tail_len + m] = v_bits[i:i + m]
            self.tail_len += m
            self.n_tokens += m
            i += m

    def append_clustered(self, k_bits: np.ndarray, v_bits: np.ndarray,
                         token_cluster: np.ndarray, centroids_bits: np.ndarray):
        """Prefill of a cluster-granular set: cluster c is partition c; its tokens are
        packed in their original order into ceil(m/T) pages, the last one partial."""
        assert self.n_tokens == 0 and self.kind == PART_CLUSTER_CENTROID
        self.clustered = True
        C = centroids_bits.shape[0]
        self.sum_vec = bf16_to_f32(centroids_bits).copy()
        for c in range(C):
            idx = np.nonzero(token_cluster == c)[0]
            m = idx.shape[0]
            self.part_tokens.append(int(m))
            self.part_resident.append(0)
            self.part_offset.append(len(self.cpu_page_table))
            for j in range(0, m, self.T):
                page = self._new_page()
                rows = idx[j:j + self.T]
                self.page_k[page, : rows.shape[0]] = k_bits[rows]
                self.page_v[page, : rows.shape[0]] = v_bits[rows]
        self.n_tokens = int(k_bits.shape[0])

    # ---- Index during decode, cluster granularity (Section 4.1 "Index") ----------------------
    def reindex(self) -> List[Tuple[int, int]]:
        """Fold the full pages of the local tail into the clusters.

        The paper says that Index also runs during decode to take in new tokens and leaves the
        rest to the algorithm.  Reading: every token of a FULL tail page, in arrival order,
        joins the cluster whose centroid scores highest against its key (the same fp32
        summation tree as Select, ties to the lower cluster); centroids stay as they are; the
        token goes to the end of that cluster (a new page when the last one is full).  A
        cluster that takes a token is no longer GPU-resident (its cached copy is stale): its
        slots are cleared, timestamps of the others untouched.  The partly filled newest
        page stays the tail.  Returns (token index in the folded run, cluster) pairs.
        """
        assert self.clustered
        T = self.T
        n_full = len(self.tail_pages) - (0 if (self.tail_pages and self.tail_len == T) else 1)
        if n_full <= 0:
            return []
        P = self.n_partitions()
        lists = [[self.cpu_page_table[self.part_offset[c] + i] for i in range(self.partition_pages(c))]
                 for c in range(P)]
        taken: List[Tuple[int, int]] = []
        touched = set()
        folded, self.tail_pages = self.tail_pages[:n_full], self.tail_pages[n_full:]
        for j, page in enumerate(folded):
            for r in range(T):
                key = bf16_to_f32(self.page_k[page, r])[None, :]              # one "query head"
                c = int(np.argmax(score_dot(key, self.sum_vec[:P])))          # first maximum
                m = self.part_tokens[c]
                if m % T == 0:
                    lists[c].append(self._new_page())
                dst = lists[c][m // T]
                self.page_k[dst, m % T] = self.page_k[page, r]
                self.page_v[dst, m % T] = self.page_v[page, r]
                self.part_tokens[c] = m + 1
                touched.add(c)
                taken.append((j * T + r, c))
        if not self.tail_pages:
            self.tail_len = 0
        # the CPU page table is laid out afresh: clusters in order, each one's pages together
        self.cpu_page_table, self.part_offset = [], []
        for c in range(P):
            self.part_offset.append(len(self.cpu_page_table))
            self.cpu_page_table.extend(lists[c])
        self.cpu_page_table.extend(self.tail_pages)
        for c in touched:
            self.part_resident[c] = 0
        gone = np.isin(self.slot_part, np.asarray(sorted(touched), dtype=self.slot_part.dtype))
        self.slot_part[gone], self.slot_pidx[gone], self.slot_ts[gone] = -1, 0, -1
        return taken

    # ---- buffer elasticity (Section 5.3, "Buffer Elasticity") ------------------------------
    def resize(self, new_slots: int) -> List[Tuple[int, int, int]]:
        """Change the set's number of GPU page table slots between steps.

        Shrinking reclaims from the TAIL of the table (Section 5.3: the tail is what is given
        back, so that the table stays compact): slots new_slots.. disappear.  Reading (the
        paper does not say what happens to a partition that straddles the cut): a partition
        with any page in the reclaimed tail becomes non-resident as a whole, so its pages below
        the cut are cleared too.  Growing appends empty slots.  Timestamps of surviving pages
        are untouched.  Returns the dropped pages as (slot, partition, page_idx) in slot order.
        """
        S = self.slot_part.shape[0]
        dropped: List[Tuple[int, int, int]] = []
        if new_slots < S:
            gone = {int(p) for p in self.slot_part[new_slots:] if p >= 0}
            for s in range(S):
                p = int(self.slot_part[s])
                if p >= 0 and (s >= new_slots or p in gone):
                    dropped.append((s, p, int(self.slot_pidx[s])))
                    self.part_resident[p] = 0
                    self.slot_part[s], self.slot_pidx[s], self.slot_ts[s] = -1, 0, -1
            self.slot_part = self.slot_part[:new_slots].copy()
            self.slot_pidx = self.slot_pidx[:new_slots].copy()
            self.slot_ts = self.slot_ts[:new_slots].copy()
        elif new_slots > S:
            grow = new_slots - S
            self.slot_part = np.concatenate([self.slot_part, np.full(grow, -1, dtype=np.int64)])
            self.slot_pidx = np.concatenate([self.slot_pidx, np.zeros(grow, dtype=np.int64)])
            self.slot_ts = np.concatenate([self.slot_ts, np.full(grow, -1, dtype=np.int64)])
        return dropped

    # ---- helpers ---------------------------------------------------------------------
    def n_partitions(self) -> int:
        return len(self.part_tokens)

    def partition_pages(self, p: int) -> int:
        return -(-self.part_tokens[p] // self.T)

    # ---- one decode step -------------------------------------------------------------
    def decode(self, q_bits: np.ndarray, want_output: bool = True
               ) -> Tuple[Optional[np.ndarray], StepTrace]:
        cfg = self.cfg
        T = self.T
        q = bf16_to_f32(q_bits)                                   # [G][d]
        P = self.n_partitions()

        # Select: score, then top-k
        if self.kind == PART_PAGE_MINMAX:
            scores = score_minmax(q, self.sum_min[:P], self.sum_max[:P])
        elif self.kind == PART_TOKEN_DOT:
            scores = score_dot(q, self.sum_vec[:P * T])
        else:
            scores = score_dot(q, self.sum_vec[:P])
        selected = topk_select(scores, cfg.topk)

        # selected candidates -> partitions of the cache manager (+ token masks)
        if self.kind == PART_TOKEN_DOT:
            parts = np.unique(selected // T)
            mask_of: Dict[int, int] = {int(p): 0 for p in parts}
            for tok in selected:
                mask_of[int(tok) // T] |= 1 << (int(tok) % T)
        else:
            parts = selected
            mask_of = {}

        # Retrieve step 1 + bucketed LRU
        n_pages_of = np.asarray([self.partition_pages(p) for p in range(P)], dtype=np.int64)
        resident = np.asarray(self.part_resident, dtype=np.int64)
        res = bucketed_lru_step(self.slot_part, self.slot_pidx, self.slot_ts, resident,
                                n_pages_of, parts, self.t, cfg.lru_buckets, cfg.evict_exact)
        self.part_resident = [int(x) for x in resident]

        # page list: selected partitions ascending, pages of a partition in order, then tail
        where: Dict[Tuple[int, int], int] = {}
        for s in np.nonzero(self.slot_part >= 0)[0]:
            where[(int(self.slot_part[s]), int(self.slot_pidx[s]))] = int(s)
        bypassed = set(res.bypass)
        pages: List[Tuple[int, int, int, int]] = []
        host_pages: List[Tuple[int, int]] = []                    # (host page, mask)
        for p in (int(x) for x in parts):
            npg = int(n_pages_of[p])
            for i in range(npg):
                valid = min(T, self.part_tokens[p] - i * T)
                mask = mask_of[p] if self.kind == PART_TOKEN_DOT else (1 << valid) - 1
                slot = -1 if p in bypassed else where[(p, i)]
                pages.append((p, i, mask, slot))
                # Retrieve step 3: Partition Offset -> slice of the CPU page table
                host_pages.append((self.cpu_page_table[self.part_offset[p] + i], mask))
        for j, page in enumerate(self.tail_pages):
            valid = self.tail_len if j == len(self.tail_pages) - 1 else T
            pages.append((-1, j, (1 << valid) - 1, -2))
            host_pages.append((page, (1 << valid) - 1))

        out = None
        if want_output:
            rows_k, rows_v = [], []
            for page, mask in host_pages:
                keep = [r for r in range(T) if (mask >> r) & 1]
                rows_k.append(self.page_k[page, keep])
                rows_v.append(self.page_v[page, keep])
            K = bf16_to_f32(np.concatenate(rows_k)) if rows_k else np.zeros((0, self.d), F32)
            V = bf16_to_f32(np.concatenate(rows_v)) if rows_v else np.zeros((0, self.d), F32)
            scale = cfg.sm_scale if cfg.sm_scale != 0.0 else 1.0 / np.sqrt(self.d)
            out = attention_fp64(q, K, V, scale)

        trace = StepTrace(selected=selected, partitions=np.asarray(parts, dtype=np.int64),
                          hits=res.hits, misses=res.misses, bypass=res.bypass,
                          evicted=res.evicted, pages=pages,
                          slot_part=self.slot_part.copy(), slot_pidx=self.slot_pidx.copy(),
                          slot_ts=self.slot_ts.copy(),
                          resident=np.asarray(self.part_resident, dtype=np.int64),
                          scores=scores)
        self.t += 1
        return out, trace


# --------------------------------------------------------------------------------------
# The library-shaped front: requests x layers x kv heads
# --------------------------------------------------------------------------------------

class SpinOracle:
    """Same call sequence as the C library: open a request, append KV, decode steps."""

    def __init__(self, cfg: OracleConfig):
        self.cfg = cfg
        self.G = cfg.num_q_heads // cfg.num_kv_heads
        self.requests: Dict[int, List[List[OracleSet]]] = {}
        self._next = 0
        self.counters = dict(steps=0, selected_partitions=0, selected_pages=0, hit_pages=0,
                             miss_pages=0, evicted_pages=0, bypass_pages=0, tail_pages=0)
        self.last_trace: Dict[Tuple[int, int, int], StepTrace] = {}

    def request_open(self, slots_per_set: int) -> int:
        r = self._next
        self._next += 1
        self.requests[r] = [[OracleSet(self.cfg, slots_per_set)
                             for _ in range(self.cfg.num_kv_heads)]
                            for _ in range(self.cfg.num_layers)]
        return r

    def request_close(self, req: int):
        del self.requests[req]

    def set_budget(self, req: int, slots_per_set: int):
        """Resize every (layer, kv head) set of a request (see OracleSet.resize)."""
        for layer in self.requests[req]:
            for st in layer:
                st.resize(slots_per_set)

    def reindex(self, req: int, layer: int):
        """Fold the full tail pages of every kv head's set of (request, layer) into its clusters."""
        return [st.reindex() for st in self.requests[req][layer]]

    def set(self, req: int, layer: int, head: int) -> OracleSet:
        return self.requests[req][layer][head]

    def append_kv(self, req: int, layer: int, k_bits: np.ndarray, v_bits: np.ndarray,
                  token_partition: Optional[np.ndarray] = None,
                  centroids_bits: Optional[np.ndarray] = None):
        """k_bits, v_bits: uint16 [n_tokens][num_kv_heads][head_dim].  Cluster prefill adds
        token_partition int [n_tokens][num_kv_heads] and centroids uint16 [C][Hkv][d]."""
        for h, st in enumerate(self.requests[req][layer]):
            if token_partition is not None:
                st.append_clustered(k_bits[:, h], v_bits[:, h], token_partition[:, h],
                                    centroids_bits[:, h])
            else:
                st.append_tokens(k_bits[:, h], v_bits[:, h])

    def decode_step(self, layer: int, req_ids: Sequence[int], q_bits: np.ndarray,
                    want_output: bool = True) -> Optional[np.ndarray]:
        """q_bits: uint16 [n_req][num_q_heads][head_dim] -> fp64 [n_req][num_q_heads][d]."""
        cfg, G = self.cfg, self.G
        out = np.zeros((len(req_ids), cfg.num_q_heads, cfg.head_dim)) if want_output else None
        for i, r in enumerate(req_ids):
            for h, st in enumerate(self.requests[r][layer]):
                o, tr = st.decode(q_bits[i, h * G:(h + 1) * G], want_output)
                if want_output:
                    out[i, h * G:(h + 1) * G] = o
                self.last_trace[(r, layer, h)] = tr
                c = self.counters
                c["steps"] += 1
                c["selected_partitions"] += len(tr.partitions)
                n_tail = sum(1 for pg in tr.pages if pg[3] == -2)
                n_byp = sum(1 for pg in tr.pages if pg[3] == -1)
                n_sel_pages = len(tr.pages) - n_tail
                n_miss = sum(st.partition_pages(p) for p in tr.misses)
                c["selected_pages"] += n_sel_pages
                c["tail_pages"] += n_tail
                c["bypass_pages"] += n_byp
                c["miss_pages"] += n_miss
                c["hit_pages"] += n_sel_pages - n_miss
                c["evicted_pages"] += len(tr.evicted)
        return out

    def step_bytes(self) -> Dict[str, int]:
        """Algorithmic traffic so far, after Eq. 1-3: summaries scanned and selected KV read
        from HBM, missed pages crossing PCIe (and written into HBM slots)."""
        page_bytes = 2 * self.cfg.page_tokens * self.cfg.head_dim * 2
        c = self.counters
        return dict(pcie=(c["miss_pages"]) * page_bytes,
                    kv_read=(c["selected_pages"] + c["tail_pages"]) * page_bytes)
