// Select (Table 1: score(q, k_sums) -> topk; Section 4.1 "Select").
//
// k_score streams the summary segments of every set of the batch once (HBM bound: 512 B per
// page for min/max summaries, 256 B per token key or centroid; a 64 KiB segment is staged in
// shared memory by four TMA bulk copies with an mbarrier each) and writes one fp32 score per
// candidate.  The summation order is fixed so that the CPU oracle reproduces every score bit
// for bit: a lane owns 8 consecutive channels (one 16-byte load) and adds them left to right;
// the 16 lanes of a row are then combined by a butterfly (xor 1, 2, 4, 8), which is the
// balanced tree over adjacent blocks; the group's query heads are added in ascending order.
// Products of two bf16 values are exact in fp32, so fused or separate multiply-add agree.
//
// In its fused form the last scoring CTA of a set (an arrival counter per set) carries on
// with that set's top-k and cache management (stages.cuh) while other sets are still being
// scored, so the step needs no top-k or cache-manager launch.  k_topk is the stand-alone
// top-k for candidate counts beyond one CTA's shared memory: a thread-block cluster per set.
#define SPIN_FILE_ID 2
#include "append_body.cuh"
#include "stages.cuh"

namespace spin {

namespace {

constexpr int kScoreThreads = 256;
constexpr int kTopkThreads = 512;

__device__ __forceinline__ void unpack8(uint4 raw, float *f) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

// d = a * b + c with a, b bf16 and c, d fp32: the product of two bf16 values is exact in fp32, so
// this is fmaf on the widened operands, one rounding, without the instructions that widen them.
__device__ __forceinline__ float fma_bf16(uint16_t a, uint16_t b, float c) {
  float d;
  asm("fma.rn.f32.bf16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
  return d;
}

// Scores of E candidates at once for this lane's 8 channels and all G heads; the 16 lanes of a
// row are combined by a butterfly.  For min/max summaries max(q*min, q*max) equals
// q * (q >= 0 ? max : min) exactly (min <= max and the products are exact), so the operand is
// picked with one bitwise blend per channel pair on the packed bf16 words (masks precomputed
// per head) instead of two multiplies and a max per channel.
// The E x G block sums of a lane go up the balanced tree together (lanes l and l^1, then l^2,
// l^4, l^8: both partners form the same sum, addition being commutative).  While more than one
// value is left in a lane, a level also halves that number: the partners keep one half of the
// values each and trade the other, so a level costs n/2 shuffles instead of n, and the
// shuffles of a level are independent of one another (their latency is paid once per level,
// not once per candidate).  After log2(E x G) levels a lane holds one (candidate, head) total;
// the heads of a candidate are then added in ascending order.
// Returns the lane's candidate total; *which = the candidate (0..E-1) it belongs to, *writer =
// this lane is the one that stores it.
template <int G, bool MINMAX, int E>
__device__ __forceinline__ float score_group(const uint4 (&lo)[E], const uint4 (&hi)[E], const uint32_t (&qw)[G][4],
                                             const uint32_t (&qsel)[G][4], uint32_t row_mask, int *which, bool *writer) {
  constexpr int N = E * G;
  static_assert(N <= 16 && (N & (N - 1)) == 0, "one value per lane of the row at most");
  constexpr int K = N == 16 ? 4 : N == 8 ? 3 : N == 4 ? 2 : N == 2 ? 1 : 0;      // trading levels
  constexpr int KG = G == 8 ? 3 : G == 4 ? 2 : G == 2 ? 1 : 0, KE = K - KG;
  float v[N];
#pragma unroll
  for (int i = 0; i < N; ++i) v[i] = -0.0f;                    // -0.0 + p = p for every p: the first term is the bare product
  // channels left to right, one rounding per add (the mixed-precision fma takes the bf16 halves
  // as they are: exact product, fp32 sum); the E x G chains advance together
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint16_t xl[N], xh[N], ql[G], qh[G];
#pragma unroll
    for (int g = 0; g < G; ++g) asm("mov.b32 {%0, %1}, %2;" : "=h"(ql[g]), "=h"(qh[g]) : "r"(qw[g][j]));
#pragma unroll
    for (int e = 0; e < E; ++e) {
      const uint32_t a = j == 0 ? lo[e].x : j == 1 ? lo[e].y : j == 2 ? lo[e].z : lo[e].w;
      const uint32_t m = j == 0 ? hi[e].x : j == 1 ? hi[e].y : j == 2 ? hi[e].z : hi[e].w;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const uint32_t w = MINMAX ? ((m & qsel[g][j]) | (a & ~qsel[g][j])) : a;
        asm("mov.b32 {%0, %1}, %2;" : "=h"(xl[e * G + g]), "=h"(xh[e * G + g]) : "r"(w));
      }
    }
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = fma_bf16(ql[i % G], xl[i], v[i]);
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = fma_bf16(qh[i % G], xh[i], v[i]);
  }
  const int lane = threadIdx.x & 15;
#pragma unroll
  for (int level = 0; level < 4; ++level) {
    if (level < K) {
      const bool up = (lane >> level) & 1;
      const int half = N >> (level + 1);
#pragma unroll
      for (int i = 0; i < N / 2; ++i)
        if (i < half) {
          const float send = up ? v[i] : v[i + half], keep = up ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(row_mask, send, 1 << level);
        }
    } else {
      v[0] = v[0] + __shfl_xor_sync(row_mask, v[0], 1 << level);
    }
  }
  // lane bit `level` chose index bit K-1-level: candidate = the top KE index bits, head = the low KG
  int e_idx = 0;
#pragma unroll
  for (int level = 0; level < KE; ++level) e_idx |= ((lane >> level) & 1) << (KE - 1 - level);
  int head_lanes = 0;                                            // the lane bits that say which head the lane holds
#pragma unroll
  for (int t = 0; t < KG; ++t) head_lanes |= 1 << (K - 1 - t);
  float tot = 0.f;
#pragma unroll
  for (int h = 0; h < G; ++h) {                                  // heads in ascending order
    int src = lane & ~head_lanes;
#pragma unroll
    for (int t = 0; t < KG; ++t) src |= ((h >> t) & 1) << (K - 1 - t);
    const float sh = G > 1 ? __shfl_sync(row_mask, v[0], src, 16) : v[0];
    tot = h == 0 ? sh : tot + sh;
  }
  *which = e_idx;
  *writer = (lane & head_lanes) == 0 && (lane >> K) == 0;
  return tot + 0.0f;                                             // -0.0 -> +0.0
}

// How the scoring kernel cuts a step into work items.  Items run in this order: the sets' tail
// items (one per set: in-grid append, tail flag), then request by request, head by head, the
// summary segments of each set (as many as that request has: mixed lengths cost no idle items).
struct ScoreGrid {
  int32_t n_sets, n_items;
  int32_t persistent;                  // 1: a resident grid draws items from a queue; 0: item = blockIdx.x
  int32_t item_prefix[kMaxBatch + 1];  // first segment item of each request (all its heads follow)
};

// One work item (uniform over the CTA): x < 0 is the tail item of batch set b, else summary
// segment x of that set.
template <int G, bool MINMAX>
__device__ __forceinline__ void score_item(const DevCtx &c, const Batch &bt, const __nv_bfloat16 *__restrict__ q,
                                           const __nv_bfloat16 *__restrict__ k_new, const __nv_bfloat16 *__restrict__ v_new,
                                           int fuse, int keys_cap, int tbl_cap, int b, int x, uint8_t *dyn_smem,
                                           unsigned long long *s_bar, uint32_t &phase_bits, const int *s_dead_in, int *s_dead) {
  const int i_req = b / c.Hkv, head = b % c.Hkv;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  if (x < 0) {
    // the set's tail CTA: appends this step's token (unless a stand-alone append already ran)
    // and tells the attention kernel that the tail page is complete
    __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
    if (bt.append_in_grid) append_edge_body(c, set, i_req, head, k_new, v_new, 1, bt.n_tokens[i_req], bt.epoch, krows);
    __syncthreads();
    if (threadIdx.x == 0) flag_publish(c.tail_ready + b, bt.epoch);
    return;
  }
  if (x == 0) dbg_ts(b, 0);
  // the host's count: the in-grid append never completes a page, so it equals the set's state
  const int n_partitions = bt.n_partitions[i_req];
  const int n_cand = c.kind == kKindToken ? n_partitions * kPageTokens : n_partitions;
  const int seg_entries = 1 << c.sum_shift;
  const int e0 = x * seg_entries;
  // the CTAs that count towards the set's arrival counter: one per non-empty segment, and
  // segment 0 even when the set has no candidate yet
  const int segs_here = max(1, (n_cand + seg_entries - 1) >> c.sum_shift);
  if (x >= segs_here) return;
  const int seg = e0 < n_cand ? c.dir_sumseg[(size_t)set * c.dir_sum + x] : 0;
  if (seg < 0 && threadIdx.x == 0) dev_error(c, kErrBounds);
  if (e0 < n_cand && seg >= 0) {
  const int n_here = min(seg_entries, n_cand - e0);
  constexpr int kEntry = MINMAX ? 2 * kRowBytes : kRowBytes;
  float *out = c.scores + (size_t)b * c.max_cand + e0;
  constexpr int kPerHalfWarp = MINMAX ? 8 : 16;          // entries of the segment per half-warp
  constexpr int kPerGroup = kPerHalfWarp / 4;            // entries per half-warp and quarter
  // The segment (or what the set has of it) comes in as four bulk copies (TMA), 16 KiB each, one
  // mbarrier per copy, issued by one thread; the warps score a quarter as soon as its barrier
  // completes, so a CTA keeps its whole 64 KiB in flight with four instructions.  The four
  // barriers are initialised once per CTA (by the kernel); a CTA that works on several items
  // carries one phase bit per barrier from item to item (phase_bits, uniform over the CTA).
  // Waits on the barriers are bounded: a copy that never lands is reported (the quarter is then
  // scored from whatever the staging area holds: the error bit says that this step's results are
  // void), and from its next item on the CTA scores nothing (its barriers' phases are no longer
  // known, and the copy may still be writing the staging area): it only counts its arrivals.
  // That decision is uniform over the CTA, so the rows' shuffles never lose a lane.
  constexpr int kGroupEntries = 16 * kPerGroup;
  const uint8_t *gseg = c.summaries + ((size_t)seg << c.sum_shift) * kEntry;
  const bool dead = *s_dead_in != 0;
  if (threadIdx.x == 0 && !dead) {
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // earlier generic accesses to the staging area
#pragma unroll
    for (int gI = 0; gI < 4; ++gI) {
      const int first = gI * kGroupEntries, cnt = min(kGroupEntries, n_here - first);
      if (cnt > 0) {
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&s_bar[gI]), bytes = (uint32_t)cnt * kEntry;
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(dyn_smem + (size_t)first * kEntry);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                     ::"r"(dst), "l"(gseg + (size_t)first * kEntry), "r"(bytes), "r"(bar) : "memory");
      }
    }
  }
  const int lane16 = threadIdx.x & 15, grp = threadIdx.x >> 4;
  // the two 16-lane rows of a warp may leave the loop at different times: each shuffles
  // only among its own lanes
  const uint32_t row_mask = 0xffffu << (threadIdx.x & 16);

  uint32_t qw[G][4], qsel[G][4];                        // the lane's 8 channels of every head (packed pairs), and the masks of their signs
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint4 raw = *reinterpret_cast<const uint4 *>(
        q + ((size_t)i_req * c.Hq + head * G + g) * kHeadDim + lane16 * 8);
    float qf[8];
    unpack8(raw, qf);
    qw[g][0] = raw.x; qw[g][1] = raw.y; qw[g][2] = raw.z; qw[g][3] = raw.w;
#pragma unroll
    for (int j = 0; j < 4; ++j)
      qsel[g][j] = (qf[2 * j] >= 0.f ? 0x0000ffffu : 0u) | (qf[2 * j + 1] >= 0.f ? 0xffff0000u : 0u);
  }
  uint8_t *stage = dyn_smem + lane16 * 16;
#pragma unroll
  for (int gI = 0; gI < 4; ++gI) {
    if (gI * kGroupEntries < n_here && !dead) {
      const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&s_bar[gI]), parity = (phase_bits >> gI) & 1u;
      uint32_t done = 0;
      for (int spin = 0; spin < (1 << 22) && !done; ++spin)
        asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n" : "=r"(done) : "r"(bar), "r"(parity) : "memory");
      if (!done) { *s_dead = 1; if (lane16 == 0) dev_error(c, kErrTimeout); }
      phase_bits ^= 1u << gI;
    }
    // the quarter's candidates of this half-warp, kE at a time (as many as give every lane of
    // the row one value to carry up the tree)
    constexpr int kE = kPerGroup * G <= 16 ? kPerGroup : 16 / G;
#pragma unroll
    for (int j0 = 0; j0 < kPerGroup; j0 += kE) {
      uint4 a0[kE], m0[kE];
      bool any = false;
#pragma unroll
      for (int u = 0; u < kE; ++u) {
        const int e = grp + 16 * (gI * kPerGroup + j0 + u);
        if (e < n_here && !dead) {
          a0[u] = *reinterpret_cast<const uint4 *>(stage + (size_t)e * kEntry);
          m0[u] = MINMAX ? *reinterpret_cast<const uint4 *>(stage + (size_t)e * kEntry + kRowBytes) : make_uint4(0, 0, 0, 0);
          any = true;
        } else {
          a0[u] = make_uint4(0, 0, 0, 0);
          m0[u] = make_uint4(0, 0, 0, 0);
        }
      }
      if (any) {                                                   // uniform over the row: a candidate exists for all its lanes or for none
        int which;
        bool writer;
        const float s0 = score_group<G, MINMAX, kE>(a0, m0, qw, qsel, row_mask, &which, &writer);
        const int e = grp + 16 * (gI * kPerGroup + j0 + which);
        if (writer && e < n_here) out[e] = s0;
      }
    }
  }
  }
  if (!fuse) return;

  // ---- fused continuation: the last CTA of the set to arrive selects and manages the cache ----
  __shared__ union { struct { TopkShared t; CacheShared c; } staged; FastShared fast; } shm;
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&c.sel_count[b], 1) == segs_here - 1;
  __syncthreads();
  if (!s_last) return;
  dbg_ts(b, 9);
  __threadfence();
  if (threadIdx.x == 0) c.sel_count[b] = 0;                 // ready for the next step
  if (fuse == 3) {
    // selection runs in the cluster kernel behind this one: tell it that this set is scored
    if (threadIdx.x == 0) flag_publish(c.scored + b, bt.epoch);
    return;
  }
  if (fuse == 2) {
    select_fast<kScoreThreads>(c, bt, b, i_req, set, dyn_smem, keys_cap, tbl_cap, shm.fast);
    return;
  }
  topk_stage<kScoreThreads, false>(c, b, n_partitions, reinterpret_cast<uint32_t *>(dyn_smem), keys_cap, shm.staged.t);
  cache_stage<kScoreThreads>(c, b, set, __ldcg(c.n_parts + b), bt.tail_pages[i_req], bt.tail_len[i_req],
                             bt.epoch, reinterpret_cast<int32_t *>(dyn_smem), shm.staged.c);
}

// The scoring kernel: one work item per CTA, or -- when scoring is long (many more items than
// CTAs fit on the GPU) and the sets' selection continues in this kernel -- a grid that is
// resident all at once and draws its items from a queue.  A dependent grid is launched once
// every CTA of this one has started: with thousands of one-item CTAs that is most of the way
// through scoring, and the host link would idle until then although the first sets' missed
// pages have long been listed.  The resident form starts all its CTAs at once and leaves room
// on some SMs, so attention CTAs move in from the beginning.
template <int G, bool MINMAX>
__global__ void __launch_bounds__(kScoreThreads, 3)
k_score(DevCtx c, Batch bt, const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_new,
        const __nv_bfloat16 *__restrict__ v_new, int fuse, int keys_cap, int tbl_cap, ScoreGrid sg) {   // fuse: 0 none, 1 staged, 2 fast, 3 flag only
  extern __shared__ __align__(16) uint8_t dyn_smem[];      // staging area; reused by the fused continuation
  pdl_launch_next();
  pdl_wait_prev();
  __shared__ int s_item[2];
  __shared__ __align__(8) unsigned long long s_bar[4];     // one per quarter of the staged segment
  __shared__ int s_dead[2];                                // [0] read at an item's start, [1] set by a wait that ran out
  uint32_t phase_bits = 0;
  const bool pers = sg.persistent != 0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int gI = 0; gI < 4; ++gI)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(&s_bar[gI])));
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    s_dead[0] = s_dead[1] = 0;
    // the first item is the CTA's own number (no storm on the counter at the start); the queue
    // hands out the items from gridDim.x on
    s_item[0] = (int)blockIdx.x;
  }
  __syncthreads();                                         // the initialised mbarriers are visible to all
  for (int it = 0;; ++it) {
    const int item = pers ? s_item[it & 1] : (int)blockIdx.x;
    if (item >= sg.n_items) break;
    int next = 0;
    if (pers && threadIdx.x == 0) next = (int)gridDim.x + atomicAdd(c.score_queue, 1);   // in flight while this item is worked on
    if (item == 0 && threadIdx.x == 0) *c.fetch_count = 0;               // new step, new miss queue
    int b = item, x = -1;                                                // the sets' tail items come first
    if (item >= sg.n_sets) {
      const int id = item - sg.n_sets;
      int lo = 0, hi = bt.n_req;                                         // request whose items hold `id`
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (sg.item_prefix[mid] <= id) lo = mid; else hi = mid;
      }
      const int segs_r = (sg.item_prefix[lo + 1] - sg.item_prefix[lo]) / c.Hkv, off = id - sg.item_prefix[lo];
      b = lo * c.Hkv + off / segs_r;
      x = off % segs_r;
    }
    score_item<G, MINMAX>(c, bt, q, k_new, v_new, fuse, keys_cap, tbl_cap, b, x, dyn_smem, s_bar, phase_bits, &s_dead[0], &s_dead[1]);
    if (!pers) return;
    if (threadIdx.x == 0) { s_item[(it + 1) & 1] = next; if (s_dead[1]) s_dead[0] = 1; }
    __syncthreads();
  }
  // the last CTA out leaves the queue ready for the next step (every other CTA has drawn its
  // last item by then)
  if (pers && threadIdx.x == 0 && atomicAdd(c.score_done, 1) == (int)gridDim.x - 1) {
    *c.score_queue = 0;
    *c.score_done = 0;
  }
}


#ifdef SPIN_TIMING
__device__ unsigned long long g_dbg_st[160][64];
__device__ __forceinline__ void dbg_st(int slot) { if (slot < 64) { g_dbg_st[blockIdx.x % 160][slot] = (unsigned long long)clock64(); } }
#else
__device__ __forceinline__ void dbg_st(int) {}
#endif

// ---------------------------------------------------------------------------------------------
// Streaming form of the scoring kernel (spin_config.resident_scoring = 2).  One CTA per SM,
// resident for the whole step, ten warps:
//   * a producer warp keeps a ring of stages filled, one TMA bulk copy per stage (a full and an
//     empty mbarrier per stage); a stage holds the summaries of 16 consecutive candidates;
//   * up to eight consumer warps, each the owner of the stages s with s % warps == its number,
//     score a stage in two phases and without a shuffle (score_stage);
//   * a helper warp prepares each work item's query heads (the packed bf16 words and, for
//     min/max summaries, the blend masks of their signs) in a small ring of slots ahead of the
//     consumers.
// The work items of a step (the sets' tail items, then every set's segments, set by set) are
// dealt out round robin, item j of CTA i being number i + j * gridDim.x: all three roles walk the
// same list without talking to each other, the first sets' summaries are the first bytes asked
// of HBM, and sets are scored in order.  Because the grid is a single wave, the kernels behind
// it (selection, attention) become resident at once and follow set by set.  Scores reach the
// set's selection CTA through a hand-over buffer whose words say themselves whether they have
// been written (take_score), so no fence stands between scoring and selection; the per-set
// arrival counter is only a hint for when to start looking.
// Measured on the Llama-shaped configuration this form scores 67 MB in 35 us against 25 us of
// the one-CTA-per-segment form with its three CTAs per SM (the eight scoring warps of an SM
// are bound by instruction latency), so it is not the default.
constexpr int kStageEntries = 16;
constexpr int kMaxStages = 16;
constexpr int kQSlots = 4;
constexpr int kStreamThreads = kScoreThreads + 64;                     // consumers, producer warp, helper warp

template <int G, bool MINMAX> struct StageLayout {
  static constexpr int kEntry = MINMAX ? 2 * kRowBytes : kRowBytes;
  static constexpr int kStride = kStageEntries * kEntry;               // one stage
  static constexpr int kQF = 0;                                        // a query slot: G x 64 words of packed bf16 pairs ...
  static constexpr int kQM = G * 64 * 4;                               // ... and G x 64 blend masks (min/max only)
  static constexpr int kQStride = kQM + (MINMAX ? G * 64 * 4 : 0);
};

struct ItemRef { int b, x; };      // x < 0: the tail item of batch set b; else summary segment x of it

__device__ __forceinline__ ItemRef resolve_item(const DevCtx &c, const Batch &bt, const ScoreGrid &sg, int item) {
  if (item < sg.n_sets) return ItemRef{item, -1};
  const int id = item - sg.n_sets;
  int lo = 0, hi = bt.n_req;                                           // request whose items hold `id`
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (sg.item_prefix[mid] <= id) lo = mid; else hi = mid;
  }
  const int segs_r = (sg.item_prefix[lo + 1] - sg.item_prefix[lo]) / c.Hkv, off = id - sg.item_prefix[lo];
  return ItemRef{lo * c.Hkv + off / segs_r, off % segs_r};
}

__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t done;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(done) : "r"(bar), "r"(parity) : "memory");
  return done;
}
// bounded: a barrier that never completes is reported, not waited for
__device__ __forceinline__ bool mbar_wait(const DevCtx &c, uint32_t bar, uint32_t parity) {
  for (int spin = 0; spin < (1 << 22); ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    __nanosleep(64);                               // a waiting warp leaves the issue slots to the scoring warps
  }
  dev_error(c, kErrTimeout);
  return false;
}
// a shared-memory word that only ever grows: wait (bounded) until it has reached `want`
__device__ __forceinline__ bool smem_wait_ge(const DevCtx &c, const int *word, int want) {
  for (int spin = 0; spin < (1 << 22); ++spin) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];\n" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(word)) : "memory");
    if (v >= want) return true;
    __nanosleep(64);
  }
  dev_error(c, kErrTimeout);
  return false;
}
__device__ __forceinline__ int smem_load_acquire(const int *word) {
  int v;
  asm volatile("ld.acquire.cta.shared.s32 %0, [%1];\n" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(word)) : "memory");
  return v;
}
__device__ __forceinline__ void smem_store_release(int *word, int v) {
  asm volatile("st.release.cta.shared.s32 [%0], %1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(word)), "r"(v) : "memory");
}

// Scoring of one stage by one warp, in two phases and without a shuffle.
// Phase 1: sixteen lanes per candidate, a lane per block of 8 channels (the lane keeps its 8
// channels of every head's query, and for min/max summaries the blend masks of their signs, in
// registers): the block is added left to right for every head, and the G block sums go back
// into the candidate's own row, into the 16-byte piece the lane has just read (its block's
// piece of the row; the row is dead once it has been read).
// Phase 2: a lane per candidate reads its 16 x G block sums (the pieces' XOR swizzle keeps lanes
// a candidate apart on different banks), combines them by the balanced tree over adjacent
// pairs, adds the heads in ascending order and writes the score.
template <int G, bool MINMAX>
__device__ __forceinline__ void score_stage(uint8_t *stage, int cnt, const uint32_t *qfp, const uint32_t *qmp, int lane,
                                            float *out) {
  static_assert(G <= 4, "the block sums of a candidate go into one 16-byte piece per block");
  constexpr int kEntry = MINMAX ? 2 * kRowBytes : kRowBytes;
  const int blk = lane & 15;
  uint32_t qw[G][4], qsel[G][4];                                       // the lane's 8 channels of every head, packed pairs
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint4 v = *reinterpret_cast<const uint4 *>(qfp + g * 64 + 4 * blk);
    qw[g][0] = v.x; qw[g][1] = v.y; qw[g][2] = v.z; qw[g][3] = v.w;
    if (MINMAX) {
      const uint4 k = *reinterpret_cast<const uint4 *>(qmp + g * 64 + 4 * blk);
      qsel[g][0] = k.x; qsel[g][1] = k.y; qsel[g][2] = k.z; qsel[g][3] = k.w;
    }
  }
  // two candidates per half-warp and iteration (candidates e and e + 2): their 2 x G chains are
  // independent, which is what fills the issue slots between two dependent adds of one chain
#pragma unroll 1
  for (int p = 0; p < kStageEntries / 4; ++p) {
    const int e0 = 4 * p + (lane >> 4);
    float v[2][4];
    uint32_t a[2][4], m[2][4];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int e = e0 + 2 * u;
#pragma unroll
      for (int g = 0; g < 4; ++g) v[u][g] = -0.0f;                     // -0.0 + p = p for every p: the first term is the bare product
      if (e < cnt) {
        const uint8_t *piece = stage + e * kEntry + (blk << 4);
        const uint4 lo = *reinterpret_cast<const uint4 *>(piece);
        const uint4 hi = MINMAX ? *reinterpret_cast<const uint4 *>(piece + kRowBytes) : make_uint4(0, 0, 0, 0);
        a[u][0] = lo.x; a[u][1] = lo.y; a[u][2] = lo.z; a[u][3] = lo.w;
        m[u][0] = hi.x; m[u][1] = hi.y; m[u][2] = hi.z; m[u][3] = hi.w;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) { a[u][j] = 0u; m[u][j] = 0u; }
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint16_t xl[2][G], xh[2][G], ql[G], qh[G];
#pragma unroll
      for (int g = 0; g < G; ++g) {
        asm("mov.b32 {%0, %1}, %2;" : "=h"(ql[g]), "=h"(qh[g]) : "r"(qw[g][j]));
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          // max(q*min, q*max) = q * (q >= 0 ? max : min) exactly: the operand is picked on the packed words
          const uint32_t w = MINMAX ? ((m[u][j] & qsel[g][j]) | (a[u][j] & ~qsel[g][j])) : a[u][j];
          asm("mov.b32 {%0, %1}, %2;" : "=h"(xl[u][g]), "=h"(xh[u][g]) : "r"(w));
        }
      }
      // channels left to right, one rounding per add; the 2 x G chains advance together
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int g = 0; g < G; ++g) v[u][g] = fma_bf16(ql[g], xl[u][g], v[u][g]);
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int g = 0; g < G; ++g) v[u][g] = fma_bf16(qh[g], xh[u][g], v[u][g]);
    }
    // the block sums go back into the candidate's row, block b into piece b ^ (e & 7): every lane of
    // the row has read its piece by now (the barrier), and lanes a candidate apart will find
    // their pieces in different banks
    __syncwarp();
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int e = e0 + 2 * u;
      if (e < cnt) {
        uint8_t *dst = stage + e * kEntry + ((blk ^ (e & 7)) << 4);
        if (G == 4) *reinterpret_cast<float4 *>(dst) = make_float4(v[u][0], v[u][1], v[u][2], v[u][3]);
        else if (G == 2) *reinterpret_cast<float2 *>(dst) = make_float2(v[u][0], v[u][1]);
        else *reinterpret_cast<float *>(dst) = v[u][0];
      }
    }
  }
  __syncwarp();
  if (lane < cnt) {
    const uint8_t *row = stage + lane * kEntry;
    const int sw = lane & 7;
    float lvl[4][G];                                                   // pending partial sums of the tree, one per level
    float tot[G];
#pragma unroll
    for (int b2 = 0; b2 < 16; ++b2) {
      float s[G];
      const uint8_t *pc = row + ((b2 ^ sw) << 4);
      if (G == 4) { const float4 t = *reinterpret_cast<const float4 *>(pc); s[0] = t.x; s[1] = t.y; s[G > 2 ? 2 : 0] = t.z; s[G > 3 ? 3 : 0] = t.w; }
      else if (G == 2) { const float2 t = *reinterpret_cast<const float2 *>(pc); s[0] = t.x; s[G > 1 ? 1 : 0] = t.y; }
      else s[0] = *reinterpret_cast<const float *>(pc);
      // binary counter: block b2 closes as many levels as it has trailing one bits
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float acc = s[g];
#pragma unroll
        for (int l = 0; l < 4; ++l) {
          if ((b2 >> l) & 1) acc = lvl[l][g] + acc;                    // earlier half + later half
          else { lvl[l][g] = acc; break; }
        }
        if (b2 == 15) tot[g] = acc;
      }
    }
    float sc = tot[0];
#pragma unroll
    for (int g = 1; g < G; ++g) sc = sc + tot[g];
    out[lane] = sc + 0.0f;                                             // -0.0 -> +0.0
  }
}

template <int G, bool MINMAX>
__global__ void __launch_bounds__(kStreamThreads, 2)
k_score_stream(DevCtx c, Batch bt, const __nv_bfloat16 *__restrict__ q, const __nv_bfloat16 *__restrict__ k_new,
               const __nv_bfloat16 *__restrict__ v_new, ScoreGrid sg, int stage_shift, int consumer_shift) {
  using SL = StageLayout<G, MINMAX>;
  const int n_stages = 1 << stage_shift, n_consumers = 1 << consumer_shift;       // powers of two: no divisions in the loops
  extern __shared__ __align__(128) uint8_t ring[];                     // [n_stages][SL::kStride], then [kQSlots][SL::kQStride]
  __shared__ __align__(8) unsigned long long s_full[kMaxStages], s_empty[kMaxStages];
  __shared__ int s_consumed[kMaxStages];                               // phases of a stage that have been scored
  __shared__ int s_qready;                                             // stage-bearing items whose query slot is prepared
  __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
  pdl_launch_next();
  const int tid = threadIdx.x;
  if (tid == 0) {
    for (int i = 0; i < n_stages; ++i) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(&s_full[i])));
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;\n" ::"r"((uint32_t)__cvta_generic_to_shared(&s_empty[i])));
      s_consumed[i] = 0;
    }
    s_qready = 0;
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  __syncthreads();                                                     // the only barrier all ten warps share
  if (tid == 0) dbg_st(0);
  pdl_wait_prev();
  if (tid == 0) dbg_st(1);
  uint8_t *qslots = ring + (size_t)n_stages * SL::kStride;
  const int seg_entries = 1 << c.sum_shift, lane = tid & 31;
  const int n_my = (int)blockIdx.x < sg.n_items ? (sg.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  auto cand_of = [&](int i_req) { return c.kind == kKindToken ? bt.n_partitions[i_req] * kPageTokens : bt.n_partitions[i_req]; };
  // entries item j of this CTA has to score (0 for a tail item) and its batch set
  auto item_work = [&](int j, int &b) -> int {
    const ItemRef r = resolve_item(c, bt, sg, (int)blockIdx.x + j * (int)gridDim.x);
    b = r.b;
    if (r.x < 0) return 0;
    const int n_cand = cand_of(r.b / c.Hkv), e0 = r.x * seg_entries;
    return e0 < n_cand ? min(seg_entries, n_cand - e0) : 0;
  };

  if (tid >= kScoreThreads + 32) {
    // ---- helper warp ----
    int prep = 0, prep_j = 0;                      // next stage-bearing item to prepare, and where the search for it goes on
    int sig = 0, sig_j = 0;                        // next one to account for
    uint32_t sig_qc = 0;                           // first stage of item `sig`
    int sig_b = 0, sig_n = -1;                     // its batch set and stage count (-1: not looked up yet)
    bool prep_done = false;
    for (int spin = 0; spin < (1 << 24); ++spin) {
      bool did = false;
      if (!prep_done && prep < sig + kQSlots) {
        int b = 0, n_here = 0;
        while (prep_j < n_my && (n_here = item_work(prep_j, b)) <= 0) ++prep_j;
        if (prep_j >= n_my) prep_done = true;
        else {
          uint8_t *slot = qslots + (size_t)(prep % kQSlots) * SL::kQStride;
          uint32_t *qf = reinterpret_cast<uint32_t *>(slot + SL::kQF);
          uint32_t *qm = reinterpret_cast<uint32_t *>(slot + SL::kQM);
          const uint32_t *qraw = reinterpret_cast<const uint32_t *>(q) + (size_t)b * (G * 64);   // heads of a set are adjacent rows
#pragma unroll
          for (int i = lane; i < G * 64; i += 32) {
            const uint32_t w = qraw[i];
            const float f0 = __uint_as_float(w << 16), f1 = __uint_as_float(w & 0xffff0000u);
            qf[i] = w;
            if (MINMAX) qm[i] = (f0 >= 0.f ? 0x0000ffffu : 0u) | (f1 >= 0.f ? 0xffff0000u : 0u);
          }
          __syncwarp();
          ++prep; ++prep_j;
          if (lane == 0) smem_store_release(&s_qready, prep);
          if (lane == 0) dbg_st(21 + prep);

          did = true;
        }
      }
      if (sig < prep) {
        if (sig_n < 0) {
          int n_here = 0;
          while ((n_here = item_work(sig_j, sig_b)) <= 0) ++sig_j;     // exists: it has been prepared
          sig_n = (n_here + kStageEntries - 1) / kStageEntries;
        }
        bool all = true;
        for (int i = 0; i < sig_n && all; ++i) {
          const uint32_t qc = sig_qc + (uint32_t)i;
          all = smem_load_acquire(&s_consumed[qc & (uint32_t)(n_stages - 1)]) > (int)(qc >> stage_shift);
        }
        if (all) {                                 // the item's stages are scored: its query slot may be reused
          sig_qc += (uint32_t)sig_n;
          ++sig; ++sig_j;
          sig_n = -1;
          did = true;
        }
      } else if (prep_done) break;
      __nanosleep(did ? 32 : 200);
    }
    if (!(prep_done && sig >= prep) && lane == 0) dev_error(c, kErrTimeout);
    return;
  }

  if (tid >= kScoreThreads) {
    // ---- producer warp: segment ids looked up a round of 32 items ahead; a lane copies one row ----
    auto lookup = [&](int j) -> int2 {                                 // (segment id or -1, entries to score)
      if (j >= n_my) return make_int2(-1, 0);
      int b;
      const int n_here = item_work(j, b);
      if (n_here <= 0) return make_int2(-1, 0);
      const ItemRef r = resolve_item(c, bt, sg, (int)blockIdx.x + j * (int)gridDim.x);
      const int set = set_index(c, bt.req[r.b / c.Hkv], bt.layer, r.b % c.Hkv);
      return make_int2(__ldcg(c.dir_sumseg + (size_t)set * c.dir_sum + r.x), n_here);
    };
    uint32_t qc = 0;                                                   // stages issued so far
    int2 mine = lookup(lane);
    for (int j0 = 0; j0 < n_my; j0 += 32) {
      const int2 next = lookup(j0 + 32 + lane);                        // in flight while this round is issued
      for (int jj = 0; jj < 32 && j0 + jj < n_my; ++jj) {
        const int seg = __shfl_sync(0xffffffffu, mine.x, jj), n_here = __shfl_sync(0xffffffffu, mine.y, jj);
        if (n_here <= 0) continue;
        if (lane == 0) dbg_st(42 + j0 + jj);
        if (seg < 0 && lane == 0) dev_error(c, kErrBounds);            // unmapped: the stages are released without rows
        const uint8_t *gseg = c.summaries + ((size_t)max(seg, 0) << c.sum_shift) * SL::kEntry;
        for (int first = 0; first < n_here; first += kStageEntries, ++qc) {
          const int st = (int)(qc & (uint32_t)(n_stages - 1)), cnt = min(kStageEntries, n_here - first);
          const uint32_t full = (uint32_t)__cvta_generic_to_shared(&s_full[st]);
          const uint32_t stage = (uint32_t)__cvta_generic_to_shared(ring + (size_t)st * SL::kStride);
          if (lane == 0) {
            mbar_wait(c, (uint32_t)__cvta_generic_to_shared(&s_empty[st]), ((qc >> stage_shift) & 1u) ^ 1u);   // its consumer is done with it
            // one bulk copy (TMA) per stage: the candidates of a stage are contiguous in their segment
            if (seg >= 0) {
              const uint32_t bytes = (uint32_t)cnt * SL::kEntry;
              asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(full), "r"(bytes) : "memory");
              asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                           ::"r"(stage), "l"(gseg + (size_t)first * SL::kEntry), "r"(bytes), "r"(full) : "memory");
            } else {
              asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(full) : "memory");
            }
          }
        }
      }
      mine = next;
    }
    return;
  }

  // ---- consumers: warp w owns the stages s of the ring with s % n_consumers == w and takes them
  // phase after phase (a stage is always consumed by the same warp: a warp that ran a whole
  // phase ahead of another on the same barrier would be let through by the parity test) ----
  const int warp = tid >> 5;
  uint32_t qc = 0;
  int ordinal = 0;                                                     // stage-bearing items so far
  for (int j = 0; j < n_my; ++j) {
    const int item = (int)blockIdx.x + j * (int)gridDim.x;
    if (item == 0 && tid == 0) *c.fetch_count = 0;                     // new step, new miss queue
    const ItemRef r = resolve_item(c, bt, sg, item);
    const int b = r.b, i_req = b / c.Hkv, head = b % c.Hkv;
    if (r.x < 0) {
      // the set's tail item (these come first in every CTA's list, so the warps are still in
      // step): appends this step's token (unless a stand-alone append already ran) and tells
      // whoever waits for it that the tail page and the set's tables are complete
      const int set = set_index(c, bt.req[i_req], bt.layer, head);
      if (bt.append_in_grid) append_edge_body(c, set, i_req, head, k_new, v_new, 1, bt.n_tokens[i_req], bt.epoch, krows);
      sync_256();
      if (tid == 0) flag_publish(c.tail_ready + b, bt.epoch);
      continue;
    }
    if (r.x == 0) dbg_ts(b, 0);
    if (tid == 0) dbg_st(2 + j);
    const int n_cand = cand_of(i_req), e0 = r.x * seg_entries;
    const int n_here = e0 < n_cand ? min(seg_entries, n_cand - e0) : 0;
    if (n_here <= 0) continue;
    if (warp >= n_consumers) { ++ordinal; continue; }
    float *out = c.score_xfer + (size_t)b * c.max_cand + e0;           // taken out by the set's selection, word by word
    const uint8_t *slot = qslots + (size_t)(ordinal % kQSlots) * SL::kQStride;
    const uint32_t *qf = reinterpret_cast<const uint32_t *>(slot + SL::kQF);
    const uint32_t *qm = reinterpret_cast<const uint32_t *>(slot + SL::kQM);
    bool q_ok = false;
    const uint32_t qc_end = qc + (uint32_t)((n_here + kStageEntries - 1) / kStageEntries);
    // the warp's own stages of this item: those whose number is its own modulo the consumer count
    for (uint32_t mine = qc + (((uint32_t)warp - qc) & (uint32_t)(n_consumers - 1)); mine < qc_end; mine += (uint32_t)n_consumers) {
      const int st = (int)(mine & (uint32_t)(n_stages - 1)), first = (int)(mine - qc) * kStageEntries;
      const int cnt = min(kStageEntries, n_here - first);
      if (!q_ok) { smem_wait_ge(c, &s_qready, ordinal + 1); q_ok = true; }
      uint8_t *stage = ring + (size_t)st * SL::kStride;
      mbar_wait(c, (uint32_t)__cvta_generic_to_shared(&s_full[st]), (mine >> stage_shift) & 1u);
      score_stage<G, MINMAX>(stage, cnt, qf, qm, lane, out + first);
      // the warp has written into the stage (block sums): order those generic-proxy accesses
      // before the bulk copy (async proxy) that will refill it
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      __syncwarp();                                                    // every lane has read the stage
      if (lane == 0) {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"((uint32_t)__cvta_generic_to_shared(&s_empty[st])) : "memory");
        smem_store_release(&s_consumed[st], (int)(mine >> stage_shift) + 1);
        // one more stage of the set is scored.  Only a hint for the set's selection CTA (when to
        // start looking): the scores carry their own arrival, so nothing here waits for them
        asm volatile("red.relaxed.gpu.global.add.s32 [%0], 1;\n" ::"l"(c.sel_count + b) : "memory");
      }
    }
    qc = qc_end;
    ++ordinal;
  }
  if (tid == 0) dbg_st(20);
}

// Stages the streaming kernel scores for a set with n_cand candidates: what its arrival counter reaches.
__host__ __device__ inline int stream_stages_of(int n_cand) { return (n_cand + kStageEntries - 1) / kStageEntries; }

// Waits (bounded) until the set's arrival counter has reached `target`, then clears it for the next step.
__device__ __forceinline__ bool wait_scored(const DevCtx &c, int b, int target) {
  if (!flag_wait(c, c.sel_count + b, target)) return false;
  c.sel_count[b] = 0;
  return true;
}

// Selection and cache management of one set per CTA, on the set's `scored` flag (the streaming
// scoring kernel raises it).  The CTA is resident from the start of the step: while its set is
// still being scored it brings the directories, the GPU page table and the snapshot of the
// partition tables into shared memory (none of them depends on this step's scores; they are
// stable once this step's append has run, which the set's tail flag says).
__global__ void __launch_bounds__(kScoreThreads)
k_select(DevCtx c, Batch bt, int keys_cap, int tbl_cap) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  __shared__ FastShared fast;
  __shared__ int s_ok;
  pdl_launch_next();
  const int tid = threadIdx.x, n_sets = bt.n_req * c.Hkv;
  for (int b = blockIdx.x; b < n_sets; b += gridDim.x) {
    const int i_req = b / c.Hkv, head = b % c.Hkv;
    const int set = set_index(c, bt.req[i_req], bt.layer, head);
    __syncthreads();                                   // the previous set's shared memory is no longer in use
    if (tid == 0) s_ok = flag_wait(c, c.tail_ready + b, bt.epoch);
    __syncthreads();
    if (!s_ok) continue;
    const int S = bt.slots[i_req];
    const FastLayout L = fast_layout(c, dyn_smem, keys_cap, S, tbl_cap);
    fast_prefetch_dirs<kScoreThreads>(c, L, set, S);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();
    fast_prefetch_gpt<kScoreThreads>(c, L, S);
    fast_prefetch_tables<kScoreThreads>(c, L, bt.n_partitions[i_req]);
    if (tid == 0) {
      const int n_cand = c.kind == kKindToken ? bt.n_partitions[i_req] * kPageTokens : bt.n_partitions[i_req];
      s_ok = wait_scored(c, b, stream_stages_of(n_cand));
      dbg_ts(b, 9);
    }
    __syncthreads();
    if (s_ok) select_fast<kScoreThreads>(c, bt, b, i_req, set, dyn_smem, keys_cap, tbl_cap, fast, true, true);
  }
  // a grid that went by the flags must still not complete before the scoring kernel has
  if (blockIdx.x == 0) pdl_wait_prev();
}

// Stand-alone top-k: one thread-block cluster per set (slices of the keys in shared memory).
// With wait_flags a cluster starts as soon as its own set is scored (the flag the scoring
// kernel's last CTA of that set raises) instead of when the whole scoring kernel is done; the
// outcome of the bounded wait is shared through the first CTA so that all CTAs of the
// cluster take the same path through the cluster barriers.
__device__ __forceinline__ void topk_cta(const DevCtx &c, const Batch &bt, int keys_cap, int manage, int tbl_cap,
                                         int wait_flags, uint8_t *dyn_smem) {
  __shared__ union { TopkShared t; FastShared f; TopkRowsShared r; } shm;   // r instead of t when the row-wise select runs
  __shared__ int s_ok;
  TopkShared &tsh = shm.t;
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int b = blockIdx.x / C, i_req = b / c.Hkv, head = b % c.Hkv, tid = threadIdx.x;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  // the first CTA is also the set's cache manager: its tables go to shared memory (behind the
  // keys' slice) before the set is scored -- they do not depend on this step's scores and are
  // stable once this step's kernels have the GPU, which the set's tail flag says -- or, without
  // flags, once the kernel before this one has completed
  const int S = bt.slots[i_req];
  const FastLayout L = fast_layout(c, dyn_smem + (((size_t)keys_cap * 4 + 15) & ~(size_t)15), 0, S, tbl_cap);
  const bool mgr = manage && rank == 0;
  if (wait_flags) {
    if (rank == 0) {
      if (tid == 0) s_ok = flag_wait(c, c.tail_ready + b, bt.epoch);
      __syncthreads();
    }
  } else {
    pdl_wait_prev();
  }
  if (mgr && (!wait_flags || s_ok)) {
    fast_prefetch_dirs<kTopkThreads>(c, L, set, S);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();
    fast_prefetch_gpt<kTopkThreads>(c, L, S);
    fast_prefetch_tables<kTopkThreads>(c, L, bt.n_partitions[i_req]);
  }
  if (wait_flags) {
    if (rank == 0 && tid == 0 && s_ok) {
      // 1: the flag the last scoring CTA of the set raises; 2: the streaming kernel's arrival counter
      const int n_cand = c.kind == kKindToken ? bt.n_partitions[i_req] * kPageTokens : bt.n_partitions[i_req];
      s_ok = wait_flags == 2 ? wait_scored(c, b, stream_stages_of(n_cand)) : flag_wait(c, c.scored + b, bt.epoch);
    }
    cluster.sync();
    const int ok = *cluster.map_shared_rank(&s_ok, 0);
    cluster.sync();                                   // the first CTA's word is not read after this
    if (!ok) return;
  }
  if (rank == 0) dbg_ts(b, 9);
  const bool first = topk_stage<kTopkThreads, true>(c, b, bt.n_partitions[i_req], reinterpret_cast<uint32_t *>(dyn_smem), keys_cap, tsh, wait_flags == 2, &shm.r);
  if (!first || !manage) return;
  const int np = __ldcg(c.n_parts + b);               // with the row-wise select, written by the cluster's other CTAs
  const int32_t *g_parts = c.parts + (size_t)b * c.max_parts;
  for (int r = tid; r < np; r += kTopkThreads) L.s_parts[r] = __ldcg(g_parts + r);
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  __syncthreads();
  cache_fast<kTopkThreads>(c, bt, b, i_req, set, L, np, shm.f);
}

__global__ void __launch_bounds__(kTopkThreads, 1)
k_topk(DevCtx c, Batch bt, int keys_cap, int manage, int tbl_cap, int wait_flags) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  pdl_launch_next();
  topk_cta(c, bt, keys_cap, manage, tbl_cap, wait_flags, dyn_smem);
  // a grid that went by the flags must still not complete before the scoring kernel has
  if (wait_flags && blockIdx.x == 0) pdl_wait_prev();
}


int sm_count_of_device() {
  static int sms_dev[kMaxDevices] = {};
  int &sms = sms_dev[current_device_slot()];
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
  }
  return sms;
}

template <int G>
void launch_score_g(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q, const __nv_bfloat16 *k_new,
                    const __nv_bfloat16 *v_new, dim3 grid, size_t smem, int fuse, int keys_cap, int tbl_cap,
                    const ScoreGrid &sg, cudaStream_t st) {
  static size_t configured_dev[kMaxDevices] = {};
  size_t &configured = configured_dev[current_device_slot()];
  if (smem > configured) {
    cudaFuncSetAttribute(k_score<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaFuncSetAttribute(k_score<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = smem;
  }
  if (sg.persistent) {
    // the resident grid: what fits on the GPU at this shared-memory size, less one CTA on 32
    // SMs (attention CTAs take that room from the start)
    static size_t occ_smem_dev[kMaxDevices] = {};
    static int occ_dev[kMaxDevices][2] = {};
    size_t &occ_smem = occ_smem_dev[current_device_slot()];
    int (&occ)[2] = occ_dev[current_device_slot()];
    if (smem != occ_smem) {
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ[1], k_score<G, true>, kScoreThreads, smem);
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ[0], k_score<G, false>, kScoreThreads, smem);
      occ_smem = smem;
    }
    const int sms = sm_count_of_device(), per_sm = occ[c.kind == kKindPage ? 1 : 0] < 1 ? 1 : occ[c.kind == kKindPage ? 1 : 0];
    int resident = per_sm * sms - (per_sm > 1 ? 32 : 0);
    if (resident > sg.n_items) resident = sg.n_items;
    grid = dim3(resident);
  }
  if (c.kind == kKindPage) launch_pdl(k_score<G, true>, grid, dim3(kScoreThreads), smem, st, 1, c, b, q, k_new, v_new, fuse, keys_cap, tbl_cap, sg);
  else launch_pdl(k_score<G, false>, grid, dim3(kScoreThreads), smem, st, 1, c, b, q, k_new, v_new, fuse, keys_cap, tbl_cap, sg);
}

template <int G>
void launch_stream_g(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q, const __nv_bfloat16 *k_new,
                     const __nv_bfloat16 *v_new, const ScoreGrid &sg, int smem_budget, cudaStream_t st) {
  int n_stages;
  static bool configured_dev[kMaxDevices] = {};
  bool &configured = configured_dev[current_device_slot()];
  if (!configured) {
    cudaFuncSetAttribute(k_score_stream<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    cudaFuncSetAttribute(k_score_stream<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    // the SMs are shared with the selection and attention CTAs that follow on the flags: ask for
    // the largest shared-memory carve-out, which an SM cannot change while CTAs are resident
    cudaFuncSetAttribute(k_score_stream<G, true>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    cudaFuncSetAttribute(k_score_stream<G, false>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    configured = true;
  }
  int grid = sm_count_of_device();
  if (grid > sg.n_items) grid = sg.n_items;
  // as many stages as the budget holds (the selection and attention CTAs share the SM), a
  // multiple of the consumer warps that take them in turn
  const int stride = c.kind == kKindPage ? StageLayout<G, true>::kStride : StageLayout<G, false>::kStride;
  const int qbytes = kQSlots * (c.kind == kKindPage ? StageLayout<G, true>::kQStride : StageLayout<G, false>::kQStride);
  int stage_shift = 1;                                                  // stages: a power of two, 2..kMaxStages
  while ((2 << stage_shift) <= kMaxStages && (size_t)(2 << stage_shift) * stride + qbytes <= (size_t)smem_budget) ++stage_shift;
  n_stages = 1 << stage_shift;
  const int consumer_shift = stage_shift < 3 ? stage_shift : 3;       // one warp per stage, eight at most
  const size_t smem = (size_t)n_stages * stride + qbytes;
  if (c.kind == kKindPage) launch_pdl(k_score_stream<G, true>, dim3(grid), dim3(kStreamThreads), smem, st, 1, c, b, q, k_new, v_new, sg, stage_shift, consumer_shift);
  else launch_pdl(k_score_stream<G, false>, dim3(grid), dim3(kStreamThreads), smem, st, 1, c, b, q, k_new, v_new, sg, stage_shift, consumer_shift);
}

}  // namespace

// Select + (fused or separate) cache management.  Returns the kernels launched.
int launch_select(const DevCtx &c, Batch &b, const __nv_bfloat16 *q, const __nv_bfloat16 *k_new,
                  const __nv_bfloat16 *v_new, int max_cand, cudaStream_t st, Prof *prof) {
  const int n_sets = b.n_req * c.Hkv;
  int segs = (max_cand + (1 << c.sum_shift) - 1) >> c.sum_shift;
  if (segs < 1) segs = 1;                         // segment 0 always runs (arrival counter, miss-queue reset)
  // fused: one CTA can hold a set's keys and the cache manager's tables in shared memory
  const size_t cache_smem = cache_stage_smem_bytes(c.max_parts, c.max_pages, c.max_slots);
  int fuse = (max_cand <= 16384 && cache_smem <= 96 * 1024) ? 1 : 0;
  int keys_cap = fuse ? max_cand : 0, tbl_cap = 0;
  size_t smem = 0;
  if (fuse) smem = cache_smem > (size_t)keys_cap * 4 ? cache_smem : (size_t)keys_cap * 4;
  {
    // the low-latency continuation: the keys and the whole GPU page table
    // of a set in shared memory
    int max_slots_batch = 0;
    for (int i = 0; i < b.n_req; ++i) max_slots_batch = b.slots[i] > max_slots_batch ? b.slots[i] : max_slots_batch;
    const size_t fs = fast_smem_bytes(max_cand, max_slots_batch, c.dir_part, c.dir_slot, c.dir_page, c.max_parts, c.max_pages, 0);
    if (max_slots_batch <= kFastSlots && max_cand <= 16384 && fs <= 100 * 1024) {
      fuse = 2;
      keys_cap = max_cand;
      smem = fs;
      // page granularity (partition j = page j of the set): if the set's partition tables fit
      // beside the rest without costing a resident CTA, the continuation snapshots them
      int max_parts_batch = 0;
      for (int i = 0; i < b.n_req; ++i) max_parts_batch = b.n_partitions[i] > max_parts_batch ? b.n_partitions[i] : max_parts_batch;
      const size_t ft = fast_smem_bytes(max_cand, max_slots_batch, c.dir_part, c.dir_slot, c.dir_page, c.max_parts, c.max_pages, max_parts_batch);
      if (c.kind != kKindCluster && max_parts_batch > 0 && ft <= 72 * 1024) { tbl_cap = max_parts_batch; smem = ft; }
    }
  }
  const size_t sel_smem = smem;                   // what the selection itself needs
  if (smem < 64 * 1024) smem = 64 * 1024;         // the scoring CTAs' staging area: one summary segment
  // not fused: the cluster kernel behind this one selects; when it also manages the cache it
  // starts set by set, on the flag the last scoring CTA of a set raises (fuse 3)
  int mgr_tbl_cap = 0;
  size_t mgr_smem = 0;
  const int manage = !fuse && plan_cache_fast(c, b, 160 * 1024, &mgr_tbl_cap, &mgr_smem) ? 1 : 0;
  if (manage) fuse = 3;
  // work items: a tail item per set, then every request's segments head by head (segment 0
  // always runs: arrival counter)
  ScoreGrid sg;
  sg.n_sets = n_sets;
  sg.item_prefix[0] = 0;
  for (int i = 0; i < b.n_req; ++i) {
    const int cand = c.kind == kKindToken ? b.n_partitions[i] * kPageTokens : b.n_partitions[i];
    int segs_r = (cand + (1 << c.sum_shift) - 1) >> c.sum_shift;
    if (segs_r < 1) segs_r = 1;
    sg.item_prefix[i + 1] = sg.item_prefix[i] + segs_r * c.Hkv;
  }
  sg.n_items = n_sets + sg.item_prefix[b.n_req];
  // Streaming form: whenever the selection can follow on the sets' flags (one CTA per set with
  // everything in shared memory, or the cluster top-k that also manages the cache).
  // (query groups of up to four heads: a candidate's block sums then fit into its own row)
  const bool stream = (fuse == 2 || fuse == 3) && c.ready && c.G <= 4 && c.resident_scoring == 2;
  if (stream) {
    // shared memory of an SM: this kernel's ring beside ONE more CTA, an attention CTA (64 KiB of
    // pages and its per-warp partials) or a selection CTA (smaller); the selection CTAs, one per
    // set, take some SMs and the first attention CTAs the others.  1 KiB per CTA is the system's.
    const int attn_smem = kChunkPages * kPageBytes + 4 * c.G * (kHeadDim + 2) * 4 + 1024;
    int n_stages = 227 * 1024 - attn_smem - 8 * 1024;
    if (n_stages > 160 * 1024) n_stages = 160 * 1024;
    b.attn_set_major = sg.n_items > 24 * sm_count_of_device() ? 1 : 0;   // a long scoring phase: sets become ready one after the other
    switch (c.G) {
      case 1: launch_stream_g<1>(c, b, q, k_new, v_new, sg, n_stages, st); break;
      case 2: launch_stream_g<2>(c, b, q, k_new, v_new, sg, n_stages, st); break;
      case 4: launch_stream_g<4>(c, b, q, k_new, v_new, sg, n_stages, st); break;
      default: launch_stream_g<4>(c, b, q, k_new, v_new, sg, n_stages, st); break;
    }
    prof_mark(prof, st, kProfScore);
    if (fuse == 2) {
      static size_t configured_dev[kMaxDevices] = {};
      size_t &configured = configured_dev[current_device_slot()];
      if (sel_smem > configured) {
        cudaFuncSetAttribute(k_select, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sel_smem);
        cudaFuncSetAttribute(k_select, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
        configured = sel_smem;
      }
      // one wave at most (the attention grid behind it launches once every CTA here has started):
      // with more sets than SMs a CTA takes several sets, in the order in which they are scored
      const int sel_grid = n_sets < sm_count_of_device() ? n_sets : sm_count_of_device();
      launch_pdl(k_select, dim3(sel_grid), dim3(kScoreThreads), sel_smem, st, 1, c, b, keys_cap, tbl_cap);
      prof_mark(prof, st, kProfTopk);
      return 2;
    }
  }
  // resident form (grid sized in launch_score_g) when scoring is many waves long
  sg.persistent = (!stream && (fuse == 2 || fuse == 3) && c.ready && c.resident_scoring >= 0 &&
                   (c.resident_scoring == 1 || (fuse == 2 && sg.n_items > 12 * sm_count_of_device()))) ? 1 : 0;
  dim3 grid(sg.n_items);
  if (!stream) b.attn_set_major = sg.persistent;
  if (!stream) {
    switch (c.G) {
      case 1: launch_score_g<1>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
      case 2: launch_score_g<2>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
      case 4: launch_score_g<4>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
      default: launch_score_g<8>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
    }
    prof_mark(prof, st, kProfScore);
  }
  if (fuse == 1 || fuse == 2) return 1;
  {
    // cluster size from the largest candidate count: slices of at most 8192 keys stay in smem
    int C = 1;
    while (C < 8 && (max_cand + C - 1) / C > 8192) C *= 2;
    int kc = (((max_cand + C - 1) / C) + 31) & ~31;     // a CTA's slice: whole rows of 32 keys
    if (kc > 16384) kc = 0;                              // too many for shared memory: re-read from L2
    static int smem_set_dev[kMaxDevices] = {};
    int &smem_set = smem_set_dev[current_device_slot()];
    int ksmem = kc * 4;
    // the cache manager runs in the same kernel when it can work on shared-memory copies
    if (manage) ksmem = ((ksmem + 15) & ~15) + (int)mgr_smem;    // the manager's tables sit behind the keys
    if (ksmem > smem_set) { cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, ksmem); smem_set = ksmem; }
    launch_pdl(k_topk, dim3(n_sets * C), dim3(kTopkThreads), (size_t)ksmem, st, C, c, b, kc, manage, mgr_tbl_cap, manage ? (stream ? 2 : 1) : 0);
    prof_mark(prof, st, kProfTopk);
    if (manage) return 2;
  }
  return 2 + launch_cache(c, b, st, prof);
}

}  // namespace spin

#ifdef SPIN_TIMING
extern "C" __attribute__((visibility("default"))) int spin_debug_timestamps_stream(unsigned long long *out) {
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(out, spin::g_dbg_st, sizeof(unsigned long long) * 160 * 64);
}
extern "C" __attribute__((visibility("default"))) int spin_debug_timestamps(unsigned long long *out) {
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(out, spin::g_dbg_ts, sizeof(unsigned long long) * 256 * 32);
}
extern "C" __attribute__((visibility("default"))) int spin_debug_cycles(unsigned long long *out) {
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(out, spin::g_dbg_ck, sizeof(unsigned long long) * 256 * 32);
}
#endif
