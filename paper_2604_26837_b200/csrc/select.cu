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

// Score of one entry for this lane's 8 channels, all G heads; the 16 lanes of the row are
// combined by the caller-visible butterfly.  For min/max summaries max(q*min, q*max) equals
// q * (q >= 0 ? max : min) exactly (min <= max and the products are exact), so the operand is
// picked with one bitwise blend per channel pair on the packed bf16 words (masks precomputed
// per head) instead of two multiplies and a max per channel.
template <int G, bool MINMAX>
__device__ __forceinline__ float score_entry(const uint4 lo, const uint4 hi, const float (&qf)[G][8],
                                             const uint32_t (&qsel)[G][4], uint32_t row_mask) {
  const uint32_t a[4] = {lo.x, lo.y, lo.z, lo.w}, m[4] = {hi.x, hi.y, hi.z, hi.w};
  float v[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float x[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t w = MINMAX ? ((m[j] & qsel[g][j]) | (a[j] & ~qsel[g][j])) : a[j];
      x[2 * j] = __uint_as_float(w << 16);
      x[2 * j + 1] = __uint_as_float(w & 0xffff0000u);
    }
    float s = qf[g][0] * x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) s = fmaf(qf[g][i], x[i], s);     // exact product, one rounding: s + q*x
    v[g] = s;
  }
  // The 16 block sums of every head go up the balanced tree (lanes l and l^1, then l^2, l^4,
  // l^8: both partners form the same sum, addition being commutative).  While more than one
  // head is left in a lane, a level also halves that number: the partners keep one half of
  // the heads each and trade the other, so a level costs n/2 shuffles instead of n.  Lane l
  // of a row ends up with the total of the head whose index is l's low bits reversed.
  const int lane = threadIdx.x & 15;
  int n = G;
#pragma unroll
  for (int level = 0; level < 4; ++level) {
    if (n > 1) {
      const bool up = (lane >> level) & 1;
      const int half = n / 2;
#pragma unroll
      for (int i = 0; i < G / 2; ++i)
        if (i < half) {
          const float send = up ? v[i] : v[i + half], keep = up ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(row_mask, send, 1 << level);
        }
      n = half;
    } else {
      v[0] = v[0] + __shfl_xor_sync(row_mask, v[0], 1 << level);
    }
  }
  // heads in ascending order, into the row's first lane
  float tot = v[0];
#pragma unroll
  for (int h = 1; h < G; ++h) {
    constexpr int kBits = G == 8 ? 3 : G == 4 ? 2 : 1;
    int src = 0;
#pragma unroll
    for (int bit = 0; bit < kBits; ++bit) src |= ((h >> bit) & 1) << (kBits - 1 - bit);
    tot = tot + __shfl_sync(row_mask, v[0], src, 16);
  }
  return tot + 0.0f;                              // -0.0 -> +0.0
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

  float qf[G][8];
  uint32_t qsel[G][4];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const uint4 raw = *reinterpret_cast<const uint4 *>(
        q + ((size_t)i_req * c.Hq + head * G + g) * kHeadDim + lane16 * 8);
    unpack8(raw, qf[g]);
#pragma unroll
    for (int j = 0; j < 4; ++j)
      qsel[g][j] = (qf[g][2 * j] >= 0.f ? 0x0000ffffu : 0u) | (qf[g][2 * j + 1] >= 0.f ? 0xffff0000u : 0u);
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
#pragma unroll
    for (int j = 0; j < kPerGroup; ++j) {
      const int slot = gI * kPerGroup + j, e = grp + 16 * slot;
      if (e < n_here && !dead) {
        const uint4 a0 = *reinterpret_cast<const uint4 *>(stage + (size_t)e * kEntry);
        const uint4 m0 = MINMAX ? *reinterpret_cast<const uint4 *>(stage + (size_t)e * kEntry + kRowBytes)
                                : make_uint4(0, 0, 0, 0);

        const float s0 = score_entry<G, MINMAX>(a0, m0, qf, qsel, row_mask);
        if (lane16 == 0) out[e] = s0;
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

// Stand-alone top-k: one thread-block cluster per set (slices of the keys in shared memory).
// With wait_flags a cluster starts as soon as its own set is scored (the flag the scoring
// kernel's last CTA of that set raises) instead of when the whole scoring kernel is done; the
// outcome of the bounded wait is shared through the first CTA so that all CTAs of the
// cluster take the same path through the cluster barriers.
__device__ __forceinline__ void topk_cta(const DevCtx &c, const Batch &bt, int keys_cap, int manage, int tbl_cap,
                                         int wait_flags, uint8_t *dyn_smem) {
  __shared__ union { TopkShared t; FastShared f; } shm;
  __shared__ int s_ok;
  TopkShared &tsh = shm.t;
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int b = blockIdx.x / C, i_req = b / c.Hkv, head = b % c.Hkv, tid = threadIdx.x;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  if (wait_flags) {
    if (rank == 0 && tid == 0) s_ok = flag_wait(c, c.scored + b, bt.epoch);
    cluster.sync();
    const int ok = *cluster.map_shared_rank(&s_ok, 0);
    cluster.sync();                                   // the first CTA's word is not read after this
    if (!ok) return;
  } else {
    pdl_wait_prev();
  }
  if (rank == 0) dbg_ts(b, 9);
  // the first CTA is also the set's cache manager: its tables start towards shared memory now
  // (behind the keys' slice) and arrive while the select runs
  const int S = bt.slots[i_req];
  const FastLayout L = fast_layout(c, dyn_smem + (((size_t)keys_cap * 4 + 15) & ~(size_t)15), 0, S, tbl_cap);
  const bool mgr = manage && rank == 0;
  if (mgr) {
    fast_prefetch_dirs<kTopkThreads>(c, L, set, S);
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
    __syncthreads();
    fast_prefetch_gpt<kTopkThreads>(c, L, S);
    fast_prefetch_tables<kTopkThreads>(c, L, bt.n_partitions[i_req]);
  }
  const bool first = topk_stage<kTopkThreads, true>(c, b, bt.n_partitions[i_req], reinterpret_cast<uint32_t *>(dyn_smem), keys_cap, tsh);
  if (!first || !manage) return;
  const int np = c.n_parts[b];
  const int32_t *g_parts = c.parts + (size_t)b * c.max_parts;
  for (int r = tid; r < np; r += kTopkThreads) L.s_parts[r] = g_parts[r];
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  __syncthreads();
  cache_fast<kTopkThreads>(c, bt, b, i_req, set, L, np, shm.f);
}

__global__ void __launch_bounds__(kTopkThreads)
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
  // resident form (grid sized in launch_score_g) when scoring is many waves long
  sg.persistent = (fuse == 2 && c.ready && c.resident_scoring >= 0 &&
                   (c.resident_scoring > 0 || sg.n_items > 12 * sm_count_of_device())) ? 1 : 0;
  dim3 grid(sg.n_items);
  b.attn_set_major = sg.persistent;
  switch (c.G) {
    case 1: launch_score_g<1>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
    case 2: launch_score_g<2>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
    case 4: launch_score_g<4>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
    default: launch_score_g<8>(c, b, q, k_new, v_new, grid, smem, fuse, keys_cap, tbl_cap, sg, st); break;
  }
  prof_mark(prof, st, kProfScore);
  if (fuse == 1 || fuse == 2) return 1;
  {
    // cluster size from the largest candidate count: slices of at most 8192 keys stay in smem
    int C = 1;
    while (C < 8 && (max_cand + C - 1) / C > 8192) C *= 2;
    int kc = (max_cand + C - 1) / C;
    if (kc > 16384) kc = 0;                              // too many for shared memory: re-read from L2
    static int smem_set_dev[kMaxDevices] = {};
    int &smem_set = smem_set_dev[current_device_slot()];
    int ksmem = kc * 4;
    // the cache manager runs in the same kernel when it can work on shared-memory copies
    if (manage) ksmem = ((ksmem + 15) & ~15) + (int)mgr_smem;    // the manager's tables sit behind the keys
    if (ksmem > smem_set) { cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, ksmem); smem_set = ksmem; }
    launch_pdl(k_topk, dim3(n_sets * C), dim3(kTopkThreads), (size_t)ksmem, st, C, c, b, kc, manage, mgr_tbl_cap, manage);
    prof_mark(prof, st, kProfTopk);
    if (manage) return 2;
  }
  return 2 + launch_cache(c, b, st, prof);
}

}  // namespace spin

#ifdef SPIN_TIMING
extern "C" __attribute__((visibility("default"))) int spin_debug_timestamps(unsigned long long *out) {
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(out, spin::g_dbg_ts, sizeof(unsigned long long) * 256 * 32);
}
#endif
