// The two per-set stages between scoring and attention, written as device functions so that
// they can run either as kernels of their own (token-granular selection over 64K+ keys uses a
// thread-block cluster per set for top-k) or as the continuation of the scoring kernel: the
// last scoring CTA of a set to finish goes straight on with that set's top-k and cache
// management while the other sets are still being scored.
//
//   topk_stage  -- Select's "-> topk" (Table 1): k best candidates, ties to the lower index,
//                  emitted ascending; token-granular selections are folded into pages + masks.
//   cache_stage -- Retrieve steps 1-3 (Section 5.2) and bucketed LRU steps 1-4 (Section 5.3):
//                  metadata only; the page bytes move in the attention kernel (or k_fetch).
#pragma once
#include <cooperative_groups.h>
#include <cstddef>

#include "spin_dev.cuh"

namespace spin {

namespace cg = cooperative_groups;

enum : int { kHit = 0, kAdmit = 1, kBypass = 2 };

__device__ __forceinline__ uint32_t order_key(float s) {
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Exclusive prefix of v over the block (thread order) and the block total.  wsum: 33 words.
template <int T>
__device__ __forceinline__ uint32_t block_scan(uint32_t v, uint32_t *wsum, uint32_t *total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) wsum[w] = inc;
  __syncthreads();
  if (w == 0) {
    uint32_t x = lane < T / 32 ? wsum[lane] : 0, xi = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t t = __shfl_up_sync(0xffffffffu, xi, o);
      if (lane >= o) xi += t;
    }
    wsum[lane] = xi - x;                         // exclusive warp offsets
    if (lane == 31) wsum[32] = xi;               // total
  }
  __syncthreads();
  const uint32_t res = wsum[w] + inc - v;
  *total = wsum[32];
  __syncthreads();                               // wsum is reused by the next call
  return res;
}

// The same with a single barrier: every thread adds up the warp totals itself.  wsum: T/32
// words that no thread still reads from an earlier call (callers alternate two buffers).
template <int T>
__device__ __forceinline__ uint32_t block_scan1(uint32_t v, uint32_t *wsum, uint32_t *total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) wsum[w] = inc;
  __syncthreads();
  uint32_t base = 0, tot = 0;
#pragma unroll
  for (int j = 0; j < T / 32; ++j) {
    const uint32_t x = wsum[j];
    base += j < w ? x : 0u;
    tot += x;
  }
  *total = tot;
  return base + inc - v;
}

// index of `p` in the ascending array a[0..n), or -1
__device__ __forceinline__ int find_sorted(const int32_t *a, int n, int p) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (a[mid] < p) lo = mid + 1; else hi = mid;
  }
  return (lo < n && a[lo] == p) ? lo : -1;
}
// largest r with off[r] <= idx (off ascending, off[0] == 0)
__device__ __forceinline__ int owner_of(const int32_t *off, int n, int idx) {
  int lo = 0, hi = n;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (off[mid] <= idx) lo = mid; else hi = mid;
  }
  return lo;
}

// The cache manager resolves the CPU page ids of missed pages itself when the copy kernel needs
// them (fetch_mode 1) or when they are one HBM read away (mirror); when they are only in pinned
// host memory and the fetch is fused into attention, the fetching warp looks them up instead,
// so that a set's page list never waits on the host link.
__device__ __forceinline__ bool resolve_in_manager(const DevCtx &c) { return c.fetch_mode != 0 || c.cpt_mirror != nullptr; }

#ifdef SPIN_TIMING
__device__ unsigned long long g_dbg_ts[256][32];
__device__ __forceinline__ void dbg_ts(int b, int slot) { if (threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); g_dbg_ts[b & 255][slot] = t; } }
__device__ __forceinline__ void dbg_ts_any(int b, int slot) { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); g_dbg_ts[b & 255][slot] = t; }
// cycle stamps of one CTA (differences within a CTA only)
__device__ unsigned long long g_dbg_ck[256][32];
__device__ __forceinline__ void dbg_ck(int b, int slot) { if (threadIdx.x == 0) g_dbg_ck[b & 255][slot] = (unsigned long long)clock64(); }
#else
__device__ __forceinline__ void dbg_ts(int, int) {}
__device__ __forceinline__ void dbg_ts_any(int, int) {}
__device__ __forceinline__ void dbg_ck(int, int) {}
#endif

// The row loops of the cluster select, unrolled just enough for the shared-memory reads of
// consecutive rows to overlap (1 -> 4: 19.3 -> 16.6 us for 65552 keys; fully unrolled the
// code's first-time instruction fetch costs more than the loops save).
constexpr int kRowUnroll = 4;
constexpr int kWideBits = 11, kWideBins = 1 << kWideBits;   // digit of the row-wise cluster select
constexpr int kGatherMax = 256;                             // a threshold bin this small is ranked directly

struct TopkShared {
  uint32_t hist[256];          // this CTA's histogram (read remotely inside a cluster)
  uint32_t ghist[256];         // histogram over the whole set
  uint32_t wsum[33];
  uint32_t cnt[2];             // this CTA's (above threshold, equal) counts
  uint32_t prefix, remaining;
  uint32_t orand[2];           // OR and AND of this CTA's keys (read remotely inside a cluster)
};

// Shared memory of the row-wise cluster select (topk_cluster_rows); only the cluster kernel holds it.
struct TopkRowsShared {
  alignas(16) uint32_t whist[2][kWideBins];    // this CTA's wide-digit histograms, alternating between passes (read
                                               //   remotely, four bins at a time: 16-byte aligned)
  uint32_t cand[kGatherMax];       // this CTA's keys of the threshold bin (read remotely)
  uint32_t gath[kGatherMax];       // the threshold bin's keys of all CTAs
  uint32_t ncand, bin_count;
  uint32_t result[2];              // threshold key and how many keys equal to it are taken
  uint32_t wcnt[32], wpg[32];      // per-warp (above | equal << 16) counts and page counts
  uint32_t rcnt[8], rpages[8];     // the same per CTA of the cluster (written by their owners)
  uint32_t wsum[33];
  uint32_t prefix, remaining;
};

static_assert(offsetof(TopkRowsShared, whist) % 16 == 0 && sizeof(uint32_t[kWideBins]) % 16 == 0, "uint4 reads of the histograms");

template <bool CLUSTER> __device__ __forceinline__ void stage_sync() {
  if constexpr (CLUSTER) cg::this_cluster().sync(); else __syncthreads();
}

// Radix select of one set by a thread-block cluster.  A CTA owns a slice of `per` consecutive
// candidates (a multiple of 32) whose keys it holds in shared memory; a warp owns R x 32
// consecutive candidates of it as R rows of 32 (lane l: candidate 32 j + l of the warp's run).
// Loads are coalesced, a row's ballot is the order of its 32 candidates (for token granularity
// also the masks of the row's two pages), so that the ordered compaction needs no scan over
// candidates and no second look at memory.
// Every pass over the keys is a ROLLED loop over rows: this code runs once per launch with cold
// instruction caches, where a straight-line instruction costs tens of cycles of fetch, so the
// number of distinct instructions on the path matters more than the work per key.
// Digits are the key's bits 31..21, 20..10 and 10..0.  A CTA's histogram is read by all CTAs of
// the cluster through distributed shared memory (each finds the threshold bin itself: no
// broadcast, one cluster barrier per pass, the histograms alternating between two buffers); a
// threshold bin of at most 256 keys is gathered by every CTA from all CTAs and ranked directly.
// Counts that other CTAs need are pushed into their shared memory before a barrier, so nothing
// is read remotely after the last one.  Cluster barriers are hardware barriers and every CTA
// executes the same sequence of them (every decision is taken on set-wide values).
// Leaves the chosen candidates, ascending, in c.sel_ids and the partitions of the cache manager
// in c.parts / c.part_mask / c.n_parts; the caller's closing cluster barrier publishes them.
// Needs per <= 2048 T (a warp's rows are numbered by its lanes, two rows each) and per keys of shared memory.
template <int T>
__device__ __forceinline__ void topk_cluster_rows(const DevCtx &c, int b, int n, int k, int per, uint32_t *s_keys,
                                                  TopkRowsShared &sh, bool xfer) {
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt = (1u << lane) - 1u;
  constexpr int W = T / 32;
  float *scores = c.scores + (size_t)b * c.max_cand;
  int32_t *sel = c.sel_ids + (size_t)b * c.max_sel;
  int32_t *parts = c.parts + (size_t)b * c.max_parts;
  const bool token = c.kind == kKindToken;
  const int lo = min(n, rank * per), m = min(n, lo + per) - lo;
  const int R = (per / 32 + W - 1) / W;                                // rows of a warp (at most 64)
  const int wbase = warp * R * 32;                                     // the warp's run starts here in the slice
  const int nvr = max(0, min(R, (m - wbase - lane + 31) >> 5));        // rows j < nvr hold a candidate of this lane
  uint32_t *mykeys = s_keys + wbase + lane;                            // row j: mykeys[32 j]
  if (rank == 0) dbg_ck(b, 0);
  if (xfer) {
    float *xfer_in = c.score_xfer + (size_t)b * c.max_cand + lo + wbase + lane;
#pragma unroll 1
    for (int j = 0; j < nvr; ++j) {
      const float sc = take_score(c, xfer_in + 32 * j);
      scores[lo + wbase + lane + 32 * j] = sc;
      mykeys[32 * j] = order_key(sc);
    }
  } else {
    // asynchronous copies: all rows in flight at once from a two-instruction loop
    const float *src = scores + lo + wbase + lane;
    const uint32_t dst = (uint32_t)__cvta_generic_to_shared(mykeys);
#pragma unroll 1
    for (int j = 0; j < nvr; ++j)
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(dst + 128u * j), "l"(src + 32 * j) : "memory");
    asm volatile("cp.async.commit_group;\n" ::: "memory");
  }
#pragma unroll 1
  for (int i = tid; i < 2 * kWideBins; i += T) (&sh.whist[0][0])[i] = 0;
  if (tid == 0) {
    sh.ncand = 0;
    if (rank == 0) {
      c.n_sel[b] = k;
      atomicAdd(&c.counters->candidates_scored, (unsigned long long)n);
    }
  }
  if (!xfer) {
    asm volatile("cp.async.wait_group 0;\n" ::: "memory");
#pragma unroll kRowUnroll
    for (int j = 0; j < nvr; ++j) mykeys[32 * j] = order_key(__uint_as_float(mykeys[32 * j]));   // a thread's own words
  }
  __syncthreads();
  if (rank == 0) { dbg_ts(b, 10); dbg_ck(b, 1); }
  uint32_t thr = 0, need_eq = (uint32_t)k;
  {
    uint32_t mask = 0, prefix = 0, remaining = (uint32_t)k;              // decided bits and their value
    int buf = 0;
    constexpr int kPer = kWideBins / T;                                // bins per thread
    constexpr uint32_t dmask = kWideBins - 1;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {
      const int shift = pass == 0 ? 21 : pass == 1 ? 10 : 0;           // the last digit repeats bit 10 (decided: harmless)
      uint32_t *hist = sh.whist[buf];
      if (pass == 2) {
        // this buffer served two passes ago; every CTA has read it since (the barrier of the pass between)
#pragma unroll 1
        for (int i = tid; i < kWideBins; i += T) hist[i] = 0;
        __syncthreads();
      }
#pragma unroll kRowUnroll
      for (int j = 0; j < nvr; ++j) {
        const uint32_t key = mykeys[32 * j];
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & dmask], 1u);
      }
      if (rank == 0) dbg_ck(b, 2 + 6 * pass);
      cluster.sync();                                                  // every CTA's histogram of this pass is complete
      if (rank == 0) { dbg_ts(b, 11 + pass); dbg_ck(b, 3 + 6 * pass); }
      // this thread's kPer bins over the whole set, best first: 16-byte reads, one batch of the
      // cluster's CTAs at a time, all reads of a batch issued before the first is used (a CTA
      // beyond the cluster's size stands for the last one and counts for nothing)
      uint32_t loc[kPer], sum = 0;
      static_assert(kPer % 4 == 0 && kPer <= 8, "a thread reads its bins of one CTA as one or two uint4");
      {
        uint32_t bins[kPer];                                           // ascending
#pragma unroll
        for (int q = 0; q < kPer / 4; ++q) {
          uint4 part[8];
#pragma unroll
          for (int r = 0; r < 8; ++r)
            part[r] = *reinterpret_cast<const uint4 *>(cluster.map_shared_rank(hist, min(r, C - 1)) + (kWideBins - kPer * (tid + 1)) + 4 * q);
          uint4 acc = make_uint4(0, 0, 0, 0);
#pragma unroll
          for (int r = 0; r < 8; ++r)
            if (r < C) { acc.x += part[r].x; acc.y += part[r].y; acc.z += part[r].z; acc.w += part[r].w; }
          bins[4 * q] = acc.x; bins[4 * q + 1] = acc.y; bins[4 * q + 2] = acc.z; bins[4 * q + 3] = acc.w;
        }
#pragma unroll
        for (int j = 0; j < kPer; ++j) { loc[j] = bins[kPer - 1 - j]; sum += loc[j]; }
      }
      if (rank == 0) dbg_ck(b, 4 + 6 * pass);
      uint32_t tot_all;
      const uint32_t before = block_scan1<T>(sum, sh.wsum + (pass & 1) * 16, &tot_all);
      if (rank == 0) dbg_ck(b, 5 + 6 * pass);
      if (before < remaining && before + sum >= remaining) {
        uint32_t cum = before;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
          if (cum < remaining && cum + loc[j] >= remaining) {
            sh.prefix = (prefix & ~(dmask << shift)) | ((uint32_t)(kWideBins - 1 - kPer * tid - j) << shift);
            sh.remaining = remaining - cum;
            sh.bin_count = loc[j];
          }
          cum += loc[j];
        }
      }
      __syncthreads();
      prefix = sh.prefix;
      remaining = sh.remaining;
      const uint32_t bin_count = sh.bin_count;
      mask |= dmask << shift;
      __syncthreads();                                                 // sh.prefix etc. are rewritten by the next pass
      if (rank == 0) dbg_ck(b, 6 + 6 * pass);
      if (shift == 0) break;                                           // the key is decided to its last bit
      if (bin_count <= (uint32_t)kGatherMax) {
        // the bin's keys of this CTA, then those of all CTAs, ranked by one thread per key
#pragma unroll kRowUnroll
        for (int j = 0; j < nvr; ++j) {
          const uint32_t key = mykeys[32 * j];
          if ((key & mask) == prefix) sh.cand[atomicAdd(&sh.ncand, 1u) & (kGatherMax - 1)] = key;
        }
        if (rank == 0) dbg_ck(b, 20);
        cluster.sync();
        if (rank == 0) dbg_ck(b, 21);
        if (tid < kGatherMax) {
          uint32_t cnt[8], val[8];
#pragma unroll
          for (int r = 0; r < 8; ++r) cnt[r] = *cluster.map_shared_rank(&sh.ncand, min(r, C - 1));
#pragma unroll
          for (int r = 0; r < 8; ++r) {
            val[r] = 0;
            if (r < C && tid < (int)cnt[r]) val[r] = cluster.map_shared_rank(sh.cand, r)[tid];
          }
          uint32_t off = 0;
#pragma unroll
          for (int r = 0; r < 8; ++r)
            if (r < C) {
              if (tid < (int)cnt[r]) sh.gath[(off + tid) & (kGatherMax - 1)] = val[r];
              off += cnt[r];
            }
        }
        __syncthreads();
        if (rank == 0) dbg_ck(b, 22);
        if (tid < (int)bin_count) {
          const uint32_t mine = sh.gath[tid];
          uint32_t gt = 0, ge = 0;
#pragma unroll 1
          for (uint32_t j = 0; j < bin_count; ++j) { const uint32_t o = sh.gath[j]; gt += o > mine; ge += o >= mine; }
          if (gt < remaining && ge >= remaining) { sh.result[0] = mine; sh.result[1] = remaining - gt; }
        }
        __syncthreads();
        if (rank == 0) dbg_ck(b, 23);
        prefix = sh.result[0];
        remaining = sh.result[1];
        break;
      }
      buf ^= 1;
    }
    thr = prefix;
    need_eq = remaining;
  }
  if (rank == 0) dbg_ts(b, 15);
  // ---- ordered compaction: everything above thr, plus the first need_eq keys equal to it ----
  // counts of this warp (row ballots), of the warps before it, of the CTAs before this one
  uint32_t wgt = 0, weq = 0;
#pragma unroll kRowUnroll
  for (int j = 0; j < R; ++j) {
    const uint32_t key = j < nvr ? mykeys[32 * j] : 0u;
    wgt += __popc(__ballot_sync(0xffffffffu, j < nvr && key > thr));
    weq += __popc(__ballot_sync(0xffffffffu, j < nvr && key == thr));
  }
  if (lane == 0) sh.wcnt[warp] = wgt | (weq << 16);                    // a slice holds fewer than 65536 candidates
  __syncthreads();
  uint32_t gt_base = 0, eq_base = 0;
  {
    uint32_t before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const uint32_t v = sh.wcnt[w];
      before += w < warp ? v : 0u;
      total += v;
    }
    if (tid < C) cluster.map_shared_rank(sh.rcnt, tid)[rank] = total;  // pushed: read locally after the barrier
    if (rank == 0) dbg_ck(b, 24);
    cluster.sync();
    if (rank == 0) dbg_ck(b, 25);
    gt_base = before & 0xffffu;
    eq_base = before >> 16;
    for (int r = 0; r < rank; ++r) { const uint32_t v = sh.rcnt[r]; gt_base += v & 0xffffu; eq_base += v >> 16; }
  }
  uint32_t row_taken[2] = {0, 0};                                      // lane l: which candidates of rows l and 32 + l were chosen
  int32_t *dst2 = token ? sel : parts;                                 // without tokens the partitions are the selection
#pragma unroll kRowUnroll
  for (int j = 0; j < R; ++j) {
    const uint32_t key = j < nvr ? mykeys[32 * j] : 0u;
    const bool g = j < nvr && key > thr, e = j < nvr && key == thr;
    const uint32_t bg = __ballot_sync(0xffffffffu, g), be = __ballot_sync(0xffffffffu, e);
    const uint32_t eq_b = eq_base + __popc(be & lt);
    const bool take = g || (e && eq_b < need_eq);
    if (take) {
      const uint32_t pos = gt_base + __popc(bg & lt) + min(eq_b, need_eq);
      const int id = lo + wbase + 32 * j + lane;
      sel[pos] = id;
      dst2[pos] = id;
    }
    const uint32_t bt = __ballot_sync(0xffffffffu, take);
    if (lane == (j & 31)) { if (j < 32) row_taken[0] = bt; else row_taken[1] = bt; }
    gt_base += __popc(bg);
    eq_base += __popc(be);
  }
  if (rank == 0) dbg_ck(b, 26);
  if (!token) {
    if (rank == 0 && tid == 0) c.n_parts[b] = k;
    return;
  }
  // ---- chosen tokens -> their pages (ascending, unique) and a 16-bit token mask per page.
  // A row is two pages: lane l numbers the pages of rows l and 32 + l.
  uint32_t *pmask = c.part_mask + (size_t)b * c.max_parts;
  uint32_t mine[2], inc[2], half_total[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    mine[h] = ((row_taken[h] & 0xffffu) != 0) + ((row_taken[h] >> 16) != 0);
    inc[h] = mine[h];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, inc[h], o);
      if (lane >= o) inc[h] += t;
    }
    half_total[h] = __shfl_sync(0xffffffffu, inc[h], 31);
  }
  if (lane == 0) sh.wpg[warp] = half_total[0] + half_total[1];
  __syncthreads();
  uint32_t pg_base = 0, pg_total = 0;
#pragma unroll
  for (int w = 0; w < W; ++w) {
    const uint32_t v = sh.wpg[w];
    pg_base += w < warp ? v : 0u;
    pg_total += v;
  }
  if (tid < C) cluster.map_shared_rank(sh.rpages, tid)[rank] = pg_total;
  if (rank == 0) dbg_ck(b, 27);
  cluster.sync();
  if (rank == 0) dbg_ck(b, 28);
  uint32_t cta_base = 0;
  for (int r = 0; r < rank; ++r) cta_base += sh.rpages[r];
#pragma unroll
  for (int h = 0; h < 2; ++h)
    if (mine[h]) {
      uint32_t at = cta_base + pg_base + (h ? half_total[0] : 0u) + inc[h] - mine[h];
      const int page = (lo + wbase + 32 * (lane + 32 * h)) >> 4;
      const uint32_t m_lo = row_taken[h] & 0xffffu, m_hi = row_taken[h] >> 16;
      if (m_lo) { parts[at] = page; pmask[at] = m_lo; ++at; }
      if (m_hi) { parts[at] = page + 1; pmask[at] = m_hi; }
    }
  if (rank == C - 1 && tid == 0) c.n_parts[b] = (int)(cta_base + pg_total);
  if (rank == 0) dbg_ck(b, 29);
}

// Top-k of one set.  With CLUSTER the set's candidates are cut into one contiguous slice per
// CTA of the cluster (keys kept in shared memory), every radix pass builds per-CTA histograms
// that all CTAs sum through distributed shared memory, and the ordered compaction starts at
// the lower-ranked CTAs' counts.  Cluster barriers are hardware barriers (nothing spins on a
// flag) and every CTA of a cluster executes the same number of them.  Without CLUSTER the
// calling CTA owns the whole set.  On return (all threads of rank 0) the partitions handed to
// the cache manager are in c.parts / c.n_parts; other ranks return false and must exit.
// xfer: the scores come from the streaming kernel's hand-over buffer (taken out into c.scores on the way)
template <int T, bool CLUSTER>
__device__ __forceinline__ bool topk_stage(const DevCtx &c, int b, int n_partitions, uint32_t *s_keys,
                                           int keys_cap, TopkShared &sh, bool xfer = false, TopkRowsShared *rows = nullptr) {
  int C = 1, rank = 0;
  if constexpr (CLUSTER) {
    cg::cluster_group cluster = cg::this_cluster();
    C = (int)cluster.num_blocks();
    rank = (int)cluster.block_rank();
  }
  const int tid = threadIdx.x;
  const int n = c.kind == kKindToken ? n_partitions * kPageTokens : n_partitions;
  const int k = min(c.topk, n);
  float *scores = c.scores + (size_t)b * c.max_cand;
  float *xfer_in = c.score_xfer + (size_t)b * c.max_cand;
  int32_t *sel = c.sel_ids + (size_t)b * c.max_sel;
  const int per = (n + C - 1) / C;
  const int lo = min(n, rank * per), m = min(n, lo + per) - lo;
  const bool cached = m <= keys_cap;

  bool selected = false;
  if constexpr (CLUSTER) {
    // slices that fit in shared memory, at most 64 rows per warp: the row-wise select
    const int per32 = (per + 31) & ~31;
    if (rows != nullptr && k < n && per32 <= 64 * T && per32 <= keys_cap) {
      if (rank == 0) dbg_ts(b, 25);
      topk_cluster_rows<T>(c, b, n, k, per32, s_keys, *rows, xfer);
      selected = true;
    }
  }
  if (!selected) {
  if (tid == 0 && rank == 0) {
    c.n_sel[b] = k;
    atomicAdd(&c.counters->candidates_scored, (unsigned long long)n);
  }
  if (tid == 0) { sh.orand[0] = 0u; sh.orand[1] = 0xffffffffu; }
  __syncthreads();
  // keys -> shared memory, with the OR and AND of the slice taken on the way
  {
    uint32_t k_or = 0, k_and = 0xffffffffu;
    if (xfer) {
#pragma unroll 4
      for (int i = tid; i < m; i += T) {
        const float sc = take_score(c, xfer_in + lo + i);
        scores[lo + i] = sc;
        const uint32_t key = order_key(sc);
        if (cached) s_keys[i] = key;
        k_or |= key; k_and &= key;
      }
    } else {
#pragma unroll 8
      for (int i = tid; i < m; i += T) {
        const uint32_t key = order_key(__ldcg(scores + lo + i));
        if (cached) s_keys[i] = key;
        k_or |= key; k_and &= key;
      }
    }
    k_or = __reduce_or_sync(0xffffffffu, k_or);
    k_and = __reduce_and_sync(0xffffffffu, k_and);
    if ((tid & 31) == 0) { atomicOr(&sh.orand[0], k_or); atomicAnd(&sh.orand[1], k_and); }
  }
  stage_sync<CLUSTER>();
  if (rank == 0) dbg_ts(b, 25);
  auto key_at = [&](int i) { return cached ? s_keys[i] : order_key(__ldcg(scores + lo + i)); };

  if (k == n) {
    for (int i = tid; i < m; i += T) sel[lo + i] = lo + i;
  } else {
    // ---- radix select: key of the k-th best candidate --------------------------------
    // The scores of one set share their sign, exponent and often some mantissa bits; a digit
    // taken there would put every key into one bin (and serialise on its counter).  The bits
    // on which all keys agree (OR == AND over the set) are decided from the start and the
    // first 8-bit digit begins at the highest bit that differs.
    uint32_t a_or = 0, a_and = 0xffffffffu;
    if constexpr (CLUSTER) {
      cg::cluster_group cluster = cg::this_cluster();
      for (int r = 0; r < C; ++r) {
        const uint32_t *ro = cluster.map_shared_rank(sh.orand, r);
        a_or |= ro[0]; a_and &= ro[1];
      }
    } else { a_or = sh.orand[0]; a_and = sh.orand[1]; }
    const uint32_t differ = a_or ^ a_and;
    int topbit = differ ? 31 - __clz(differ) : -1;                 // -1: all keys are equal
    uint32_t mask = topbit >= 31 ? 0u : ~((2u << max(topbit, 0)) - 1u);
    if (topbit < 0) mask = 0xffffffffu;
    uint32_t prefix = a_and & mask, remaining = k;
    for (; topbit >= 0;) {
      const int shift = max(0, topbit + 1 - 8), width = topbit + 1 - shift;
      const uint32_t dmask = (1u << width) - 1u;
      if (tid < 256) sh.hist[tid] = 0;
      __syncthreads();
      for (int i = tid; i < m; i += T) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) atomicAdd(&sh.hist[(key >> shift) & dmask], 1u);
      }
      stage_sync<CLUSTER>();                          // every CTA's histogram is complete
      for (int bin = tid; bin < 256; bin += T) {
        uint32_t tot = 0;
        if constexpr (CLUSTER) {
          cg::cluster_group cluster = cg::this_cluster();
#pragma unroll
          for (int r = 0; r < 8; ++r) tot += r < C ? cluster.map_shared_rank(sh.hist, r)[bin] : 0u;   // loads issued together
        } else {
          tot = sh.hist[bin];
        }
        sh.ghist[bin] = tot;
      }
      stage_sync<CLUSTER>();                          // remote reads done before hist is reused
      if (tid < 32) {
        // lane l owns bins 255-8l .. 248-8l (descending); find where the count from the
        // top reaches `remaining`
        uint32_t loc[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { loc[j] = sh.ghist[255 - 8 * tid - j]; sum += loc[j]; }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
          if (tid >= o) inc += t;
        }
        const uint32_t before = inc - sum;
        if (before < remaining && inc >= remaining) {
          uint32_t cum = before;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (cum < remaining && cum + loc[j] >= remaining) {
              sh.prefix = prefix | ((uint32_t)(255 - 8 * tid - j) << shift);
              sh.remaining = remaining - cum;
            }
            cum += loc[j];
          }
        }
      }
      __syncthreads();
      prefix = sh.prefix;
      remaining = sh.remaining;
      mask |= dmask << shift;
      topbit = shift - 1;
    }
    const uint32_t thr = prefix, need_eq = remaining;
    if (rank == 0) dbg_ts(b, 26);
    // ---- counts of this slice, offsets from the lower-ranked slices ---------------------
    uint32_t run_gt = 0, run_eq = 0;
    if constexpr (CLUSTER) {
      if (tid < 2) sh.cnt[tid] = 0;
      __syncthreads();
      uint32_t gt = 0, eq = 0;
      for (int i = tid; i < m; i += T) {
        const uint32_t key = key_at(i);
        gt += key > thr;
        eq += key == thr;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, o);
        eq += __shfl_xor_sync(0xffffffffu, eq, o);
      }
      if ((tid & 31) == 0) { atomicAdd(&sh.cnt[0], gt); atomicAdd(&sh.cnt[1], eq); }
      cg::cluster_group cluster = cg::this_cluster();
      cluster.sync();
      for (int r = 0; r < rank; ++r) {
        const uint32_t *rc = cluster.map_shared_rank(sh.cnt, r);
        run_gt += rc[0];
        run_eq += rc[1];
      }
    }
    // ---- ordered compaction: everything above thr, plus the first need_eq equal to it --
    if (m <= 60000) {
      // every thread owns a contiguous run of the slice: one block scan in all
      const int E = (m + T - 1) / T, r0 = min(m, tid * E), r1 = min(m, r0 + E);
      uint32_t gt = 0, eq = 0;
      for (int i = r0; i < r1; ++i) { const uint32_t key = key_at(i); gt += key > thr; eq += key == thr; }
      uint32_t total;
      const uint32_t ex = block_scan<T>(gt | (eq << 16), sh.wsum, &total);
      uint32_t gt_before = run_gt + (ex & 0xffffu), eq_before = run_eq + (ex >> 16);
      for (int i = r0; i < r1; ++i) {
        const uint32_t key = key_at(i);
        if (key > thr || (key == thr && eq_before < need_eq)) sel[gt_before + min(eq_before, need_eq)] = lo + i;
        gt_before += key > thr;
        eq_before += key == thr;
      }
    } else {
      for (int base = 0; base < m; base += T) {
        const int i = base + tid;
        uint32_t gt = 0, eq = 0;
        if (i < m) {
          const uint32_t key = key_at(i);
          gt = key > thr;
          eq = key == thr;
        }
        uint32_t total;
        const uint32_t ex = block_scan<T>(gt | (eq << 16), sh.wsum, &total);
        const uint32_t gt_before = run_gt + (ex & 0xffffu), eq_before = run_eq + (ex >> 16);
        if (gt || (eq && eq_before < need_eq))
          sel[gt_before + min(eq_before, need_eq)] = lo + i;
        run_gt += total & 0xffffu;
        run_eq += total >> 16;
      }
    }
  }
  }
  if (rank == 0) dbg_ts(b, 27);
  stage_sync<CLUSTER>();     // selections of all slices are written; no remote smem is read after this
  if (rank != 0) return false;
  dbg_ts(b, 28);
  if (selected) { dbg_ts(b, 29); return true; }      // the row-wise select wrote the partitions itself

  // ---- candidates -> partitions of the cache manager (first CTA of the cluster) ----------
  int32_t *parts = c.parts + (size_t)b * c.max_parts;
  if (c.kind != kKindToken) {
    for (int i = tid; i < k; i += T) parts[i] = __ldcg(sel + i);
    if (tid == 0) c.n_parts[b] = k;
    __syncthreads();
    return true;
  }
  // chosen tokens (ascending) -> their pages (ascending, unique) + a 16-bit token mask per page.
  // Every thread owns a contiguous run of the selection: one block scan numbers the pages.
  uint32_t *pmask = c.part_mask + (size_t)b * c.max_parts;
  for (int i = tid; i < k; i += T) pmask[i] = 0;
  const int E = (k + T - 1) / T, r0 = min(k, tid * E), r1 = min(k, r0 + E);
  const int page_before = r0 > 0 && r0 < k ? (__ldcg(sel + r0 - 1) >> 4) : -1;
  uint32_t firsts = 0;
  {
    int pp = page_before;
    for (int i = r0; i < r1; ++i) { const int pg = __ldcg(sel + i) >> 4; firsts += pg != pp; pp = pg; }
  }
  uint32_t run;
  const uint32_t ex = block_scan<T>(firsts, sh.wsum, &run);      // its barriers also order the zeroing above
  {
    int pp = page_before, rank_ = (int)ex - 1;
    uint32_t acc = 0;
    for (int i = r0; i < r1; ++i) {
      const int tok = __ldcg(sel + i), pg = tok >> 4;
      if (pg != pp) {
        if (acc) atomicOr(&pmask[rank_], acc);
        acc = 0;
        ++rank_;
        parts[rank_] = pg;
        pp = pg;
      }
      acc |= 1u << (tok & 15);
    }
    if (acc) atomicOr(&pmask[rank_], acc);
  }
  if (tid == 0) c.n_parts[b] = (int)run;
  __syncthreads();
  dbg_ts(b, 29);
  return true;
}

struct CacheShared {
  uint32_t hist[kMaxBuckets + 2];
  uint32_t wsum[33];
  int32_t hostpage[512];       // CPU page ids of the first missed pages (looked up early)
  int x, need, demand, evicted, qbase, admit_pages, bypass_pages;
};

__host__ __device__ inline size_t cache_stage_smem_bytes(int max_parts, int max_pages, int max_slots) {
  return (size_t)(6 * max_parts + 1 + max_pages) * 4 + (size_t)((max_slots + 31) / 32) * 4 + 16;
}

// Cache manager of one set, run by all T threads of one CTA.  `np_in` partitions are read
// from c.parts (ascending).  smem: cache_stage_smem_bytes() of dynamic shared memory.
template <int T>
__device__ __forceinline__ void cache_stage(const DevCtx &c, int b, int set, int np_in, int tail_pages,
                                            int tail_len, int epoch, int32_t *smem, CacheShared &sh) {
  int32_t *s_parts = smem;                          // [max_parts]
  int32_t *s_tokens = s_parts + c.max_parts;        // [max_parts]
  int32_t *s_pageoff = s_tokens + c.max_parts;      // [max_parts + 1]
  int32_t *s_missoff = s_pageoff + c.max_parts + 1; // [max_parts] offset into the free list
  int32_t *s_missbefore = s_missoff + c.max_parts;  // [max_parts] missed pages of earlier partitions
  int32_t *s_state = s_missbefore + c.max_parts;    // [max_parts]
  int32_t *s_free = s_state + c.max_parts;          // [max_pages]
  uint32_t *s_hit = reinterpret_cast<uint32_t *>(s_free + c.max_pages);   // [max_slots/32]
  const int tid = threadIdx.x;
  const SetState st = c.state[set];
  const int S = st.slots, n = c.n_buckets, t = st.step;
  const int top = min(t, n - 1);
  int np = np_in;
  const int32_t *g_parts = c.parts + (size_t)b * c.max_parts;
  const size_t pl = (size_t)b * (c.max_pages + c.tail_cap);
  int32_t *page_src = c.page_src + pl, *page_slot = c.page_slot + pl;
  int32_t *page_part = c.page_part + pl, *page_pidx = c.page_pidx + pl;
  uint32_t *page_mask = c.page_mask + pl;
  int32_t *page_fill = c.page_fill + pl;
  int4 *page_desc = c.page_desc + pl;
  if (tid == 0) c.att_count[b] = 0;

  // ---- step 1: hit/miss classification, page demand ------------------------------------
  uint32_t run_all = 0, run_miss = 0;
  for (int base = 0; base < np; base += T) {
    const int r = base + tid;
    uint32_t npg = 0, miss = 0;
    if (r < np) {
      const int p = __ldcg(g_parts + r);
      const MetaEntry *m = meta_at(c, set, p);
      int tokens = 0, res = 1;
      if (m) { tokens = m->tokens; res = m->resident; } else dev_error(c, kErrBounds);
      npg = (tokens + kPageTokens - 1) / kPageTokens;
      miss = res ? 0 : 1;
      s_parts[r] = p;
      s_tokens[r] = tokens;
      s_state[r] = res ? kHit : kAdmit;
    }
    uint32_t tot_a, tot_m;
    const uint32_t ex_a = block_scan<T>(npg, sh.wsum, &tot_a);
    const uint32_t ex_m = block_scan<T>(miss ? npg : 0, sh.wsum, &tot_m);
    if (r < np) {
      s_pageoff[r] = run_all + ex_a;
      s_missoff[r] = run_miss + ex_m;
      s_missbefore[r] = run_miss + ex_m;
    }
    run_all += tot_a;
    run_miss += tot_m;
  }
  if (tid == 0) {
    s_pageoff[np] = run_all;
    sh.evicted = 0;
    sh.admit_pages = 0;
    sh.bypass_pages = 0;
  }
  int total_pages = (int)run_all;
  const int demand = (int)run_miss;
  if (total_pages > c.max_pages) {
    // more pages than the scratch holds: drop the partitions that do not fit, report it
    if (tid == 0) dev_error(c, kErrPageList);
    __syncthreads();
    while (np > 0 && s_pageoff[np] > c.max_pages) --np;
    total_pages = s_pageoff[np];
  }
  for (int i = tid; i < (S + 31) / 32; i += T) s_hit[i] = 0;
  for (int i = tid; i < kMaxBuckets + 2; i += T) sh.hist[i] = 0;
  __syncthreads();

  // Retrieve step 3, started early: the Partition Offset / CPU page table entries of the
  // missed pages live in pinned host memory, two dependent reads over the host link.  They
  // are issued here and consumed after the table scans below, which hides their latency.
  int early_i = 0, early_off = -1, early_host = -1;
  if (resolve_in_manager(c) && tid < demand && np > 0) {
    const int r = owner_of(s_missbefore, np, tid);
    early_i = tid - s_missbefore[r];
    const int32_t *off = off_lookup(c, set, s_parts[r]);
    if (off) early_off = *off;
  }

  // ---- step 2: one scan of the GPU page table: promote, demote, histogram ---------------
  for (int s = tid; s < S; s += T) {
    GptEntry *e = gpt_at(c, set, s);
    if (!e) { dev_error(c, kErrBounds); continue; }
    const int4 raw = *reinterpret_cast<const int4 *>(e);
    const int part = raw.x, phys = raw.y, pidx = raw.z;
    int ts = raw.w;
    if (c.trace) {
      c.evict_trace[((size_t)set * c.max_slots + s) * 2] = -1;
      c.evict_trace[((size_t)set * c.max_slots + s) * 2 + 1] = -1;
    }
    if (part < 0) { atomicAdd(&sh.hist[0], 1u); continue; }
    const int r = find_sorted(s_parts, np, part);
    if (r >= 0) {
      atomicOr(&s_hit[s >> 5], 1u << (s & 31));
      if (ts != top) e->ts = top;
      const int idx = s_pageoff[r] + pidx;
      page_src[idx] = phys;
      page_slot[idx] = s;
    } else {
      if (t > n - 1 && ts > 0) { --ts; e->ts = ts; }
      atomicAdd(&sh.hist[ts + 1], 1u);
    }
  }
  __syncthreads();

  if (early_off >= 0) {
    const int32_t *hp = cpt_lookup(c, set, early_off + early_i);
    if (hp) early_host = *hp;
  }

  // ---- step 3: threshold and eviction; free slots in ascending order --------------------
  if (tid == 0) {
    int x = -2, need = 0x7fffffff;                // nothing is <= -2: no eviction
    if (demand > 0) {
      x = n - 1;
      uint32_t cum = 0;
      for (int bk = -1; bk < n; ++bk) {
        cum += sh.hist[bk + 1];
        if ((int)cum >= demand) { x = bk; need = demand - (int)(cum - sh.hist[bk + 1]); break; }
      }
    }
    sh.x = x;
    sh.need = need;                               // pages still missing once every older bucket is gone
  }
  __syncthreads();
  const int x = sh.x;
  const bool exact = c.evict_exact && demand > 0 && x >= 0;
  if (exact) {
    // exact-demand variant: of bucket x only the first `need` pages in slot order are taken;
    // their partitions are marked non-resident here, and the sweep below takes every page of
    // bucket x whose partition carries the mark (a partition goes whole)
    const int need = sh.need;
    uint32_t seen = 0;
    for (int base = 0; base < S; base += T) {
      const int s = base + tid;
      uint32_t in_x = 0;
      int part = -1;
      if (s < S) {
        const GptEntry *e = gpt_at(c, set, s);
        if (e && e->partition >= 0 && !((s_hit[s >> 5] >> (s & 31)) & 1u) && e->ts == x) { in_x = 1; part = e->partition; }
      }
      uint32_t tot;
      const uint32_t ex = block_scan<T>(in_x, sh.wsum, &tot);
      if (in_x && (int)(seen + ex) < need) {
        MetaEntry *m = meta_at(c, set, part);
        if (m) m->resident = 0;
      }
      seen += tot;
    }
    __syncthreads();
  }
  uint32_t run_free = 0;
  if (demand > 0) {
    for (int base = 0; base < S; base += T) {
      const int s = base + tid;
      uint32_t fr = 0;
      if (s < S) {
        GptEntry *e = gpt_at(c, set, s);
        if (e) {
          const int part = e->partition;
          if (part < 0) fr = 1;
          else if (!((s_hit[s >> 5] >> (s & 31)) & 1u) && e->ts <= x &&
                   !(exact && e->ts == x && meta_at(c, set, part) && meta_at(c, set, part)->resident != 0)) {
            MetaEntry *m = meta_at(c, set, part);
            if (m) m->resident = 0;
            if (c.trace) {
              c.evict_trace[((size_t)set * c.max_slots + s) * 2] = part;
              c.evict_trace[((size_t)set * c.max_slots + s) * 2 + 1] = e->page_idx;
            }
            e->partition = -1;
            e->page_idx = 0;
            e->ts = -1;
            atomicAdd(&sh.evicted, 1);
            fr = 1;
          }
        }
      }
      uint32_t tot;
      const uint32_t ex = block_scan<T>(fr, sh.wsum, &tot);
      if (fr && run_free + ex < (uint32_t)c.max_pages) s_free[run_free + ex] = s;
      run_free += tot;
    }
  }
  __syncthreads();

  sh.hostpage[tid] = early_host;

  // ---- step 4: admission (whole partitions; what does not fit is bypassed) --------------
  if (demand > (int)run_free) {
    if (tid == 0) {
      int used = 0;
      for (int r = 0; r < np; ++r) {
        if (s_state[r] == kHit) continue;
        const int npg = (s_tokens[r] + kPageTokens - 1) / kPageTokens;
        if (npg <= (int)run_free - used) { s_missoff[r] = used; used += npg; }
        else s_state[r] = kBypass;
      }
      sh.demand = used;
    }
  } else if (tid == 0) sh.demand = demand;
  __syncthreads();
  if (tid == 0) sh.qbase = (sh.demand > 0 && c.fetch_mode != 0) ? atomicAdd(c.fetch_count, sh.demand) : 0;
  __syncthreads();
  const int qbase = sh.qbase;

  for (int r = tid; r < np; r += T) {
    c.part_state[(size_t)b * c.max_parts + r] = s_state[r];
    if (s_state[r] == kAdmit) {
      MetaEntry *m = meta_at(c, set, s_parts[r]);
      if (m) m->resident = 1;
    }
  }
  int my_admit = 0, my_bypass = 0;
  for (int idx = tid; idx < total_pages; idx += T) {
    const int r = owner_of(s_pageoff, np, idx);
    const int i = idx - s_pageoff[r], p = s_parts[r], state = s_state[r];
    const int valid = min(kPageTokens, s_tokens[r] - i * kPageTokens);
    page_mask[idx] = c.kind == kKindToken ? c.part_mask[(size_t)b * c.max_parts + r]
                                           : ((1u << valid) - 1u);
    page_part[idx] = p;
    page_pidx[idx] = i;
    page_fill[idx] = -1;
    // work order of the attention kernel: pages that cross the host link first, so that all
    // of them are requested by the first CTAs and overlap the hits' HBM traffic
    const int pos = state == kHit ? demand + (s_pageoff[r] - s_missbefore[r]) + i : s_missbefore[r] + i;
    if (state == kHit) { page_desc[pos] = make_int4(page_src[idx], -1, (int)page_mask[idx], idx); continue; }
    // lookup step 3: Partition Offset -> slice of the CPU page table (pinned host memory)
    const int mi = s_missbefore[r] + i;
    // with the fetch fused into attention the fetching warp resolves the CPU page id itself
    // (fill = -2); otherwise it is resolved here, from the early batch where possible
    int host_page = -2;
    if (resolve_in_manager(c)) {
      host_page = mi < T ? sh.hostpage[mi] : -1;
      if (host_page < 0) {
        const int32_t *off = off_lookup(c, set, p);
        const int32_t *hp = off ? cpt_lookup(c, set, *off + i) : nullptr;
        if (hp) host_page = *hp;
      }
      if (host_page < 0) { dev_error(c, kErrBounds); page_src[idx] = 0; page_mask[idx] = 0; page_desc[pos] = make_int4(0, -1, 0, idx); continue; }
    }
    if (state == kAdmit) {
      const int slot = s_free[s_missoff[r] + i];
      GptEntry *e = gpt_at(c, set, slot);
      const int phys = e->phys;
      e->partition = p;
      e->page_idx = i;
      e->ts = top;
      page_src[idx] = phys;
      page_slot[idx] = slot;
      if (c.fetch_mode == 0) {
        page_fill[idx] = host_page;               // the attention kernel brings it in (-2: and looks it up)
      } else {
        const int qi = qbase + s_missoff[r] + i;
        if (qi < c.fetch_cap) c.fetch_queue[qi] = FetchItem{host_page, phys};
        else dev_error(c, kErrBounds);
      }
      page_desc[pos] = make_int4(phys, page_fill[idx], (int)page_mask[idx], idx);
      ++my_admit;
    } else {
      page_src[idx] = host_page == -2 ? -1 : ~host_page;
      page_slot[idx] = -1;
      page_desc[pos] = host_page == -2 ? make_int4(-1, -2, (int)page_mask[idx], idx)
                                       : make_int4(~host_page, -1, (int)page_mask[idx], idx);
      ++my_bypass;
    }
  }
  if (my_admit) atomicAdd(&sh.admit_pages, my_admit);
  if (my_bypass) atomicAdd(&sh.bypass_pages, my_bypass);

  // ---- local tail: always attended -------------------------------------------------------
  for (int j = tid; j < tail_pages; j += T) {
    const int idx = total_pages + j;
    page_src[idx] = c.tail_phys[(size_t)set * c.tail_cap + j];
    page_mask[idx] = j == tail_pages - 1 ? ((1u << tail_len) - 1u) : 0xffffu;
    page_slot[idx] = -2;
    page_fill[idx] = -1;
    page_desc[idx] = make_int4(page_src[idx], -1, (int)page_mask[idx], idx);
    page_part[idx] = -1;
    page_pidx[idx] = j;
  }
  __syncthreads();
  if (tid == 0) {
    c.n_pages[b] = total_pages + tail_pages;
    c.n_parts[b] = np;
    c.state[set].step = t + 1;
    Counters *k = c.counters;
    const int miss_pages = sh.admit_pages + sh.bypass_pages;
    atomicAdd(&k->set_steps, 1ull);
    atomicAdd(&k->selected_partitions, (unsigned long long)np);
    atomicAdd(&k->selected_pages, (unsigned long long)total_pages);
    atomicAdd(&k->tail_pages, (unsigned long long)tail_pages);
    atomicAdd(&k->hit_pages, (unsigned long long)(total_pages - miss_pages));
    atomicAdd(&k->miss_pages, (unsigned long long)miss_pages);
    atomicAdd(&k->evicted_pages, (unsigned long long)sh.evicted);
    atomicAdd(&k->bypass_pages, (unsigned long long)sh.bypass_pages);
    c.n_miss[b] = 0;                             // no early list on this path: both flags go up together
    flag_publish(c.ready1 + b, epoch);
    flag_publish(c.ready + b, epoch);            // attention may start on this set
  }
}

// ---------------------------------------------------------------------------------------------
// Fast path of the fused continuation: top-k + cache manager of one set by one CTA, for sets
// whose candidate keys and GPU page table both fit in shared memory (partition and cluster
// granularity, up to kFastSlots slots).  Same results as topk_stage + cache_stage; what differs
// is latency: the directories and the whole GPU page table are brought into shared memory by
// cp.async while the radix select runs, the compaction and the free-slot scan need one block
// scan each, and the page table is written back once at the end.  The time this takes is the
// time before the set's missed pages can start to cross the host link.
constexpr int kFastSlots = 1024;


constexpr int kFastDigitBits = 11, kFastBins = 1 << kFastDigitBits;
constexpr int kFastSmall = 32;               // a threshold bin this small is finished by one warp

struct FastShared {
  uint32_t wor[32], wand[32];  // per-warp OR / AND of the keys
  uint32_t cand[kFastSmall];   // keys of the threshold bin
  uint32_t ncand, bin_count;
  uint32_t wsum[33];
  uint32_t lhist[kMaxBuckets + 2];
  uint32_t prefix, remaining;
  int x, need, demand, evicted, qbase, admit_pages, bypass_pages;
};

__host__ __device__ inline size_t fast_smem_bytes(int n_keys, int slots, int dir_part, int dir_slot, int dir_page,
                                                  int max_parts, int max_pages, int tbl_cap) {
  size_t b = (size_t)((n_keys + 3) / 4 * 4) * 4;                 // keys
  b += (size_t)slots * 16;                                       // GPU page table copy
  b += (size_t)((2 * dir_part + dir_slot + dir_page + 3) / 4 * 4) * 4;   // the four directories
  b += (size_t)(7 * max_parts + 4 + 2 * max_pages) * 4;          // cache manager tables, free list, host ids
  b += (size_t)((slots + 31) / 32 + 4) * 4;                      // hit bitmask
  b += (size_t)((tbl_cap + 3) / 4 * 4) * 16 + 16;                // snapshot of the set's three partition tables
  b += (size_t)2048 * 4;                                         // digit histogram of the select
  return b + 64;
}

// Host side: can one CTA run the cache manager of every set of this batch on shared-memory
// copies (cache_fast), and if so with how large a snapshot of the partition tables?
inline bool plan_cache_fast(const DevCtx &c, const Batch &b, size_t smem_limit, int *tbl_cap, size_t *smem) {
  int max_slots_batch = 0, max_parts_batch = 0;
  for (int i = 0; i < b.n_req; ++i) {
    max_slots_batch = b.slots[i] > max_slots_batch ? b.slots[i] : max_slots_batch;
    max_parts_batch = b.n_partitions[i] > max_parts_batch ? b.n_partitions[i] : max_parts_batch;
  }
  const size_t fs = fast_smem_bytes(0, max_slots_batch, c.dir_part, c.dir_slot, c.dir_page, c.max_parts, c.max_pages, 0);
  *tbl_cap = 0;
  *smem = fs;
  if (max_slots_batch > 1024 || fs > 96 * 1024) return false;
  if (c.kind != kKindCluster && max_parts_batch > 0) {
    const size_t ft = fast_smem_bytes(0, max_slots_batch, c.dir_part, c.dir_slot, c.dir_page, c.max_parts, c.max_pages, max_parts_batch);
    if (ft <= smem_limit) { *tbl_cap = max_parts_batch; *smem = ft; }
  }
  return true;
}

__device__ __forceinline__ void cp_async4(void *smem_dst, const void *gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async16_ca(void *smem_dst, const void *gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

struct FastLayout {
  uint32_t *s_keys;
  int4 *s_gpt;
  int32_t *s_mdir, *s_gdir, *s_odir, *s_cdir, *s_parts, *s_tokens, *s_off, *s_pageoff, *s_missoff, *s_missbefore, *s_state, *s_free, *s_host;
  uint32_t *s_hit;
  // Optional snapshot of the set's Meta-partition, Partition Offset and CPU page tables (entries
  // [0, tbl_cap), 0 = none): taken while the radix select runs, so that classifying the
  // selection and finding the missed pages' host ids costs no further trip to memory.
  int2 *s_meta;
  int32_t *s_offt, *s_cptt;
  int tbl_cap;
  uint32_t *s_hist;            // [kFastBins]
};

__device__ __forceinline__ FastLayout fast_layout(const DevCtx &c, uint8_t *dyn, int n_keys, int S, int tbl_cap) {
  FastLayout L;
  L.s_keys = reinterpret_cast<uint32_t *>(dyn);
  L.s_gpt = reinterpret_cast<int4 *>(L.s_keys + (n_keys + 3) / 4 * 4);
  L.s_mdir = reinterpret_cast<int32_t *>(L.s_gpt + S);
  L.s_gdir = L.s_mdir + c.dir_part;
  L.s_odir = L.s_gdir + c.dir_slot;
  L.s_cdir = L.s_odir + c.dir_part;
  L.s_parts = L.s_mdir + (2 * c.dir_part + c.dir_slot + c.dir_page + 3) / 4 * 4;
  L.s_tokens = L.s_parts + c.max_parts;
  L.s_off = L.s_tokens + c.max_parts;            // Partition Offset entries of the selected partitions
  L.s_pageoff = L.s_off + c.max_parts;           // [max_parts + 1]
  L.s_missoff = L.s_pageoff + c.max_parts + 1;
  L.s_missbefore = L.s_missoff + c.max_parts;
  L.s_state = L.s_missbefore + c.max_parts;
  L.s_free = L.s_state + c.max_parts + 3;        // [max_pages]
  L.s_host = L.s_free + c.max_pages;             // [max_pages] CPU page ids of missed pages
  L.s_hit = reinterpret_cast<uint32_t *>(L.s_host + c.max_pages);
  const uintptr_t t = (reinterpret_cast<uintptr_t>(L.s_hit + (S + 31) / 32 + 4) + 15) & ~(uintptr_t)15;
  const int tc = (tbl_cap + 3) / 4 * 4;
  L.tbl_cap = tbl_cap;
  L.s_meta = reinterpret_cast<int2 *>(t);
  L.s_offt = reinterpret_cast<int32_t *>(L.s_meta + tc);
  L.s_cptt = L.s_offt + tc;
  L.s_hist = reinterpret_cast<uint32_t *>(L.s_cptt + tc);
  return L;
}
// true when the snapshot also holds the two host-side tables (read from their HBM copies)
__device__ __forceinline__ bool fast_snap_host(const DevCtx &c, const FastLayout &L) {
  return L.tbl_cap > 0 && resolve_in_manager(c) && c.off_mirror && c.cpt_mirror;
}

// Directories of the Meta-partition table and of the GPU page table (and, when this CTA
// resolves CPU page ids, of the Partition Offset and CPU page tables) -> shared memory (one
// cp.async group; the caller waits for it and barriers before fast_prefetch_gpt).
template <int T>
__device__ __forceinline__ void fast_prefetch_dirs(const DevCtx &c, const FastLayout &L, int set, int S) {
  const int tid = threadIdx.x, n_gdir = (S + (1 << c.seg_shift) - 1) >> c.seg_shift;
#pragma unroll 1
  for (int i = tid; i < c.dir_part; i += T) cp_async4(L.s_mdir + i, c.dir_meta + (size_t)set * c.dir_part + i);
#pragma unroll 1
  for (int i = tid; i < n_gdir; i += T) cp_async4(L.s_gdir + i, c.dir_gpt + (size_t)set * c.dir_slot + i);
  if (resolve_in_manager(c)) {
#pragma unroll 1
    for (int i = tid; i < c.dir_part; i += T) cp_async4(L.s_odir + i, c.dir_off + (size_t)set * c.dir_part + i);
#pragma unroll 1
    for (int i = tid; i < c.dir_page; i += T) cp_async4(L.s_cdir + i, c.dir_cpt + (size_t)set * c.dir_page + i);
  }
  asm volatile("cp.async.commit_group;\n" ::: "memory");
}
// The set's whole GPU page table -> shared memory (one cp.async group).
template <int T>
__device__ __forceinline__ void fast_prefetch_gpt(const DevCtx &c, const FastLayout &L, int S) {
  const int tid = threadIdx.x, seg_mask = (1 << c.seg_shift) - 1;
#pragma unroll 1
  for (int s_ = tid; s_ < S; s_ += T) {
    const int seg = L.s_gdir[s_ >> c.seg_shift];
    if (seg >= 0) cp_async16_ca(L.s_gpt + s_, c.gpt_pool + ((size_t)seg << c.seg_shift) + (s_ & seg_mask));
    else { dev_error(c, kErrBounds); L.s_gpt[s_] = make_int4(-1, 0, 0, -1); }
  }
  asm volatile("cp.async.commit_group;\n" ::: "memory");
}

// The first min(n_part, tbl_cap) entries of the set's partition tables -> shared memory (one
// cp.async group; needs the directories in shared memory).
template <int T>
__device__ __forceinline__ void fast_prefetch_tables(const DevCtx &c, const FastLayout &L, int n_part) {
  const int tid = threadIdx.x, seg_mask = (1 << c.seg_shift) - 1, n = min(n_part, L.tbl_cap);
#pragma unroll 1
  for (int e = 2 * tid; e < n; e += 2 * T) {
    const int seg = L.s_mdir[e >> c.seg_shift];
    if (seg >= 0) cp_async16_ca(L.s_meta + e, c.meta_pool + ((size_t)seg << c.seg_shift) + (e & seg_mask));
    else { L.s_meta[e] = make_int2(0, 1); L.s_meta[e + 1] = make_int2(0, 1); }
  }
  if (fast_snap_host(c, L))
#pragma unroll 1
    for (int e = 4 * tid; e < n; e += 4 * T) {
      const int oseg = L.s_odir[e >> c.seg_shift];
      const int cseg = (e >> c.seg_shift) < c.dir_page ? L.s_cdir[e >> c.seg_shift] : -1;
      if (oseg >= 0) cp_async16_ca(L.s_offt + e, c.off_mirror + ((size_t)oseg << c.seg_shift) + (e & seg_mask));
      else for (int j = 0; j < 4; ++j) L.s_offt[e + j] = -1;
      if (cseg >= 0) cp_async16_ca(L.s_cptt + e, c.cpt_mirror + ((size_t)cseg << c.seg_shift) + (e & seg_mask));
      else for (int j = 0; j < 4; ++j) L.s_cptt[e + j] = -1;
    }
  asm volatile("cp.async.commit_group;\n" ::: "memory");
}

template <int T>
__device__ __forceinline__ void cache_fast(const DevCtx &c, const Batch &bt, int b, int i_req, int set,
                                           const FastLayout &L, int np_sel, FastShared &sh);

// prefetched: the caller has already issued fast_prefetch_dirs, waited for it behind a barrier,
// and issued fast_prefetch_gpt / fast_prefetch_tables (a CTA that waits for its set to be
// scored brings the tables in while it waits)
template <int T>
__device__ __forceinline__ void select_fast(const DevCtx &c, const Batch &bt, int b, int i_req, int set,
                                            uint8_t *dyn, int keys_cap, int tbl_cap, FastShared &sh,
                                            bool prefetched = false, bool xfer = false) {
  const int tid = threadIdx.x;
  const bool token = c.kind == kKindToken;
  const int n = token ? bt.n_partitions[i_req] * kPageTokens : bt.n_partitions[i_req];
  const int k = min(c.topk, n);
  const int S = bt.slots[i_req];
  // keys that do not fit in shared memory are re-read from the scores (L2 resident: the
  // scoring CTAs have just written them); the launcher avoids that for large sets
  const bool cached = n <= keys_cap;

  const FastLayout L = fast_layout(c, dyn, keys_cap, S, tbl_cap);
  uint32_t *s_keys = L.s_keys;
  int32_t *s_parts = L.s_parts;
  int32_t *s_sel = token ? L.s_host : L.s_parts;     // chosen candidates; tokens are folded into pages below

  dbg_ts(b, 1);
  // ---- directories on their way (consumed after the keys are loaded) ------------------------
  if (!prefetched) fast_prefetch_dirs<T>(c, L, set, S);

  float *scores = c.scores + (size_t)b * c.max_cand;
  float *xfer_in = c.score_xfer + (size_t)b * c.max_cand;
  auto key_at = [&](int i) { return cached ? s_keys[i] : order_key(__ldcg(scores + i)); };
  // keys -> shared memory, with the OR and AND of all keys taken on the way (see the select)
  uint32_t k_or = 0, k_and = 0xffffffffu;
  if (xfer) {
    // scores come through the hand-over buffer: taken out (pattern restored) and kept in c.scores
#pragma unroll 4
    for (int i = tid; i < n; i += T) {
      const float sc = take_score(c, xfer_in + i);
      scores[i] = sc;
      const uint32_t key = order_key(sc);
      if (cached) s_keys[i] = key;
      k_or |= key; k_and &= key;
    }
    if (!cached) { __threadfence_block(); __syncthreads(); }       // key_at re-reads c.scores written by other threads
  } else {
#pragma unroll 8
    for (int i = tid; i < n; i += T) {
      const uint32_t key = order_key(__ldcg(scores + i));
      if (cached) s_keys[i] = key;
      k_or |= key; k_and &= key;
    }
  }
  k_or = __reduce_or_sync(0xffffffffu, k_or);
  k_and = __reduce_and_sync(0xffffffffu, k_and);
  if ((tid & 31) == 0) { sh.wor[tid >> 5] = k_or; sh.wand[tid >> 5] = k_and; }
#pragma unroll 1
  for (int i = tid; i < kFastBins; i += T) L.s_hist[i] = 0;
  if (tid == 0) {
    sh.ncand = 0;
    c.n_sel[b] = k;
    atomicAdd(&c.counters->candidates_scored, (unsigned long long)n);
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  __syncthreads();

  dbg_ts(b, 2);
  // ---- the GPU page table on its way (consumed after top-k) ---------------------------------
  if (!prefetched) {
    fast_prefetch_gpt<T>(c, L, S);
    fast_prefetch_tables<T>(c, L, bt.n_partitions[i_req]);
  }

  // ---- top-k: wide-digit radix select, one-scan ordered compaction ---------------------------
  int32_t *g_sel = c.sel_ids + (size_t)b * c.max_sel;
  int32_t *g_parts = c.parts + (size_t)b * c.max_parts;
  if (k == n) {
#pragma unroll 1
    for (int i = tid; i < n; i += T) { s_sel[i] = i; g_sel[i] = i; }
  } else {
    // Radix select with wide digits.  The scores of one set share their sign, exponent and often
    // a few mantissa bits: the bits on which all keys agree (OR == AND) are skipped, and the
    // first digit is the next kFastDigitBits bits.  One histogram then leaves a handful of keys
    // in the bin of the k-th best, which one warp ranks directly; a bin that is still crowded
    // goes round again on the following bits.
    uint32_t a_or = 0, a_and = 0xffffffffu;
#pragma unroll
    for (int j = 0; j < T / 32; ++j) { a_or |= sh.wor[j]; a_and &= sh.wand[j]; }
    const uint32_t differ = a_or ^ a_and;                          // bits on which some keys differ
    uint32_t thr = a_and, need_eq = k;                             // differ == 0: all keys are equal
    if (differ != 0) {
      int topbit = 31 - __clz(differ);                             // highest undecided bit
      uint32_t mask = topbit == 31 ? 0u : ~((2u << topbit) - 1u);  // decided bits
      uint32_t prefix = a_and & mask, remaining = k;
      int wb = 0;
      constexpr int kPer = kFastBins / T;
#pragma unroll 1
      for (;;) {
        const int shift = max(0, topbit + 1 - kFastDigitBits), width = topbit + 1 - shift;
        const uint32_t dmask = (1u << width) - 1u;
#pragma unroll 1
        for (int i = tid; i < n; i += T) {
          const uint32_t key = key_at(i);
          if ((key & mask) == prefix) atomicAdd(&L.s_hist[(key >> shift) & dmask], 1u);
        }
        __syncthreads();
        dbg_ts(b, 16);
        uint32_t loc[kPer], sum = 0;                               // this thread's bins, best first
#pragma unroll
        for (int j = 0; j < kPer; ++j) { loc[j] = L.s_hist[kFastBins - 1 - kPer * tid - j]; sum += loc[j]; }
        uint32_t tot;
        const uint32_t before = block_scan1<T>(sum, sh.wsum + wb, &tot);
        wb ^= 16;
        if (before < remaining && before + sum >= remaining) {
          uint32_t cum = before;
#pragma unroll
          for (int j = 0; j < kPer; ++j) {
            if (cum < remaining && cum + loc[j] >= remaining) {
              sh.prefix = prefix | ((uint32_t)(kFastBins - 1 - kPer * tid - j) << shift);
              sh.remaining = remaining - cum;
              sh.bin_count = loc[j];
            }
            cum += loc[j];
          }
        }
        __syncthreads();
        dbg_ts(b, 30);
        prefix = sh.prefix;
        remaining = sh.remaining;
        mask |= dmask << shift;
        const uint32_t m = sh.bin_count;
        if (shift == 0) break;                                     // the key is decided to its last bit
        if (m <= (uint32_t)kFastSmall) {
          // the bin's keys, gathered in any order; warp 0 finds the one with `remaining - 1` above it
#pragma unroll 1
          for (int i = tid; i < n; i += T) {
            const uint32_t key = key_at(i);
            if ((key & mask) == prefix) sh.cand[atomicAdd(&sh.ncand, 1u) & (kFastSmall - 1)] = key;
          }
          __syncthreads();
          if (tid < 32) {
            const uint32_t mine = tid < (int)m ? sh.cand[tid] : 0u;
            uint32_t gt = 0, ge = 0;
#pragma unroll 1
            for (uint32_t j = 0; j < m; ++j) {
              const uint32_t o = __shfl_sync(0xffffffffu, mine, (int)j);
              gt += o > mine; ge += o >= mine;
            }
            if (tid < (int)m && gt < remaining && ge >= remaining) { sh.prefix = mine; sh.remaining = remaining - gt; }
          }
          __syncthreads();
          prefix = sh.prefix;
          remaining = sh.remaining;
          break;
        }
        topbit = shift - 1;
#pragma unroll 1
        for (int i = tid; i < kFastBins; i += T) L.s_hist[i] = 0;
        __syncthreads();
      }
      thr = prefix;
      need_eq = remaining;
    }
    dbg_ts(b, 17);
    // every thread owns a contiguous run of candidates: one block scan (both counts packed into
    // a word) places all of them in index order
    const int E = (n + T - 1) / T, lo = min(n, tid * E), hi = min(n, lo + E);
    uint32_t cnt = 0;                                              // above: low half, equal: high half
#pragma unroll 1
    for (int i = lo; i < hi; ++i) { const uint32_t key = key_at(i); cnt += (key > thr) + ((uint32_t)(key == thr) << 16); }
    uint32_t tot_cnt;
    const uint32_t ex = block_scan1<T>(cnt, sh.wsum + 8, &tot_cnt);
    uint32_t gt_before = ex & 0xffffu, eq_before = ex >> 16;
#pragma unroll 1
    for (int i = lo; i < hi; ++i) {
      const uint32_t key = key_at(i);
      if (key > thr || (key == thr && eq_before < need_eq)) {
        const uint32_t pos = gt_before + min(eq_before, need_eq);
        s_sel[pos] = i; g_sel[pos] = i;
      }
      gt_before += key > thr;
      eq_before += key == thr;
    }
  }
  __syncthreads();
  int np = k;
  if (!token) {
#pragma unroll 1
    for (int i = tid; i < k; i += T) g_parts[i] = s_sel[i];
  } else {
    // chosen tokens (ascending) -> their pages (ascending, unique) + a 16-bit token mask per page
    uint32_t *s_mask = reinterpret_cast<uint32_t *>(L.s_free);
#pragma unroll 1
    for (int i = tid; i < k; i += T) s_mask[i] = 0;
    __syncthreads();
    uint32_t run = 0;
#pragma unroll 1
    for (int base = 0; base < k; base += T) {
      const int i = base + tid;
      uint32_t first = 0;
      int tok = 0;
      if (i < k) {
        tok = s_sel[i];
        first = (i == 0) || ((s_sel[i - 1] >> 4) != (tok >> 4));
      }
      uint32_t total;
      const uint32_t ex = block_scan<T>(first, sh.wsum, &total);
      if (i < k) {
        const uint32_t rank_ = run + ex + first - 1;
        if (first) { s_parts[rank_] = tok >> 4; g_parts[rank_] = tok >> 4; }
        atomicOr(&s_mask[rank_], 1u << (tok & 15));
      }
      run += total;
    }
    np = (int)run;
    __syncthreads();
    uint32_t *g_mask = c.part_mask + (size_t)b * c.max_parts;
#pragma unroll 1
    for (int i = tid; i < np; i += T) g_mask[i] = s_mask[i];
  }
  dbg_ts(b, 3);
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");     // page table copy and table snapshot have landed
  __syncthreads();
  cache_fast<T>(c, bt, b, i_req, set, L, np, sh);
}


// Cache manager on the shared-memory copy of the page table.  Before the call: L.s_parts holds
// the np_sel selected partitions (ascending), fast_prefetch_dirs has completed, and
// fast_prefetch_gpt has been issued (its group may still be in flight).
template <int T>
__device__ __forceinline__ void cache_fast(const DevCtx &c, const Batch &bt, int b, int i_req, int set,
                                           const FastLayout &L, int np_sel, FastShared &sh) {
  const int tid = threadIdx.x;
  const int S = bt.slots[i_req], t = bt.step[i_req], nb = c.n_buckets, top = min(t, nb - 1);
  const int tail_pages = bt.tail_pages[i_req], tail_len = bt.tail_len[i_req];
  const int seg_mask = (1 << c.seg_shift) - 1;
  int4 *s_gpt = L.s_gpt;
  int32_t *s_mdir = L.s_mdir, *s_gdir = L.s_gdir, *s_parts = L.s_parts, *s_tokens = L.s_tokens;
  int32_t *s_pageoff = L.s_pageoff, *s_missoff = L.s_missoff, *s_missbefore = L.s_missbefore;
  int32_t *s_state = L.s_state, *s_free = L.s_free, *s_host = L.s_host, *s_off = L.s_off;
  const bool snap_host = fast_snap_host(c, L);
  uint32_t *s_hit = L.s_hit;
  if (tid == 0) { c.att_count[b] = 0; sh.evicted = 0; sh.admit_pages = 0; sh.bypass_pages = 0; }
  // ---- cache manager step 1: Meta-partition lookups, classification, page demand ------------
  int np = np_sel;
  uint32_t run_all = 0, run_miss = 0;
#pragma unroll 1
  for (int base = 0; base < np; base += T) {
    const int r = base + tid;
    uint32_t npg = 0, miss = 0;
    if (r < np) {
      const int p = s_parts[r];
      const int seg = s_mdir[p >> c.seg_shift];
      int tokens = 0, res = 1;
      if (seg >= 0) {
        const int2 m = p < L.tbl_cap ? L.s_meta[p]
                                     : *reinterpret_cast<const int2 *>(c.meta_pool + ((size_t)seg << c.seg_shift) + (p & seg_mask));
        tokens = m.x; res = m.y;
      } else dev_error(c, kErrBounds);
      npg = (tokens + kPageTokens - 1) / kPageTokens;
      miss = res ? 0 : 1;
      s_tokens[r] = tokens;
      s_state[r] = res ? kHit : kAdmit;
      if (miss && resolve_in_manager(c)) {
        // Retrieve step 3, first half: where the partition's pages start in the CPU page table
        const int oseg = L.s_odir[p >> c.seg_shift];
        s_off[r] = (snap_host && p < L.tbl_cap) ? L.s_offt[p]
                   : oseg >= 0 ? (c.off_mirror ? c.off_mirror : c.off_pool)[((size_t)oseg << c.seg_shift) + (p & seg_mask)] : -1;
      }
    }
    // two single-barrier scans on buffers of their own: each one's barrier also separates the
    // other buffer's reads from its next writes
    uint32_t tot_a, tot_m;
    const uint32_t ex_a = block_scan1<T>(npg, sh.wsum, &tot_a);
    const uint32_t ex_m = block_scan1<T>(miss ? npg : 0, sh.wsum + 16, &tot_m);
    if (r < np) {
      s_pageoff[r] = run_all + ex_a;
      s_missoff[r] = run_miss + ex_m;
      s_missbefore[r] = run_miss + ex_m;
    }
    run_all += tot_a;
    run_miss += tot_m;
  }
  dbg_ts(b, 18);
  if (tid == 0) s_pageoff[np] = run_all;
  int total_pages = (int)run_all;
  int demand = (int)run_miss;
  if (total_pages > c.max_pages) {
    // more pages than the list holds (reported): whole partitions are dropped from the end
    if (tid == 0) dev_error(c, kErrPageList);
    __syncthreads();
#pragma unroll 1
    while (np > 0 && s_pageoff[np] > c.max_pages) --np;
    total_pages = s_pageoff[np];
    demand = np < np_sel ? s_missbefore[np] : demand;
  }
#pragma unroll 1
  for (int i = tid; i < (S + 31) / 32; i += T) s_hit[i] = 0;
#pragma unroll 1
  for (int i = tid; i < kMaxBuckets + 2; i += T) sh.lhist[i] = 0;
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");     // the GPU page table copy has landed
  __syncthreads();

  dbg_ts(b, 4);
  // ---- the early list: Retrieve step 3 for the missed pages, then they may start to move -----
  // Which pages are missing and where they live in host memory is known before a single slot
  // has been freed.  With the fetch fused into attention those descriptors (slot still open,
  // x = -3) are published now under the set's first flag: the attention CTAs that own them
  // put the pages on the host link while this CTA goes on to promote, evict and admit, and
  // pick the slot up from page_src once the second flag is set.
  const size_t pl = (size_t)b * (c.max_pages + c.tail_cap);
  int32_t *page_src = c.page_src + pl, *page_slot = c.page_slot + pl;
  int32_t *page_part = c.page_part + pl, *page_pidx = c.page_pidx + pl;
  uint32_t *page_mask = c.page_mask + pl;
  int32_t *page_fill = c.page_fill + pl;
  int4 *page_desc = c.page_desc + pl;
  const bool early = c.fetch_mode == 0;
#pragma unroll 1
  for (int mi = tid; mi < demand; mi += T) {
    const int r = owner_of(s_missbefore, np, mi);
    const int i = mi - s_missbefore[r], p = s_parts[r];
    int host_page = -2;                     // -2: the fetching warp resolves it (host tables only)
    if (resolve_in_manager(c)) {
      // second half: the CPU page table entry (directory in shared memory, one global read)
      const int e = s_off[r] + i;
      const int cseg = (s_off[r] >= 0 && (e >> c.seg_shift) < c.dir_page) ? L.s_cdir[e >> c.seg_shift] : -1;
      host_page = (snap_host && e >= 0 && e < L.tbl_cap && e < bt.n_partitions[i_req]) ? L.s_cptt[e]
                  : cseg >= 0 ? (c.cpt_mirror ? c.cpt_mirror : c.cpt_pool)[((size_t)cseg << c.seg_shift) + (e & seg_mask)] : -1;
      if (host_page < -1) host_page = -1;
    }
    s_host[mi] = host_page;
    if (early) {
      const int idx = s_pageoff[r] + i;
      const int valid = min(kPageTokens, s_tokens[r] - i * kPageTokens);
      const uint32_t pmask = c.kind == kKindToken ? c.part_mask[(size_t)b * c.max_parts + r] : ((1u << valid) - 1u);
      page_part[idx] = p;
      page_pidx[idx] = i;
      page_desc[mi] = host_page == -1 ? make_int4(0, -1, 0, idx) : make_int4(-3, host_page, (int)pmask, idx);
    }
  }
  __syncthreads();
  if (tid == 0) {
    c.n_pages[b] = total_pages + tail_pages;
    c.n_miss[b] = early ? demand : 0;
    flag_publish(c.ready1 + b, bt.epoch);
  }

  dbg_ts(b, 19);
  // ---- step 2: one pass over the page table copy: promote, demote, histogram ----------------
#pragma unroll 1
  for (int s_ = tid; s_ < S; s_ += T) {
    int4 e = s_gpt[s_];
    if (c.trace) {
      c.evict_trace[((size_t)set * c.max_slots + s_) * 2] = -1;
      c.evict_trace[((size_t)set * c.max_slots + s_) * 2 + 1] = -1;
    }
    if (e.x < 0) { atomicAdd(&sh.lhist[0], 1u); continue; }
    const int r = find_sorted(s_parts, np, e.x);
    if (r >= 0) {
      atomicOr(&s_hit[s_ >> 5], 1u << (s_ & 31));
      e.w = top;
      const int idx = s_pageoff[r] + e.z;
      page_src[idx] = e.y;
      page_slot[idx] = s_;
    } else {
      if (t > nb - 1 && e.w > 0) --e.w;
      atomicAdd(&sh.lhist[e.w + 1], 1u);
    }
    s_gpt[s_] = e;
  }
  __syncthreads();

  dbg_ts(b, 5);
  // ---- step 3: threshold, eviction, free slots in ascending order (one scan) ----------------
  if (tid == 0) {
    int x = -2, need = 0x7fffffff;
    if (demand > 0) {
      x = nb - 1;
      uint32_t cum = 0;
#pragma unroll 1
      for (int bk = -1; bk < nb; ++bk) {
        cum += sh.lhist[bk + 1];
        if ((int)cum >= demand) { x = bk; need = demand - (int)(cum - sh.lhist[bk + 1]); break; }
      }
    }
    sh.x = x;
    sh.need = need;                               // pages still missing once every older bucket is gone
  }
  __syncthreads();
  const int x = sh.x;
  const bool exact = c.evict_exact && demand > 0 && x >= 0;
  if (exact) {
    // exact-demand variant (see cache_stage): mark the partitions of the first `need` pages
    // of bucket x in slot order
    const int need = sh.need;
    const int E = (S + T - 1) / T, lo = min(S, tid * E), hi = min(S, lo + E);
    uint32_t in_x = 0;
#pragma unroll 1
    for (int s_ = lo; s_ < hi; ++s_) {
      const int4 e = s_gpt[s_];
      in_x += e.x >= 0 && !((s_hit[s_ >> 5] >> (s_ & 31)) & 1u) && e.w == x;
    }
    uint32_t tot;
    uint32_t rank_ = block_scan<T>(in_x, sh.wsum, &tot);
#pragma unroll 1
    for (int s_ = lo; s_ < hi; ++s_) {
      const int4 e = s_gpt[s_];
      if (e.x >= 0 && !((s_hit[s_ >> 5] >> (s_ & 31)) & 1u) && e.w == x) {
        if ((int)rank_ < need) {
          const int seg = s_mdir[e.x >> c.seg_shift];
          if (seg >= 0) c.meta_pool[((size_t)seg << c.seg_shift) + (e.x & seg_mask)].resident = 0;
        }
        ++rank_;
      }
    }
    __syncthreads();
  }
  dbg_ts(b, 20);
  uint32_t run_free = 0;
  if (demand > 0) {
    const int E = (S + T - 1) / T, lo = min(S, tid * E), hi = min(S, lo + E);
    uint32_t nfree = 0;
#pragma unroll 1
    for (int s_ = lo; s_ < hi; ++s_) {
      int4 e = s_gpt[s_];
      if (e.x < 0) { ++nfree; continue; }
      if (!((s_hit[s_ >> 5] >> (s_ & 31)) & 1u) && e.w <= x) {
        const int seg = s_mdir[e.x >> c.seg_shift];
        if (exact && e.w == x && seg >= 0 &&
            c.meta_pool[((size_t)seg << c.seg_shift) + (e.x & seg_mask)].resident != 0) continue;   // spared
        if (seg >= 0) c.meta_pool[((size_t)seg << c.seg_shift) + (e.x & seg_mask)].resident = 0;
        if (c.trace) {
          c.evict_trace[((size_t)set * c.max_slots + s_) * 2] = e.x;
          c.evict_trace[((size_t)set * c.max_slots + s_) * 2 + 1] = e.z;
        }
        s_gpt[s_] = make_int4(-1, e.y, 0, -1);
        atomicAdd(&sh.evicted, 1);
        ++nfree;
      }
    }
    uint32_t tot;
    uint32_t pos = block_scan<T>(nfree, sh.wsum, &tot);
#pragma unroll 1
    for (int s_ = lo; s_ < hi; ++s_)
      if (s_gpt[s_].x < 0) { if (pos < (uint32_t)c.max_pages) s_free[pos] = s_; ++pos; }
    run_free = tot;
  }
  dbg_ts(b, 21);
  __syncthreads();

  dbg_ts(b, 6);
  // ---- step 4: admission --------------------------------------------------------------------
  if (demand > (int)run_free) {
    if (tid == 0) {
      int used = 0;
#pragma unroll 1
      for (int r = 0; r < np; ++r) {
        if (s_state[r] == kHit) continue;
        const int npg = (s_tokens[r] + kPageTokens - 1) / kPageTokens;
        if (npg <= (int)run_free - used) { s_missoff[r] = used; used += npg; }
        else s_state[r] = kBypass;
      }
      sh.demand = used;
    }
  } else if (tid == 0) sh.demand = demand;
  __syncthreads();
  if (tid == 0) sh.qbase = (sh.demand > 0 && c.fetch_mode != 0) ? atomicAdd(c.fetch_count, sh.demand) : 0;
  __syncthreads();
  const int qbase = sh.qbase;
  dbg_ts(b, 22);
#pragma unroll 1
  for (int r = tid; r < np; r += T) {
    c.part_state[(size_t)b * c.max_parts + r] = s_state[r];
    if (s_state[r] == kAdmit) {
      const int p = s_parts[r], seg = s_mdir[p >> c.seg_shift];
      if (seg >= 0) c.meta_pool[((size_t)seg << c.seg_shift) + (p & seg_mask)].resident = 1;
    }
  }
  int my_admit = 0, my_bypass = 0;
  dbg_ts(b, 23);
#pragma unroll 1
  for (int idx = tid; idx < total_pages; idx += T) {
    const int r = owner_of(s_pageoff, np, idx);
    const int i = idx - s_pageoff[r], p = s_parts[r], state = s_state[r];
    const int valid = min(kPageTokens, s_tokens[r] - i * kPageTokens);
    const uint32_t pmask = c.kind == kKindToken ? c.part_mask[(size_t)b * c.max_parts + r] : ((1u << valid) - 1u);
    page_mask[idx] = pmask;
    page_part[idx] = p;
    page_pidx[idx] = i;
    page_fill[idx] = -1;
    const int pos = state == kHit ? demand + (s_pageoff[r] - s_missbefore[r]) + i : s_missbefore[r] + i;
    if (state == kHit) { page_desc[pos] = make_int4(page_src[idx], -1, (int)pmask, idx); continue; }
    const int mi = s_missbefore[r] + i;
    // the CPU page id found for the early list (-2: left to the fetching warp, which then reads
    // the two pinned host tables itself, so that no page list waits on the host link)
    const int host_page = s_host[mi];
    if (host_page == -1) {
      dev_error(c, kErrBounds);
      page_src[idx] = 0; page_mask[idx] = 0;
      if (!early) page_desc[pos] = make_int4(0, -1, 0, idx);
      continue;
    }
    if (state == kAdmit) {
      const int slot = s_free[s_missoff[r] + i];
      const int phys = s_gpt[slot].y;
      s_gpt[slot] = make_int4(p, phys, i, top);
      page_src[idx] = phys;                  // what the owner of an early descriptor comes back for
      page_slot[idx] = slot;
      if (c.fetch_mode == 0) page_fill[idx] = host_page;
      else {
        const int qi = qbase + s_missoff[r] + i;
        if (qi < c.fetch_cap) c.fetch_queue[qi] = FetchItem{host_page, phys};
        else dev_error(c, kErrBounds);
        page_desc[pos] = make_int4(phys, -1, (int)pmask, idx);
      }
      ++my_admit;
    } else {
      // bypassed: attended from host memory, never cached (no slot)
      page_src[idx] = host_page == -2 ? -1 : ~host_page;
      page_slot[idx] = -1;
      if (!early) page_desc[pos] = make_int4(~host_page, -1, (int)pmask, idx);
      ++my_bypass;
    }
  }
  dbg_ts(b, 24);
  if (my_admit) atomicAdd(&sh.admit_pages, my_admit);
  if (my_bypass) atomicAdd(&sh.bypass_pages, my_bypass);
#pragma unroll 1
  for (int j = tid; j < tail_pages; j += T) {
    const int idx = total_pages + j;
    const int src = c.tail_phys[(size_t)set * c.tail_cap + j];
    const uint32_t m = j == tail_pages - 1 ? ((1u << tail_len) - 1u) : 0xffffu;
    page_src[idx] = src;
    page_mask[idx] = m;
    page_slot[idx] = -2;
    page_fill[idx] = -1;
    page_desc[idx] = make_int4(src, -1, (int)m, idx);
    page_part[idx] = -1;
    page_pidx[idx] = j;
  }
  __syncthreads();
  dbg_ts(b, 7);
  if (tid == 0) {
    c.n_pages[b] = total_pages + tail_pages;
    c.n_parts[b] = np;
    c.state[set].step = t + 1;
    flag_publish(c.ready + b, bt.epoch);
    // the counters go last: the flag's fence should not have to wait for them
    Counters *kc = c.counters;
    const int miss_pages = sh.admit_pages + sh.bypass_pages;
    atomicAdd(&kc->set_steps, 1ull);
    atomicAdd(&kc->selected_partitions, (unsigned long long)np);
    atomicAdd(&kc->selected_pages, (unsigned long long)total_pages);
    atomicAdd(&kc->tail_pages, (unsigned long long)tail_pages);
    atomicAdd(&kc->hit_pages, (unsigned long long)(total_pages - miss_pages));
    atomicAdd(&kc->miss_pages, (unsigned long long)miss_pages);
    atomicAdd(&kc->evicted_pages, (unsigned long long)sh.evicted);
    atomicAdd(&kc->bypass_pages, (unsigned long long)sh.bypass_pages);
  }
  // ---- the page table goes back in one sweep; attention does not wait for it -----------------
#pragma unroll 1
  for (int s_ = tid; s_ < S; s_ += T) {
    const int seg = s_gdir[s_ >> c.seg_shift];
    if (seg >= 0) *reinterpret_cast<int4 *>(c.gpt_pool + ((size_t)seg << c.seg_shift) + (s_ & seg_mask)) = s_gpt[s_];
  }
  dbg_ts(b, 8);
}

}  // namespace spin
