// Select (Table 1: score(q, k_sums) -> topk; Section 4.1 "Select").
//
// k_score streams the summary segments of every set of the batch once (HBM bound: 512 B per
// page for min/max summaries, 256 B per token key or centroid) and writes one fp32 score per
// candidate.  The summation order is fixed so that the CPU oracle reproduces every score bit
// for bit: a lane owns 8 consecutive channels (one 16-byte load) and adds them left to right;
// the 16 lanes of a row are then combined by a butterfly (xor 1, 2, 4, 8), which is the
// balanced tree over adjacent blocks; the group's query heads are added in ascending order.
// Products of two bf16 values are exact in fp32, so fused or separate multiply-add agree.
//
// k_topk keeps, per set, the k best candidates (ties -> lower index) with a 4-pass radix
// select on order-preserving keys followed by one ordered compaction, and emits them in
// ascending index order.  For token-granular selection it also folds the chosen tokens into
// their pages with a 16-bit token mask per page.
#include <cooperative_groups.h>

#include "spin_dev.cuh"

namespace cg = cooperative_groups;

namespace spin {

namespace {

__device__ __forceinline__ void unpack8(uint4 raw, float *f) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ uint4 ld_stream16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
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
  float tot = 0.f;
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
    s = s + __shfl_xor_sync(row_mask, s, 1);
    s = s + __shfl_xor_sync(row_mask, s, 2);
    s = s + __shfl_xor_sync(row_mask, s, 4);
    s = s + __shfl_xor_sync(row_mask, s, 8);
    tot = g == 0 ? s : tot + s;
  }
  return tot + 0.0f;                              // -0.0 -> +0.0
}

template <int G, bool MINMAX>
__global__ void __launch_bounds__(256)
k_score(DevCtx c, Batch bt, const __nv_bfloat16 *__restrict__ q) {
  const int b = blockIdx.y, i_req = b / c.Hkv, head = b % c.Hkv;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  pdl_launch_next();
  pdl_wait_prev();
  if (blockIdx.x == 0 && b == 0 && threadIdx.x == 0) *c.fetch_count = 0;   // new step, new miss queue
  const SetState st = c.state[set];
  const int n_cand = c.kind == kKindToken ? st.n_partitions * kPageTokens : st.n_partitions;
  const int seg_entries = 1 << c.sum_shift;
  const int e0 = blockIdx.x * seg_entries;
  if (e0 >= n_cand) return;
  const int seg = c.dir_sumseg[(size_t)set * c.dir_sum + blockIdx.x];
  if (seg < 0) { if (threadIdx.x == 0) dev_error(c, kErrBounds); return; }
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
  const int n_here = min(seg_entries, n_cand - e0);
  constexpr int kEntry = MINMAX ? 2 * kRowBytes : kRowBytes;
  const uint8_t *base = c.summaries + ((size_t)seg << c.sum_shift) * kEntry + lane16 * 16;
  float *out = c.scores + (size_t)b * c.max_cand + e0;

  // two entries per half-warp and iteration, all their loads issued before any arithmetic
  for (int e = grp; e < n_here; e += 32) {
    const bool two = e + 16 < n_here;
    const uint4 z = make_uint4(0, 0, 0, 0);
    const uint4 a0 = ld_stream16(base + (size_t)e * kEntry);
    const uint4 m0 = MINMAX ? ld_stream16(base + (size_t)e * kEntry + kRowBytes) : z;
    const uint4 a1 = two ? ld_stream16(base + (size_t)(e + 16) * kEntry) : z;
    const uint4 m1 = (MINMAX && two) ? ld_stream16(base + (size_t)(e + 16) * kEntry + kRowBytes) : z;
    const float s0 = score_entry<G, MINMAX>(a0, m0, qf, qsel, row_mask);
    if (lane16 == 0) out[e] = s0;
    if (two) {
      const float s1 = score_entry<G, MINMAX>(a1, m1, qf, qsel, row_mask);
      if (lane16 == 0) out[e + 16] = s1;
    }
  }
}

__device__ __forceinline__ uint32_t order_key(float s) {
  const uint32_t u = __float_as_uint(s);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kTopkThreads = 512;

// Exclusive prefix of v over the block (thread order) and the block total.
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
    uint32_t x = lane < kTopkThreads / 32 ? wsum[lane] : 0, xi = x;
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

// One thread-block cluster per set: the candidates are cut into one contiguous slice per CTA
// (keys kept in shared memory), every radix pass builds per-CTA histograms that all CTAs sum
// through distributed shared memory, and the ordered compaction uses the lower-ranked CTAs'
// counts as its offset.  A cluster of one CTA is the small-set case (a few thousand pages);
// token-granular selection over 64K+ keys uses 8 CTAs.  Cluster barriers are hardware
// barriers (no flag spinning); every CTA of a cluster executes the same number of them.
__global__ void __launch_bounds__(kTopkThreads)
k_topk(DevCtx c, Batch bt, int keys_cap) {
  extern __shared__ uint32_t s_keys[];                 // [keys_cap] order-preserving keys of this slice
  __shared__ uint32_t hist[256];                       // this CTA's histogram (read remotely)
  __shared__ uint32_t ghist[256];                      // cluster-wide histogram
  __shared__ uint32_t wsum[33];
  __shared__ uint32_t cnt[2];                          // this CTA's (above threshold, equal) counts
  __shared__ uint32_t sh_prefix, sh_remaining;
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks(), rank = (int)cluster.block_rank();
  const int b = blockIdx.x / C, i_req = b / c.Hkv, head = b % c.Hkv, tid = threadIdx.x;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  pdl_launch_next();
  pdl_wait_prev();
  const SetState st = c.state[set];
  const int n = c.kind == kKindToken ? st.n_partitions * kPageTokens : st.n_partitions;
  const int k = min(c.topk, n);
  const float *scores = c.scores + (size_t)b * c.max_cand;
  int32_t *sel = c.sel_ids + (size_t)b * c.max_sel;
  const int per = (n + C - 1) / C;
  const int lo = min(n, rank * per), m = min(n, lo + per) - lo;
  const bool cached = m <= keys_cap;

  if (tid == 0 && rank == 0) {
    c.n_sel[b] = k;
    atomicAdd(&c.counters->candidates_scored, (unsigned long long)n);
  }
  if (cached)
    for (int i = tid; i < m; i += kTopkThreads) s_keys[i] = order_key(scores[lo + i]);
  __syncthreads();
  auto key_at = [&](int i) { return cached ? s_keys[i] : order_key(scores[lo + i]); };

  if (k == n) {
    for (int i = tid; i < m; i += kTopkThreads) sel[lo + i] = lo + i;
  } else {
    // ---- radix select: key of the k-th best candidate --------------------------------
    uint32_t prefix = 0, mask = 0, remaining = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      for (int i = tid; i < m; i += kTopkThreads) {
        const uint32_t key = key_at(i);
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
      }
      cluster.sync();                                   // every CTA's histogram is complete
      if (tid < 256) {
        uint32_t tot = 0;
        for (int r = 0; r < C; ++r) tot += cluster.map_shared_rank(hist, r)[tid];
        ghist[tid] = tot;
      }
      cluster.sync();                                   // remote reads done before hist is reused
      if (tid < 32) {
        // lane l owns bins 255-8l .. 248-8l (descending); find where the count from the
        // top reaches `remaining`
        uint32_t loc[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { loc[j] = ghist[255 - 8 * tid - j]; sum += loc[j]; }
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
              sh_prefix = prefix | ((uint32_t)(255 - 8 * tid - j) << shift);
              sh_remaining = remaining - cum;
            }
            cum += loc[j];
          }
        }
      }
      __syncthreads();
      prefix = sh_prefix;
      remaining = sh_remaining;
      mask |= 255u << shift;
    }
    const uint32_t thr = prefix, need_eq = remaining;
    // ---- counts of this slice, offsets from the lower-ranked slices ---------------------
    if (tid < 2) cnt[tid] = 0;
    __syncthreads();
    {
      uint32_t gt = 0, eq = 0;
      for (int i = tid; i < m; i += kTopkThreads) {
        const uint32_t key = key_at(i);
        gt += key > thr;
        eq += key == thr;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        gt += __shfl_xor_sync(0xffffffffu, gt, o);
        eq += __shfl_xor_sync(0xffffffffu, eq, o);
      }
      if ((tid & 31) == 0) { atomicAdd(&cnt[0], gt); atomicAdd(&cnt[1], eq); }
    }
    cluster.sync();
    uint32_t run_gt = 0, run_eq = 0;
    for (int r = 0; r < rank; ++r) {
      const uint32_t *rc = cluster.map_shared_rank(cnt, r);
      run_gt += rc[0];
      run_eq += rc[1];
    }
    // ---- ordered compaction: everything above thr, plus the first need_eq equal to it --
    for (int base = 0; base < m; base += kTopkThreads) {
      const int i = base + tid;
      uint32_t gt = 0, eq = 0;
      if (i < m) {
        const uint32_t key = key_at(i);
        gt = key > thr;
        eq = key == thr;
      }
      uint32_t total;
      const uint32_t ex = block_scan(gt | (eq << 16), wsum, &total);
      const uint32_t gt_before = run_gt + (ex & 0xffffu), eq_before = run_eq + (ex >> 16);
      if (gt || (eq && eq_before < need_eq))
        sel[gt_before + min(eq_before, need_eq)] = lo + i;
      run_gt += total & 0xffffu;
      run_eq += total >> 16;
    }
  }
  cluster.sync();            // selections of all slices are written; nobody reads remote smem after this
  if (rank != 0) return;

  // ---- candidates -> partitions of the cache manager (first CTA of the cluster) ----------
  int32_t *parts = c.parts + (size_t)b * c.max_parts;
  if (c.kind != kKindToken) {
    for (int i = tid; i < k; i += kTopkThreads) parts[i] = __ldcg(sel + i);
    if (tid == 0) c.n_parts[b] = k;
    return;
  }
  uint32_t *pmask = c.part_mask + (size_t)b * c.max_parts;
  for (int i = tid; i < k; i += kTopkThreads) pmask[i] = 0;
  __syncthreads();
  uint32_t run = 0;
  for (int base = 0; base < k; base += kTopkThreads) {
    const int i = base + tid;
    uint32_t first = 0;
    int tok = 0;
    if (i < k) {
      tok = __ldcg(sel + i);
      first = (i == 0) || ((__ldcg(sel + i - 1) >> 4) != (tok >> 4));
    }
    uint32_t total;
    const uint32_t ex = block_scan(first, wsum, &total);
    if (i < k) {
      const uint32_t rank_ = run + ex + first - 1;
      if (first) parts[rank_] = tok >> 4;
      atomicOr(&pmask[rank_], 1u << (tok & 15));
    }
    run += total;
  }
  if (tid == 0) c.n_parts[b] = (int)run;
}

template <int G>
void launch_score_g(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q, dim3 grid, cudaStream_t st) {
  if (c.kind == kKindPage) launch_pdl(k_score<G, true>, grid, dim3(256), 0, st, 1, c, b, q);
  else launch_pdl(k_score<G, false>, grid, dim3(256), 0, st, 1, c, b, q);
}

}  // namespace

int launch_select(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q, int max_cand,
                  cudaStream_t st, Prof *prof) {
  const int n_sets = b.n_req * c.Hkv;
  int segs = (max_cand + (1 << c.sum_shift) - 1) >> c.sum_shift;
  if (segs < 1) segs = 1;                         // the first block also resets the miss queue
  dim3 grid(segs, n_sets);
  switch (c.G) {
    case 1: launch_score_g<1>(c, b, q, grid, st); break;
    case 2: launch_score_g<2>(c, b, q, grid, st); break;
    case 4: launch_score_g<4>(c, b, q, grid, st); break;
    default: launch_score_g<8>(c, b, q, grid, st); break;
  }
  prof_mark(prof, st, kProfScore);
  {
    // cluster size from the largest candidate count: slices of at most 8192 keys stay in smem
    int C = 1;
    while (C < 8 && (max_cand + C - 1) / C > 8192) C *= 2;
    int keys_cap = (max_cand + C - 1) / C;
    if (keys_cap > 16384) keys_cap = 0;                  // too many for shared memory: re-read from L2
    static int smem_set = 0;
    const int smem = keys_cap * 4;
    if (smem > smem_set) { cudaFuncSetAttribute(k_topk, cudaFuncAttributeMaxDynamicSharedMemorySize, smem); smem_set = smem; }
    launch_pdl(k_topk, dim3(n_sets * C), dim3(kTopkThreads), (size_t)smem, st, C, c, b, keys_cap);
  }
  prof_mark(prof, st, kProfTopk);
  return 2;
}

}  // namespace spin
