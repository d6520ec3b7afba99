// Index during decode for cluster granularity (Section 4.1: Index "is invoked ... periodically
// in decode to take in new tokens"; which tokens go where is the algorithm's business).
// spin_reindex folds the FULL pages of a (request, layer)'s local tail into the clusters:
//
//   k_assign         every tail token's key against every centroid of its set, in the same
//                    fp32 summation order as Select; the best cluster (ties to the lower id)
//   (host)           the clusters' new page lists and the set's CPU page table / Partition
//                    Offset layout, a destination row for every token
//   k_move_rows      K/V rows from the HBM tail pages to their rows in pinned host memory
//   k_reindex_apply  new token counts in the Meta-partition table; a cluster that took a
//                    token loses its (stale) GPU residency: flag and slots cleared; the tail
//                    shrinks to the partly filled newest page
#define SPIN_FILE_ID 5
#include "spin_dev.cuh"

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

// One CTA per (tail token, kv head): 16 rows of 16 lanes walk the centroids, a lane owning 8
// channels.  Summation order as in Select (8 channels left to right, then the balanced tree
// over the 16 blocks), so the CPU oracle reproduces every score and with it every choice.
__global__ void __launch_bounds__(256)
k_assign(DevCtx c, int req, int layer, int n_clusters, int32_t *__restrict__ assign) {
  __shared__ float s_best[16];
  __shared__ int s_arg[16];
  const int t = blockIdx.x, head = blockIdx.y, set = set_index(c, req, layer, head);
  const int lane16 = threadIdx.x & 15, grp = threadIdx.x >> 4;
  const uint32_t row_mask = 0xffffu << (threadIdx.x & 16);
  const int32_t phys = c.tail_phys[(size_t)set * c.tail_cap + t / kPageTokens];
  if (phys < 0 || phys >= c.n_gpu_pages) { if (threadIdx.x == 0) { dev_error(c, kErrBounds); assign[(size_t)t * c.Hkv + head] = 0; } return; }
  const uint8_t *krow = c.gpu_pages + (size_t)phys * kPageBytes + (size_t)(t % kPageTokens) * kRowBytes;
  float kf[8];
  unpack8(*reinterpret_cast<const uint4 *>(krow + lane16 * 16), kf);
  float best = -INFINITY;
  int arg = 0x7fffffff;
  for (int cl = grp; cl < n_clusters; cl += 16) {
    const uint8_t *srow = summary_at(c, set, cl);
    if (!srow) { if (lane16 == 0) dev_error(c, kErrBounds); continue; }
    float x[8];
    unpack8(*reinterpret_cast<const uint4 *>(srow + lane16 * 16), x);
    float s = kf[0] * x[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) s = fmaf(kf[i], x[i], s);
    s = s + __shfl_xor_sync(row_mask, s, 1);
    s = s + __shfl_xor_sync(row_mask, s, 2);
    s = s + __shfl_xor_sync(row_mask, s, 4);
    s = s + __shfl_xor_sync(row_mask, s, 8);
    s = s + 0.0f;
    if (s > best) { best = s; arg = cl; }          // ascending ids: the first maximum stays
  }
  if (lane16 == 0) { s_best[grp] = best; s_arg[grp] = arg; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float b = s_best[0];
    int a = s_arg[0];
    for (int g = 1; g < 16; ++g)
      if (s_best[g] > b || (s_best[g] == b && s_arg[g] < a)) { b = s_best[g]; a = s_arg[g]; }
    assign[(size_t)t * c.Hkv + head] = a == 0x7fffffff ? 0 : a;
  }
}

// Row (token t, head h) of the folded tail pages -> row dest[t][h] (host page * 16 + row).
__global__ void __launch_bounds__(256)
k_move_rows(DevCtx c, int req, int layer, const int64_t *__restrict__ dest, int n_tokens) {
  const int piece = threadIdx.x & 15;
  const size_t rows = (size_t)n_tokens * c.Hkv;
  for (size_t row = (size_t)blockIdx.x * 16 + (threadIdx.x >> 4); row < rows; row += (size_t)gridDim.x * 16) {
    const int t = (int)(row / c.Hkv), head = (int)(row % c.Hkv), set = set_index(c, req, layer, head);
    const int32_t phys = c.tail_phys[(size_t)set * c.tail_cap + t / kPageTokens];
    const int64_t d = dest[row];
    if (phys < 0 || phys >= c.n_gpu_pages || d < 0 || (d >> 4) >= c.n_host_pages) { if (piece == 0) dev_error(c, kErrBounds); continue; }
    const uint8_t *src = c.gpu_pages + (size_t)phys * kPageBytes + (size_t)(t % kPageTokens) * kRowBytes + piece * 16;
    uint8_t *dst = c.host_pages + (size_t)(d >> 4) * kPageBytes + (size_t)(d & 15) * kRowBytes + piece * 16;
    *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(src);
    *reinterpret_cast<uint4 *>(dst + kHalfPageBytes) = *reinterpret_cast<const uint4 *>(src + kHalfPageBytes);
  }
}

struct ReindexArgs {
  int32_t req, layer, n_clusters, n_folded_pages;
  int32_t tail_first, tail_pages, tail_len, n_host_pages;      // the sets' tail after the fold
};

// One CTA per kv head.  new_tokens: [Hkv][n_clusters]; touched: [Hkv][ceil(n_clusters / 32)].
__global__ void __launch_bounds__(256)
k_reindex_apply(DevCtx c, ReindexArgs a, const int32_t *__restrict__ new_tokens, const uint32_t *__restrict__ touched) {
  extern __shared__ int32_t s_tail[];
  const int head = blockIdx.x, set = set_index(c, a.req, a.layer, head), tid = threadIdx.x;
  const int words = (a.n_clusters + 31) / 32;
  const uint32_t *mine = touched + (size_t)head * words;
  for (int cl = tid; cl < a.n_clusters; cl += 256) {
    MetaEntry *m = meta_at(c, set, cl);
    if (!m) { dev_error(c, kErrBounds); continue; }
    m->tokens = new_tokens[(size_t)head * a.n_clusters + cl];
    if ((mine[cl >> 5] >> (cl & 31)) & 1u) m->resident = 0;
  }
  const int S = c.state[set].slots;
  for (int s = tid; s < S; s += 256) {
    GptEntry *e = gpt_at(c, set, s);
    if (!e) { dev_error(c, kErrBounds); continue; }
    const int p = e->partition;
    if (p >= 0 && p < a.n_clusters && ((mine[p >> 5] >> (p & 31)) & 1u)) { e->partition = -1; e->page_idx = 0; e->ts = -1; }
  }
  // the HBM tail pages rotate: the partly filled newest page becomes tail page 0
  int32_t *tp = c.tail_phys + (size_t)set * c.tail_cap;
  for (int j = tid; j < c.tail_cap; j += 256) s_tail[j] = tp[j];
  __syncthreads();
  for (int j = tid; j < c.tail_cap; j += 256) tp[j] = s_tail[(j + a.n_folded_pages) % c.tail_cap];
  if (tid == 0) {
    SetState *s = c.state + set;
    s->tail_first = a.tail_first;
    s->tail_pages = a.tail_pages;
    s->tail_len = a.tail_len;
    s->n_host_pages = a.n_host_pages;
  }
}

}  // namespace

int launch_assign(const DevCtx &c, int req, int layer, int n_clusters, int n_tokens, int32_t *assign, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  k_assign<<<dim3(n_tokens, c.Hkv), 256, 0, st>>>(c, req, layer, n_clusters, assign);
  return 1;
}

int launch_move_rows(const DevCtx &c, int req, int layer, const int64_t *dest, int n_tokens, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const size_t rows = (size_t)n_tokens * c.Hkv;
  int grid = (int)((rows + 15) / 16);
  if (grid > 1184) grid = 1184;
  k_move_rows<<<grid, 256, 0, st>>>(c, req, layer, dest, n_tokens);
  return 1;
}

int launch_reindex_apply(const DevCtx &c, int req, int layer, int n_clusters, int n_folded_pages, int tail_first,
                         int tail_pages, int tail_len, int n_host_pages, const int32_t *new_tokens,
                         const uint32_t *touched, cudaStream_t st) {
  ReindexArgs a{req, layer, n_clusters, n_folded_pages, tail_first, tail_pages, tail_len, n_host_pages};
  k_reindex_apply<<<c.Hkv, 256, (size_t)c.tail_cap * 4, st>>>(c, a, new_tokens, touched);
  return 1;
}

}  // namespace spin
