// Index + Offload (Section 4.1): write appended K/V rows through to the pinned host tier,
// keep the newest page in an HBM tail page, and turn a completed page into a candidate
// partition with its summary (per-channel min/max of the keys, or the key rows themselves
// for token-granular selection).  The host runtime has already mapped the segments and
// filled the host-side tables (Partition Offset, CPU page table) for the pages touched here.
#define SPIN_FILE_ID 1
#include "append_body.cuh"

namespace spin {

namespace {

// Pages completely covered by this call's tokens that are not the newest page: all 16 rows
// come from the input; the page is written to the host tier and indexed.
__global__ void __launch_bounds__(256)
k_append_bulk(DevCtx c, int req, int layer, const __nv_bfloat16 *__restrict__ k,
              const __nv_bfloat16 *__restrict__ v, int first_page, int first_token_of_call,
              uint8_t *__restrict__ stage, const int32_t *__restrict__ stage_hp) {
  __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
  const int head = blockIdx.y, page = first_page + blockIdx.x, tid = threadIdx.x;
  const int set = set_index(c, req, layer, head);
  const int r = tid >> 4, piece = tid & 15;
  const size_t tok = (size_t)page * kPageTokens + r - first_token_of_call;
  const size_t in_off = (tok * c.Hkv + head) * kHeadDim * 2 + piece * 16;
  uint4 kk = ld16(reinterpret_cast<const uint8_t *>(k) + in_off);
  uint4 vv = ld16(reinterpret_cast<const uint8_t *>(v) + in_off);
  const size_t unit = (size_t)head * gridDim.x + blockIdx.x;        // head-major, as host pages are handed out
  int32_t host_page;
  if (stage) {
    host_page = stage_hp[unit];
  } else {
    const int32_t *hp = cpt_at(c, set, page);
    if (!hp) { if (tid == 0) dev_error(c, 1u); return; }
    host_page = *hp;
  }
  if (tid == 0) cpt_mirror_set(c, set, page, host_page);
  // Offload: straight to the page's place in pinned host memory, or -- asynchronous offload --
  // into an HBM staging slot from which copy-engine transfers move it on the library's own stream
  uint8_t *dst = c.host_pages + (size_t)host_page * kPageBytes + r * kRowBytes + piece * 16;
  if (stage) dst = stage + unit * kPageBytes + r * kRowBytes + piece * 16;
  st16(dst, kk);
  st16(dst + kHalfPageBytes, vv);
  st16(reinterpret_cast<uint8_t *>(krows[r]) + piece * 16, kk);
  __syncthreads();
  index_page(c, set, page, krows, tid);
}

// Stand-alone edge append: one CTA per (kv head, request).
__global__ void __launch_bounds__(256)
k_append_edge(DevCtx c, AppendEdgeArgs a, const __nv_bfloat16 *__restrict__ k,
              const __nv_bfloat16 *__restrict__ v, int n_new) {
  __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
  const int head = blockIdx.x, i = blockIdx.y;
  pdl_launch_next();
  pdl_wait_prev();
  append_edge_body(c, set_index(c, a.req[i], a.layer, head), i, head, k, v, n_new, a.n_tokens[i], -1, krows);
}

// Cluster prefill: row `tok` of head `h` goes to row dest[tok][h] of the host tier (page id *
// 16 + row), where the host runtime has packed each cluster's tokens in their original order.
__global__ void __launch_bounds__(256)
k_cluster_scatter(DevCtx c, const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                  const int64_t *__restrict__ dest, int n_tokens) {
  const int piece = threadIdx.x & 15;
  const size_t rows = (size_t)n_tokens * c.Hkv;
  for (size_t row = (size_t)blockIdx.x * 16 + (threadIdx.x >> 4); row < rows; row += (size_t)gridDim.x * 16) {
    const int64_t d = dest[row];
    uint8_t *dst = c.host_pages + (size_t)(d >> 4) * kPageBytes + (size_t)(d & 15) * kRowBytes + piece * 16;
    st16(dst, ld16(reinterpret_cast<const uint8_t *>(k) + row * kRowBytes + piece * 16));
    st16(dst + kHalfPageBytes, ld16(reinterpret_cast<const uint8_t *>(v) + row * kRowBytes + piece * 16));
  }
}

// The same through a staging slot in HBM (asynchronous offload): lrow[token][head] = the row's
// place in its set's logical page order (CPU-page-table index * 16 + row); the rows whose page
// lies in [p0, p0 + m) go to the slot, laid out head-major ([head][page - p0], the order in
// which copy-engine transfers then move the pages to host memory), the others are left for
// another pass.
__global__ void __launch_bounds__(256)
k_cluster_scatter_staged(DevCtx c, const __nv_bfloat16 *__restrict__ k, const __nv_bfloat16 *__restrict__ v,
                         const int32_t *__restrict__ lrow, int n_tokens, int p0, int m, uint8_t *__restrict__ stage) {
  const int piece = threadIdx.x & 15;
  const size_t rows = (size_t)n_tokens * c.Hkv;
  for (size_t row = (size_t)blockIdx.x * 16 + (threadIdx.x >> 4); row < rows; row += (size_t)gridDim.x * 16) {
    const int32_t d = lrow[row];
    const int lp = d >> 4;
    if (lp < p0 || lp >= p0 + m) continue;
    const int head = (int)(row % c.Hkv);
    uint8_t *dst = stage + ((size_t)head * m + (lp - p0)) * kPageBytes + (size_t)(d & 15) * kRowBytes + piece * 16;
    st16(dst, ld16(reinterpret_cast<const uint8_t *>(k) + row * kRowBytes + piece * 16));
    st16(dst + kHalfPageBytes, ld16(reinterpret_cast<const uint8_t *>(v) + row * kRowBytes + piece * 16));
  }
}

// Centroids [C][Hkv][d] -> the summary rows of each head's set.
__global__ void __launch_bounds__(256)
k_copy_centroids(DevCtx c, int req, int layer, const __nv_bfloat16 *__restrict__ cen, int n_clusters) {
  const int piece = threadIdx.x & 15;
  const size_t rows = (size_t)n_clusters * c.Hkv;
  for (size_t row = (size_t)blockIdx.x * 16 + (threadIdx.x >> 4); row < rows; row += (size_t)gridDim.x * 16) {
    const int cl = (int)(row / c.Hkv), head = (int)(row % c.Hkv);
    uint8_t *s = summary_at(c, set_index(c, req, layer, head), cl);
    if (!s) { if (piece == 0) dev_error(c, 1u); continue; }
    st16(s + piece * 16, ld16(reinterpret_cast<const uint8_t *>(cen) + row * kRowBytes + piece * 16));
  }
}

// Step inputs that live in pinned host memory (q, new k/v) are brought into the staging
// buffers by one small kernel of zero-copy reads instead of one copy-engine transfer each.
__global__ void __launch_bounds__(256)
k_stage_in(uint4 *dq, const uint4 *sq, int nq, uint4 *dk, const uint4 *sk, uint4 *dv, const uint4 *sv, int nkv) {
  pdl_launch_next();
  pdl_wait_prev();
  const int total = nq + 2 * nkv;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    if (i < nq) dq[i] = sq[i];
    else if (i < nq + nkv) dk[i - nq] = sk[i - nq];
    else dv[i - nq - nkv] = sv[i - nq - nkv];
  }
}

}  // namespace

int launch_stage_in(void *dq, const void *sq, size_t q_bytes, void *dk, const void *sk, void *dv, const void *sv,
                    size_t kv_bytes, cudaStream_t st) {
  const int nq = (int)(q_bytes / 16), nkv = (int)(kv_bytes / 16);
  if (nq + nkv == 0) return 0;
  int grid = (nq + 2 * nkv + 255) / 256;
  if (grid > 64) grid = 64;
  launch_pdl(k_stage_in, dim3(grid), dim3(256), 0, st, 1, reinterpret_cast<uint4 *>(dq), reinterpret_cast<const uint4 *>(sq), nq,
             reinterpret_cast<uint4 *>(dk), reinterpret_cast<const uint4 *>(sk), reinterpret_cast<uint4 *>(dv),
             reinterpret_cast<const uint4 *>(sv), nkv);
  return 1;
}

int launch_append_bulk(const DevCtx &c, int req, int layer, const __nv_bfloat16 *k,
                       const __nv_bfloat16 *v, int first_page, int n_pages, int first_token_of_call,
                       cudaStream_t st, Prof *prof, uint8_t *stage, const int32_t *stage_hp) {
  if (n_pages <= 0) return 0;
  k_append_bulk<<<dim3(n_pages, c.Hkv), 256, 0, st>>>(c, req, layer, k, v, first_page, first_token_of_call, stage, stage_hp);
  prof_mark(prof, st, kProfAppend);
  return 1;
}

int launch_append_edge(const DevCtx &c, const AppendEdgeArgs &a, const __nv_bfloat16 *k,
                       const __nv_bfloat16 *v, int n_new, cudaStream_t st, Prof *prof) {
  launch_pdl(k_append_edge, dim3(c.Hkv, a.n_req), dim3(256), 0, st, 1, c, a, k, v, n_new);
  prof_mark(prof, st, kProfAppend);
  return 1;
}

int launch_cluster_scatter(const DevCtx &c, int req, int layer, const __nv_bfloat16 *k,
                           const __nv_bfloat16 *v, const int64_t *dest_row, int n_tokens,
                           cudaStream_t st) {
  size_t rows = (size_t)n_tokens * c.Hkv;
  int grid = (int)((rows + 15) / 16 < 148 * 16 ? (rows + 15) / 16 : 148 * 16);
  if (grid < 1) grid = 1;
  k_cluster_scatter<<<grid, 256, 0, st>>>(c, k, v, dest_row, n_tokens);
  return 1;
}

int launch_cluster_scatter_staged(const DevCtx &c, const __nv_bfloat16 *k, const __nv_bfloat16 *v, const int32_t *lrow,
                                  int n_tokens, int p0, int m, uint8_t *stage, cudaStream_t st) {
  size_t rows = (size_t)n_tokens * c.Hkv;
  int grid = (int)((rows + 15) / 16 < 148 * 16 ? (rows + 15) / 16 : 148 * 16);
  if (grid < 1) grid = 1;
  k_cluster_scatter_staged<<<grid, 256, 0, st>>>(c, k, v, lrow, n_tokens, p0, m, stage);
  return 1;
}

int launch_copy_centroids(const DevCtx &c, int req, int layer, const __nv_bfloat16 *cen,
                          int n_clusters, cudaStream_t st) {
  size_t rows = (size_t)n_clusters * c.Hkv;
  int grid = (int)((rows + 15) / 16 < 148 * 4 ? (rows + 15) / 16 : 148 * 4);
  if (grid < 1) grid = 1;
  k_copy_centroids<<<grid, 256, 0, st>>>(c, req, layer, cen, n_clusters);
  return 1;
}

}  // namespace spin
