// Index + Offload (Section 4.1): write appended K/V rows through to the pinned host tier,
// keep the newest page in an HBM tail page, and turn a completed page into a candidate
// partition with its summary (per-channel min/max of the keys, or the key rows themselves
// for token-granular selection).  The host runtime has already mapped the segments and
// filled the host-side tables (Partition Offset, CPU page table) for the pages touched here.
#include "spin_dev.cuh"

namespace spin {

namespace {

// 256 threads; thread t moves the 16-byte piece (t & 15) of row (t >> 4).
__device__ __forceinline__ uint4 ld16(const void *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st16(void *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

// min / max over the 16 key rows held in shared memory, per channel; bf16 compares are done
// in fp32 (exact).  Thread c < 128 handles channel c.
__device__ __forceinline__ void write_minmax(const DevCtx &c, int set, int part,
                                             const __nv_bfloat16 (*krows)[kHeadDim], int tid) {
  if (tid < kHeadDim) {
    float mn = __bfloat162float(krows[0][tid]), mx = mn;
#pragma unroll
    for (int r = 1; r < kPageTokens; ++r) {
      float x = __bfloat162float(krows[r][tid]);
      mn = fminf(mn, x);
      mx = fmaxf(mx, x);
    }
    uint8_t *s = summary_at(c, set, part);
    if (!s) { dev_error(c, 1u); return; }
    __nv_bfloat16 *o = reinterpret_cast<__nv_bfloat16 *>(s);
    o[tid] = __float2bfloat16(mn);            // exact: mn is one of the bf16 inputs
    o[kHeadDim + tid] = __float2bfloat16(mx);
  }
}

__device__ __forceinline__ void write_token_summaries(const DevCtx &c, int set, int part,
                                                      const __nv_bfloat16 (*krows)[kHeadDim], int tid) {
  uint8_t *s = summary_at(c, set, part * kPageTokens);
  if (!s) { dev_error(c, 1u); return; }
  int r = tid >> 4, piece = tid & 15;
  st16(s + r * kRowBytes + piece * 16, ld16(reinterpret_cast<const uint8_t *>(krows[r]) + piece * 16));
}

__device__ __forceinline__ void index_page(const DevCtx &c, int set, int part,
                                           const __nv_bfloat16 (*krows)[kHeadDim], int tid) {
  if (c.kind == kKindPage) write_minmax(c, set, part, krows, tid);
  else write_token_summaries(c, set, part, krows, tid);
  if (tid == 0) {
    MetaEntry *m = meta_at(c, set, part);
    if (m) { m->tokens = kPageTokens; m->resident = 0; } else dev_error(c, 1u);
  }
}

// Pages completely covered by this call's tokens that are not the newest page: all 16 rows
// come from the input; the page is written to the host tier and indexed.
__global__ void __launch_bounds__(256)
k_append_bulk(DevCtx c, int req, int layer, const __nv_bfloat16 *__restrict__ k,
              const __nv_bfloat16 *__restrict__ v, int first_page, int first_token_of_call) {
  __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
  const int head = blockIdx.y, page = first_page + blockIdx.x, tid = threadIdx.x;
  const int set = set_index(c, req, layer, head);
  const int r = tid >> 4, piece = tid & 15;
  const size_t tok = (size_t)page * kPageTokens + r - first_token_of_call;
  const size_t in_off = (tok * c.Hkv + head) * kHeadDim * 2 + piece * 16;
  uint4 kk = ld16(reinterpret_cast<const uint8_t *>(k) + in_off);
  uint4 vv = ld16(reinterpret_cast<const uint8_t *>(v) + in_off);
  const int32_t *hp = cpt_at(c, set, page);
  if (!hp) { if (tid == 0) dev_error(c, 1u); return; }
  uint8_t *dst = c.host_pages + (size_t)(*hp) * kPageBytes + r * kRowBytes + piece * 16;
  st16(dst, kk);
  st16(dst + kHalfPageBytes, vv);
  st16(reinterpret_cast<uint8_t *>(krows[r]) + piece * 16, kk);
  __syncthreads();
  index_page(c, set, page, krows, tid);
}

// The pages at the edges of an append, one CTA per set: (1) the old tail page, if this call
// completes it and moves on, is indexed from its HBM copy plus the new rows; (2) the newest
// page receives its new rows in the host tier and in the HBM tail page.  Also the only form
// needed for single-token decode appends.  k, v: [n_req][n_new][Hkv][d].
__global__ void __launch_bounds__(256)
k_append_edge(DevCtx c, AppendEdgeArgs a, const __nv_bfloat16 *__restrict__ k,
              const __nv_bfloat16 *__restrict__ v, int n_new) {
  __shared__ __align__(16) __nv_bfloat16 krows[kPageTokens][kHeadDim];
  const int head = blockIdx.x, i = blockIdx.y, tid = threadIdx.x;
  pdl_launch_next();
  pdl_wait_prev();
  const int set = set_index(c, a.req[i], a.layer, head);
  const int r = tid >> 4, piece = tid & 15;
  SetState st = c.state[set];
  const int n0 = st.n_tokens, n1 = n0 + n_new;
  const uint8_t *kin = reinterpret_cast<const uint8_t *>(k) + (size_t)i * n_new * c.Hkv * kRowBytes;
  const uint8_t *vin = reinterpret_cast<const uint8_t *>(v) + (size_t)i * n_new * c.Hkv * kRowBytes;
  auto in_off = [&](int tok) { return ((size_t)(tok - n0) * c.Hkv + head) * kRowBytes + piece * 16; };

  if (c.kind == kKindCluster) {
    // decode tokens of a clustered set only extend the always-attended tail
    int tail_pages = st.tail_pages, tail_len = st.tail_len;
    for (int tok = n0; tok < n1; ++tok) {
      if (tail_pages == 0 || tail_len == kPageTokens) { ++tail_pages; tail_len = 0; }
      if (tail_pages > c.tail_cap) { if (tid == 0) dev_error(c, 1u); break; }
      if (tid < 16) {
        const int32_t *hp = cpt_at(c, set, st.tail_first + tail_pages - 1);
        if (!hp) { dev_error(c, 1u); }
        else {
          uint4 kk = ld16(kin + in_off(tok)), vv = ld16(vin + in_off(tok));
          size_t o = (size_t)tail_len * kRowBytes + piece * 16;
          uint8_t *h = c.host_pages + (size_t)(*hp) * kPageBytes + o;
          uint8_t *g = c.gpu_pages + (size_t)c.tail_phys[(size_t)set * c.tail_cap + tail_pages - 1] * kPageBytes + o;
          st16(h, kk); st16(h + kHalfPageBytes, vv);
          st16(g, kk); st16(g + kHalfPageBytes, vv);
        }
      }
      ++tail_len;
    }
    if (tid == 0) {
      SetState *s = &c.state[set];
      s->n_tokens = n1;
      s->tail_pages = tail_pages;
      s->tail_len = tail_len;
      s->n_host_pages = st.tail_first + tail_pages;
    }
    return;
  }

  const int j0 = n0 > 0 ? (n0 - 1) / kPageTokens : -1;      // old tail page
  const int j_end = (n1 - 1) / kPageTokens;                 // newest page after the call
  uint8_t *tail = c.gpu_pages + (size_t)c.tail_phys[(size_t)set * c.tail_cap] * kPageBytes;

  if (j0 >= 0 && j0 < j_end) {
    // the old tail page is complete after this call (or was already) and stops being the tail
    const int have = n0 - j0 * kPageTokens;                 // rows already in the HBM tail page
    uint4 kk;
    if (r < have) {
      kk = ld16(tail + r * kRowBytes + piece * 16);
    } else {
      const int tok = j0 * kPageTokens + r;
      kk = ld16(kin + in_off(tok));
      uint4 vv = ld16(vin + in_off(tok));
      const int32_t *hp = cpt_at(c, set, j0);
      if (hp) {
        uint8_t *dst = c.host_pages + (size_t)(*hp) * kPageBytes + r * kRowBytes + piece * 16;
        st16(dst, kk);
        st16(dst + kHalfPageBytes, vv);
      } else if (piece == 0) dev_error(c, 1u);
    }
    st16(reinterpret_cast<uint8_t *>(krows[r]) + piece * 16, kk);
    __syncthreads();
    index_page(c, set, j0, krows, tid);
    __syncthreads();                                        // tail rows are read before rewritten
  }
  {
    const int lo = max(n0, j_end * kPageTokens) - j_end * kPageTokens;   // first new row
    const int hi = n1 - j_end * kPageTokens;                             // one past last row
    if (r >= lo && r < hi) {
      const int tok = j_end * kPageTokens + r;
      uint4 kk = ld16(kin + in_off(tok)), vv = ld16(vin + in_off(tok));
      const int32_t *hp = cpt_at(c, set, j_end);
      if (hp) {
        uint8_t *dst = c.host_pages + (size_t)(*hp) * kPageBytes + r * kRowBytes + piece * 16;
        st16(dst, kk);
        st16(dst + kHalfPageBytes, vv);
      } else if (piece == 0) dev_error(c, 1u);
      st16(tail + r * kRowBytes + piece * 16, kk);
      st16(tail + kHalfPageBytes + r * kRowBytes + piece * 16, vv);
    }
  }
  if (tid == 0) {
    SetState *s = &c.state[set];
    s->n_tokens = n1;
    s->n_partitions = j_end;
    s->n_host_pages = j_end + 1;
    s->tail_first = j_end;
    s->tail_pages = 1;
    s->tail_len = n1 - j_end * kPageTokens;
  }
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

}  // namespace

int launch_append_bulk(const DevCtx &c, int req, int layer, const __nv_bfloat16 *k,
                       const __nv_bfloat16 *v, int first_page, int n_pages, int first_token_of_call,
                       cudaStream_t st, Prof *prof) {
  if (n_pages <= 0) return 0;
  k_append_bulk<<<dim3(n_pages, c.Hkv), 256, 0, st>>>(c, req, layer, k, v, first_page, first_token_of_call);
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

int launch_copy_centroids(const DevCtx &c, int req, int layer, const __nv_bfloat16 *cen,
                          int n_clusters, cudaStream_t st) {
  size_t rows = (size_t)n_clusters * c.Hkv;
  int grid = (int)((rows + 15) / 16 < 148 * 4 ? (rows + 15) / 16 : 148 * 4);
  if (grid < 1) grid = 1;
  k_copy_centroids<<<grid, 256, 0, st>>>(c, req, layer, cen, n_clusters);
  return 1;
}

}  // namespace spin
