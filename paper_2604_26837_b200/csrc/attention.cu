// Attention over the selected pages plus the local tail (Section 4.1 "Attention"): paged GQA
// decode attention, split over chunks of the page list and merged by log-sum-exp.
//
// k_attn_split: one CTA per (set, chunk of 16 pages); each warp walks pages of the chunk.
// A half-warp owns one token row at a time: lane l holds channels 8l..8l+7 of the K and V
// row (one 16-byte load each), dots them with the group's query heads, reduces over the 16
// lanes and folds the row into a running (max, sum, weighted V) per head.  A page's 8 KiB
// are requested before any arithmetic on them, so a warp keeps a whole page in flight.
// Pages are read from HBM slots, or straight from pinned host memory when bypassed.
// k_attn_merge: combines the chunks' (max, sum, output) triples and writes bf16.
#include <cstdio>

#include "../../include/spin.h"
#include "spin_dev.cuh"

namespace spin {

namespace {

constexpr int kAttnWarps = 4;
constexpr int kPartStride = kHeadDim + 2;       // per head: 128 outputs, max, sum

__device__ __forceinline__ void unpack8(uint4 raw, float *f) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = __uint_as_float(w[i] << 16);
    f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

template <int G>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn_split(DevCtx c, Batch bt, const __nv_bfloat16 *__restrict__ q) {
  __shared__ float sh[kAttnWarps][G][kPartStride];
  const int b = blockIdx.y, chunk = blockIdx.x;
  const int np = c.n_pages[b];
  const int first = chunk * kChunkPages;
  if (first >= np) return;
  const int last = min(np, first + kChunkPages);
  const int i_req = b / c.Hkv, head = b % c.Hkv;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, l16 = lane & 15, half = lane >> 4;
  const uint32_t row_mask = 0xffffu << (lane & 16);
  const size_t pl = (size_t)b * (c.max_pages + c.tail_cap);

  // logits in base 2: q is pre-scaled by sm_scale * log2(e)
  const float qs = c.sm_scale * 1.4426950408889634f;
  float qf[G][8], m[G], l[G], o[G][8];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    unpack8(*reinterpret_cast<const uint4 *>(q + ((size_t)i_req * c.Hq + head * G + g) * kHeadDim + l16 * 8), qf[g]);
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) { qf[g][i] *= qs; o[g][i] = 0.f; }
  }

  for (int pg = first + warp; pg < last; pg += kAttnWarps) {
    const uint8_t *page = page_ptr(c, c.page_src[pl + pg]);
    const uint32_t mask = c.page_mask[pl + pg];
    uint4 kraw[8], vraw[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int row = 2 * it + half;
      if ((mask >> row) & 1u) {
        kraw[it] = *reinterpret_cast<const uint4 *>(page + row * kRowBytes + l16 * 16);
        vraw[it] = *reinterpret_cast<const uint4 *>(page + kHalfPageBytes + row * kRowBytes + l16 * 16);
      }
    }
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int row = 2 * it + half;
      if (!((mask >> row) & 1u)) continue;
      float kf[8], vf[8];
      unpack8(kraw[it], kf);
      unpack8(vraw[it], vf);
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float s = qf[g][0] * kf[0];
#pragma unroll
        for (int i = 1; i < 8; ++i) s = fmaf(qf[g][i], kf[i], s);
        s += __shfl_xor_sync(row_mask, s, 1);
        s += __shfl_xor_sync(row_mask, s, 2);
        s += __shfl_xor_sync(row_mask, s, 4);
        s += __shfl_xor_sync(row_mask, s, 8);
        const float mn = fmaxf(m[g], s);
        const float corr = exp2f(m[g] - mn), p = exp2f(s - mn);
        l[g] = l[g] * corr + p;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[g][i] = fmaf(o[g][i], corr, p * vf[i]);
        m[g] = mn;
      }
    }
  }
  // fold the two half-warps, then the warps of the CTA
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m[g], 16);
    const float l2 = __shfl_xor_sync(0xffffffffu, l[g], 16);
    const float mn = fmaxf(m[g], m2);
    const float a = m[g] == -INFINITY ? 0.f : exp2f(m[g] - mn);
    const float a2 = m2 == -INFINITY ? 0.f : exp2f(m2 - mn);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float o2 = __shfl_xor_sync(0xffffffffu, o[g][i], 16);
      o[g][i] = o[g][i] * a + o2 * a2;
    }
    l[g] = l[g] * a + l2 * a2;
    m[g] = mn;
    if (half == 0) {
#pragma unroll
      for (int i = 0; i < 8; ++i) sh[warp][g][l16 * 8 + i] = o[g][i];
      if (l16 == 0) { sh[warp][g][kHeadDim] = mn; sh[warp][g][kHeadDim + 1] = l[g]; }
    }
  }
  __syncthreads();
  float *out = c.att_part + ((size_t)b * c.max_chunks + chunk) * G * kPartStride;
  for (int e = threadIdx.x; e < G * kHeadDim; e += kAttnWarps * 32) {
    const int g = e / kHeadDim, ch = e % kHeadDim;
    float mn = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) mn = fmaxf(mn, sh[w][g][kHeadDim]);
    float acc = 0.f, ls = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float mw = sh[w][g][kHeadDim];
      const float a = mw == -INFINITY ? 0.f : exp2f(mw - mn);
      acc += sh[w][g][ch] * a;
      ls += sh[w][g][kHeadDim + 1] * a;
    }
    out[g * kPartStride + ch] = acc;
    if (ch == 0) { out[g * kPartStride + kHeadDim] = mn; out[g * kPartStride + kHeadDim + 1] = ls; }
  }
}

// grid: (G, batch sets); 128 threads = channels
__global__ void __launch_bounds__(kHeadDim)
k_attn_merge(DevCtx c, Batch bt, __nv_bfloat16 *__restrict__ out) {
  const int b = blockIdx.y, g = blockIdx.x, ch = threadIdx.x;
  const int i_req = b / c.Hkv, head = b % c.Hkv;
  const int n_chunks = (c.n_pages[b] + kChunkPages - 1) / kChunkPages;
  const float *part = c.att_part + ((size_t)b * c.max_chunks * c.G + g) * kPartStride;
  const size_t stride = (size_t)c.G * kPartStride;
  float mn = -INFINITY;
  for (int k = 0; k < n_chunks; ++k) mn = fmaxf(mn, part[k * stride + kHeadDim]);
  float acc = 0.f, ls = 0.f;
  for (int k = 0; k < n_chunks; ++k) {
    const float mk = part[k * stride + kHeadDim];
    const float a = mk == -INFINITY ? 0.f : exp2f(mk - mn);
    acc += part[k * stride + ch] * a;
    ls += part[k * stride + kHeadDim + 1] * a;
  }
  const float r = ls > 0.f ? acc / ls : 0.f;
  out[((size_t)i_req * c.Hq + head * c.G + g) * kHeadDim + ch] = __float2bfloat16(r);
}

}  // namespace

int launch_attention(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q,
                     __nv_bfloat16 *out, int max_pages_hint, cudaStream_t st, Prof *prof) {
  const int n_sets = b.n_req * c.Hkv;
  int chunks = (max_pages_hint + kChunkPages - 1) / kChunkPages;
  if (chunks < 1) chunks = 1;
  if (chunks > c.max_chunks) chunks = c.max_chunks;
  dim3 grid(chunks, n_sets);
  switch (c.G) {
    case 1: k_attn_split<1><<<grid, kAttnWarps * 32, 0, st>>>(c, b, q); break;
    case 2: k_attn_split<2><<<grid, kAttnWarps * 32, 0, st>>>(c, b, q); break;
    case 4: k_attn_split<4><<<grid, kAttnWarps * 32, 0, st>>>(c, b, q); break;
    default: k_attn_split<8><<<grid, kAttnWarps * 32, 0, st>>>(c, b, q); break;
  }
  prof_mark(prof, st, kProfAttnSplit);
  k_attn_merge<<<dim3(c.G, n_sets), kHeadDim, 0, st>>>(c, b, out);
  prof_mark(prof, st, kProfAttnMerge);
  return 2;
}

}  // namespace spin

// ---------------------------------------------------------------------------------------
// Allocation-free paged attention (see spin_paged_attention_static in spin.h).
//
// The split-K partials of this variant live in a fixed array that is part of the library
// image, so a caller that must not (or cannot) allocate device memory -- code running inside
// someone else's memory budget, a latency-critical loop that may not touch the allocator, a
// plug-in that is only handed its input and output buffers -- can still run the split + merge
// pair.  Every GPU that loads the library carries these 8 MiB until the process exits.
namespace spin {
namespace {
constexpr size_t kStaticPartialFloats = (size_t)2 << 20;                  // 8 MiB of fp32
__device__ __align__(256) static float g_static_partials[kStaticPartialFloats];
constexpr int kMaxDevices = 64;
float *g_static_partials_addr[kMaxDevices] = {};                          // per device, set up once
}  // namespace
}  // namespace spin

extern "C" int spin_paged_attention_static(const void *q, const void *page_pool,
                                           const int32_t *page_ids, const uint32_t *page_masks,
                                           const int32_t *n_pages, int32_t n_sets,
                                           int32_t list_stride, int32_t group, float sm_scale,
                                           void *out, void *cuda_stream) {
  using namespace spin;
  if (!q || !page_pool || !page_ids || !page_masks || !n_pages || !out || n_sets < 1 || list_stride < 1) {
    fprintf(stderr, "spin_paged_attention_static: null pointer or non-positive size\n");
    return SPIN_ERR_INVALID;
  }
  if (group != 1 && group != 2 && group != 4 && group != 8) {
    fprintf(stderr, "spin_paged_attention_static: group must be 1, 2, 4 or 8 (got %d)\n", group);
    return SPIN_ERR_INVALID;
  }
  const int chunks = (list_stride + kChunkPages - 1) / kChunkPages;
  const size_t need = (size_t)n_sets * chunks * group * (kHeadDim + 2);
  if (need > kStaticPartialFloats) {
    fprintf(stderr,
            "spin_paged_attention_static: n_sets (%d) x ceil(list_stride/16) (%d) x group (%d) x 130 = %zu "
            "floats of split-K scratch exceed the built-in %zu; use fewer sets per call or the context API\n",
            n_sets, chunks, group, need, kStaticPartialFloats);
    return SPIN_ERR_INVALID;
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
    fprintf(stderr, "spin_paged_attention_static: no usable current CUDA device\n");
    return SPIN_ERR_CUDA;
  }
  if (!g_static_partials_addr[dev]) {
    // In host code the array's name is only a stand-in for the symbol: the address the
    // kernels can use has to be asked for, once per device, with that device current.
    float *p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void **>(&p), g_static_partials);
    if (e != cudaSuccess || !p) {
      fprintf(stderr, "spin_paged_attention_static: cudaGetSymbolAddress failed: %s\n", cudaGetErrorString(e));
      return SPIN_ERR_CUDA;
    }
    g_static_partials_addr[dev] = p;
  }
  DevCtx c{};
  c.num_layers = 1; c.Hq = group; c.Hkv = 1; c.G = group;
  c.max_pages = list_stride; c.tail_cap = 0; c.max_chunks = chunks;
  c.sm_scale = sm_scale != 0.f ? sm_scale : 0.08838834764831845f;
  c.gpu_pages = const_cast<uint8_t *>(reinterpret_cast<const uint8_t *>(page_pool));
  c.host_pages = nullptr;
  c.page_src = const_cast<int32_t *>(page_ids);
  c.page_mask = const_cast<uint32_t *>(page_masks);
  c.n_pages = const_cast<int32_t *>(n_pages);
  c.att_part = g_static_partials_addr[dev];
  Batch b{};
  b.n_req = n_sets;
  launch_attention(c, b, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out),
                   list_stride, reinterpret_cast<cudaStream_t>(cuda_stream), nullptr);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    fprintf(stderr, "spin_paged_attention_static: launch failed: %s\n", cudaGetErrorString(e));
    return SPIN_ERR_CUDA;
  }
  return SPIN_OK;
}
