// Attention over the selected pages plus the local tail (Section 4.1 "Attention"), fused with
// the page fetch of Retrieve step 4 (Section 5.2): paged GQA decode attention, split over
// chunks of the page list and merged by log-sum-exp.
//
// k_attn: one CTA (4 warps) per (set, chunk of 8 pages).  Each warp owns two pages of the
// chunk.  It requests both pages at once with 16-byte cp.async copies into XOR-swizzled
// shared memory (a page is one contiguous 8 KiB run: 16 K rows then 16 V rows) -- from an
// HBM slot for a hit, straight from pinned host memory for a miss -- so every missed page of
// the step is in flight on the host link while the hits are being attended from HBM.  A
// missed page that was admitted to the cache is written from shared memory into its HBM
// slot after use (that is the fetch); a bypassed page is only attended.  QK^T and PV run on
// mma.sync m16n8k16 bf16 tiles with fp32 accumulators (query heads padded to M = 16, the
// page's 16 tokens as N resp. K): at ~4 flop/byte the kernel is HBM/PCIe bound and tensor
// tiles are used to take instruction issue off the critical path, which is also why the
// 64..128-row tcgen05 tiles (>90% padding at GQA 4) are not.  The last CTA of a set to finish
// (a counter cleared by the cache-manager kernel) merges the set's partials and writes bf16.
#define SPIN_FILE_ID 4
#include <cstdio>

#include "../../include/spin.h"
#include "spin_dev.cuh"

namespace spin {

#ifdef SPIN_TIMING
__device__ unsigned long long g_dbg_ta[256][16];
__device__ __forceinline__ void dbg_ta(int b, int slot) { if (threadIdx.x == 0) { unsigned long long t; asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t)); g_dbg_ta[b & 255][slot] = t; } }
#else
__device__ __forceinline__ void dbg_ta(int, int) {}
#endif

namespace {

constexpr int kAttnWarps = 4;
constexpr int kPartStride = kHeadDim + 2;       // per head: 128 outputs, max, sum

__device__ __forceinline__ uint32_t smem_u32(const void *p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Byte offset of the 16-byte piece `chunk` (0..15) of row `row` (0..31: K rows, then V rows)
// inside a page staged in shared memory.  Pieces are XOR-swizzled by the row so that the 8
// rows an ldmatrix touches fall into 8 different bank groups.
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
  return (uint32_t)(row * kRowBytes + ((chunk ^ (row & 7)) << 4));
}

// One warp requests one page: 16 copies of 16 bytes per lane, 512 contiguous bytes per instruction.
__device__ __forceinline__ void request_page(uint32_t sdst, const uint8_t *src, int lane) {
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int piece = j * 32 + lane;              // 0..511
    const int row = piece >> 4, chunk = piece & 15;
    cp_async16(sdst + swz(row, chunk), src + (size_t)piece * 16);
  }
}

struct WarpAcc {
  float m, l;                 // running max (base-2 logits) and partial sum of this lane's row
  float o[16][4];             // 16 n-tiles of 8 channels; [.][0..1] = row lane/4, [.][2..3] = row+8 (unused, zero)
};

// Attend one staged page: S = Q K^T (16 x 16), online softmax, O += P V.
__device__ __forceinline__ void attend_page(uint32_t spage, const uint32_t (&qa)[8][2], uint32_t mask,
                                            float scale2, WarpAcc &acc, int lane) {
  float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  const int mat = lane >> 3, r8 = lane & 7;
  {
    const int token = r8 + ((mat >> 1) << 3);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4(spage + swz(token, 2 * ks + (mat & 1)), b0, b1, b2, b3);
      mma_bf16(s[0], qa[ks][0], 0u, qa[ks][1], 0u, b0, b1);
      mma_bf16(s[1], qa[ks][0], 0u, qa[ks][1], 0u, b2, b3);
    }
  }
  // this lane's row = lane/4; its tokens: nt*8 + (lane%4)*2 + {0,1}
  float p[2][2];
  float mx = -INFINITY;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int tok = nt * 8 + (lane & 3) * 2 + j;
      const float v = ((mask >> tok) & 1u) ? s[nt][j] * scale2 : -INFINITY;
      p[nt][j] = v;
      mx = fmaxf(mx, v);
    }
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
  mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
  const float mn = fmaxf(acc.m, mx);
  const float base = mn == -INFINITY ? 0.f : mn;           // all masked so far: every p is 0
  const float corr = exp2f(acc.m - base);                  // acc.m = -inf -> 0
  float psum = 0.f;
#pragma unroll
  for (int nt = 0; nt < 2; ++nt)
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      p[nt][j] = exp2f(p[nt][j] - base);
      psum += p[nt][j];
    }
  acc.l = acc.l * corr + psum;
  acc.m = mn;
  const uint32_t pa0 = pack_bf16(p[0][0], p[0][1]), pa2 = pack_bf16(p[1][0], p[1][1]);
  {
    const int token = r8 + ((mat & 1) << 3);
#pragma unroll
    for (int nb = 0; nb < 8; ++nb) {
      uint32_t b0, b1, b2, b3;
      ldmatrix_x4_trans(spage + swz(kPageTokens + token, 2 * nb + (mat >> 1)), b0, b1, b2, b3);
      acc.o[2 * nb][0] *= corr; acc.o[2 * nb][1] *= corr;
      acc.o[2 * nb + 1][0] *= corr; acc.o[2 * nb + 1][1] *= corr;
      mma_bf16(acc.o[2 * nb], pa0, 0u, pa2, 0u, b0, b1);
      mma_bf16(acc.o[2 * nb + 1], pa0, 0u, pa2, 0u, b2, b3);
    }
  }
}

// Retrieve step 4 for one admitted miss: the staged page goes to its HBM slot.
__device__ __forceinline__ void store_page(const uint8_t *spage_generic, uint8_t *dst, int lane) {
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int piece = j * 32 + lane;
    const int row = piece >> 4, chunk = piece & 15;
    *reinterpret_cast<uint4 *>(dst + (size_t)piece * 16) =
        *reinterpret_cast<const uint4 *>(spage_generic + swz(row, chunk));
  }
}

// A page that came over the host link goes to the HBM slot it was admitted to.  With an early
// descriptor (open_idx >= 0) the slot is read from page_src once the set's second flag is up
// (long since, as a rule: the page took microseconds to arrive); a bypassed page has none.
__device__ __forceinline__ void fetched_page_to_slot(const DevCtx &c, const Batch &bt, int b, size_t pl,
                                                     const uint8_t *spage_generic, int slot_page, int open_idx,
                                                     bool slots_known, int lane) {
  if (open_idx >= 0) {
    int ok = 1;
    if (!slots_known) {
      if (lane == 0) ok = flag_wait(c, c.ready + b, bt.epoch);
      ok = __shfl_sync(0xffffffffu, ok, 0);
    }
    slot_page = ok ? __ldcg(c.page_src + pl + open_idx) : -1;
    if (slot_page >= c.n_gpu_pages) { if (lane == 0) dev_error(c, kErrBounds); slot_page = -1; }
  }
  if (slot_page >= 0) store_page(spage_generic, c.gpu_pages + (size_t)slot_page * kPageBytes, lane);
}

template <int G>
__device__ __forceinline__ void attn_cta(const DevCtx &c, const Batch &bt, const __nv_bfloat16 *__restrict__ q,
                                         __nv_bfloat16 *__restrict__ out, uint8_t *smem_pages) {
  __shared__ float sh[kAttnWarps][G][kPartStride];
  __shared__ int sh_last;
  // launch order: chunk 0 of every set first (the chunks that hold the missed pages), or set by set
  const int b = bt.attn_set_major ? blockIdx.y : blockIdx.x, chunk = bt.attn_set_major ? blockIdx.x : blockIdx.y;
  const int first = chunk * kChunkPages;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int np = 0, nm = 0;                      // pages in the set's list; how many of them are early descriptors
  if (c.ready) {
    // A set raises two flags.  The first says that its missed pages are listed (the leading
    // n_miss descriptors, slot still open): a warp requests those of its pages at once, so the
    // pages cross the host link while the cache manager is still freeing slots for them.  For
    // its other pages a warp waits for the second flag (complete list) and for the tail page.
    __shared__ int sh_ok, sh_np, sh_nm;
    if (threadIdx.x == 0) {
      const int ok = flag_wait(c, c.ready1 + b, bt.epoch);
      // a count beyond the list's stride can neither read past the set's row nor leave the merge
      // waiting for chunks that no CTA of the grid owns
      sh_np = ok ? max(0, min(c.n_pages[b], c.max_pages + c.tail_cap)) : 0;
      sh_nm = ok ? c.n_miss[b] : 0;
      sh_ok = ok;
    }
    __syncthreads();
    if (!sh_ok) return;
    np = sh_np; nm = sh_nm;
  } else {
    pdl_wait_prev();
    np = max(0, min(c.n_pages[b], c.max_pages + c.tail_cap));
  }
  if (chunk == 0) dbg_ta(b, 10);
  if (first >= np) return;
  const int last = min(np, first + kChunkPages);
  const int i_req = b / c.Hkv, head = b % c.Hkv;
  const size_t pl = (size_t)b * (c.max_pages + c.tail_cap);

  // the warp's two pages.  Early descriptors lead the list, so the first page is early whenever
  // the second is.  Requests go out, and are waited for, in this order: early pages, then (after
  // the second flag) the others, of which the one that has to cross the host link comes last.
  int pg[2] = {first + warp, first + warp + kAttnWarps};
  int n_mine = (pg[0] < last) + (pg[1] < last);
  const int n_early = (n_mine >= 1 && pg[0] < nm) + (n_mine >= 2 && pg[1] < nm);
  int src[2] = {0, 0}, fill[2] = {-1, -1}, open_idx[2] = {-1, -1};
  uint32_t mask[2] = {0, 0};
  auto describe = [&](int i) {
    if (c.page_desc) {                      // work-ordered descriptors written by the cache manager
      const int4 dsc = c.page_desc[pl + pg[i]];
      src[i] = dsc.x; fill[i] = dsc.y; mask[i] = (uint32_t)dsc.z;
      const bool open = dsc.x == -3;        // early descriptor: page_src[dsc.w] names the slot later
      if (open) { open_idx[i] = dsc.w; src[i] = 0; }
      if (fill[i] == -2) {
        // Retrieve step 3 for a missed page: Partition Offset -> CPU page table, both in pinned
        // host memory (two dependent reads over the host link, all lanes read the same words)
        const int set = set_index(c, bt.req[i_req], bt.layer, head);
        const int32_t *off = off_lookup(c, set, c.page_part[pl + dsc.w]);
        const int32_t *hp = off ? cpt_lookup(c, set, *off + c.page_pidx[pl + dsc.w]) : nullptr;
        const int host_page = hp ? *hp : -1;
        if (host_page < 0) { src[i] = -1; fill[i] = c.n_host_pages; }       // fails the range check below
        else if (open || src[i] >= 0) fill[i] = host_page;                  // fetched (admitted, or not yet known)
        else { src[i] = ~host_page; fill[i] = -1; }                         // bypassed: attend from host
      }
      if (open && fill[i] < 0) { src[i] = -1; fill[i] = c.n_host_pages; }   // an early descriptor always names a host page
    } else {                                // plain lists, attended in the order given
      src[i] = c.page_src[pl + pg[i]];
      mask[i] = c.page_mask[pl + pg[i]];
    }
    // a descriptor that points outside the pools is dropped (and reported), never followed
    const bool ok = (src[i] >= 0 ? src[i] < c.n_gpu_pages : ~src[i] < c.n_host_pages) && fill[i] < c.n_host_pages;
    if (!ok) { if (lane == 0) dev_error(c, kErrBounds); src[i] = 0; fill[i] = -1; mask[i] = 0; open_idx[i] = -1; }
  };
  uint8_t *spage[2] = {smem_pages + (size_t)(2 * warp) * kPageBytes, smem_pages + (size_t)(2 * warp + 1) * kPageBytes};
  auto request = [&](int i) {
    const uint8_t *from = fill[i] >= 0 ? c.host_pages + (size_t)fill[i] * kPageBytes : page_ptr(c, src[i]);
    request_page(smem_u32(spage[i]), from, lane);
  };
  // one cp.async group per page slot, in slot order (an empty group where the warp has no page)
#pragma unroll
  for (int i = 0; i < 2; ++i)
    if (i < n_early) { describe(i); request(i); cp_async_commit(); }
  if (n_early < n_mine) {
    if (c.ready) {
      int ok = 1;
      if (lane == 0) ok = flag_wait(c, c.ready + b, bt.epoch) && flag_wait(c, c.tail_ready + b, bt.epoch);
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) n_mine = n_early;            // reported by the wait: the warp attends what it has and the CTA still arrives
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
      if (i >= n_early && i < n_mine) describe(i);
    if (n_early == 0 && n_mine == 2 && (fill[0] >= 0 || src[0] < 0) && !(fill[1] >= 0 || src[1] < 0)) {
      int t = src[0]; src[0] = src[1]; src[1] = t;
      t = fill[0]; fill[0] = fill[1]; fill[1] = t;
      t = open_idx[0]; open_idx[0] = open_idx[1]; open_idx[1] = t;
      uint32_t u = mask[0]; mask[0] = mask[1]; mask[1] = u;
    }
#pragma unroll
    for (int i = 0; i < 2; ++i)
      if (i >= n_early && i < n_mine) { request(i); cp_async_commit(); }
  }
#pragma unroll
  for (int i = 0; i < 2; ++i)
    if (i >= n_mine) cp_async_commit();
  if (chunk == 0) dbg_ta(b, 11);

  // Q as A-operand fragments: row = lane/4 (query head, zero beyond G), 8 k-steps of 16 channels
  uint32_t qa[8][2];
  {
    const int row = lane >> 2;
    const uint32_t *qrow = reinterpret_cast<const uint32_t *>(q + ((size_t)i_req * c.Hq + head * G + (row < G ? row : 0)) * kHeadDim);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qa[ks][0] = row < G ? qrow[ks * 8 + (lane & 3)] : 0u;
      qa[ks][1] = row < G ? qrow[ks * 8 + 4 + (lane & 3)] : 0u;
    }
  }
  WarpAcc acc;
  acc.m = -INFINITY;
  acc.l = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) { acc.o[i][0] = acc.o[i][1] = acc.o[i][2] = acc.o[i][3] = 0.f; }
  const float scale2 = c.sm_scale * 1.4426950408889634f;

  cp_async_wait<1>();
  __syncwarp();
  if (chunk == 0) dbg_ta(b, 12);
  if (n_mine >= 1) {
    attend_page(smem_u32(spage[0]), qa, mask[0], scale2, acc, lane);
    if (fill[0] >= 0) fetched_page_to_slot(c, bt, b, pl, spage[0], src[0], open_idx[0], n_early < 1, lane);
  }
  cp_async_wait<0>();
  __syncwarp();
  if (chunk == 0) dbg_ta(b, 13);
  if (n_mine >= 2) {
    attend_page(smem_u32(spage[1]), qa, mask[1], scale2, acc, lane);
    if (fill[1] >= 0) fetched_page_to_slot(c, bt, b, pl, spage[1], src[1], open_idx[1], n_early < 2, lane);
  }

  // row sums live in the 4 lanes of a quad
  acc.l += __shfl_xor_sync(0xffffffffu, acc.l, 1);
  acc.l += __shfl_xor_sync(0xffffffffu, acc.l, 2);
  {
    const int row = lane >> 2;
    if (row < G) {
#pragma unroll
      for (int nt = 0; nt < 16; ++nt) {
        sh[warp][row][nt * 8 + (lane & 3) * 2] = acc.o[nt][0];
        sh[warp][row][nt * 8 + (lane & 3) * 2 + 1] = acc.o[nt][1];
      }
      if ((lane & 3) == 0) { sh[warp][row][kHeadDim] = acc.m; sh[warp][row][kHeadDim + 1] = acc.l; }
    }
  }
  __syncthreads();
  const int n_chunks = (np + kChunkPages - 1) / kChunkPages;
  float *part = c.att_part + ((size_t)b * c.max_chunks + chunk) * G * kPartStride;
  for (int e = threadIdx.x; e < G * kHeadDim; e += kAttnWarps * 32) {
    const int g = e / kHeadDim, ch = e % kHeadDim;
    float mn = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) mn = fmaxf(mn, sh[w][g][kHeadDim]);
    float a_o = 0.f, a_l = 0.f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float mw = sh[w][g][kHeadDim];
      const float a = mw == -INFINITY ? 0.f : exp2f(mw - mn);
      a_o += sh[w][g][ch] * a;
      a_l += sh[w][g][kHeadDim + 1] * a;
    }
    if (n_chunks == 1) {
      // only chunk of the set: finish here
      out[((size_t)i_req * c.Hq + head * G + g) * kHeadDim + ch] = __float2bfloat16(a_l > 0.f ? a_o / a_l : 0.f);
    } else {
      part[g * kPartStride + ch] = a_o;
      if (ch == 0) { part[g * kPartStride + kHeadDim] = mn; part[g * kPartStride + kHeadDim + 1] = a_l; }
    }
  }
  if (n_chunks == 1) return;
  // the last CTA of the set to get here merges all partials (log-sum-exp)
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) sh_last = atomicAdd(&c.att_count[b], 1) == n_chunks - 1;
  __syncthreads();
  if (!sh_last) return;
  dbg_ta(b, 14);
  __threadfence();
  // merge.  Nothing here grows with the number of chunks: the per-chunk (max, sum) pairs are
  // reduced to the set's max and denominator first (a thread's pairs all belong to one head,
  // the stride being a multiple of the group), then the outputs are accumulated over tiles of
  // kMergeTile chunks whose weights exp2(m_k - m) sit in shared memory.
  constexpr int kThreads = kAttnWarps * 32, kMergeTile = 512;
  static_assert(kThreads == kHeadDim, "thread t of the merge owns channel t of every head");
  const float *parts = c.att_part + (size_t)b * c.max_chunks * G * kPartStride;
  float *s_red = reinterpret_cast<float *>(smem_pages);           // [kThreads]
  float *s_mx = s_red + kThreads;                                 // [G] the set's max per head
  float *s_den = s_mx + G;                                        // [G]
  float *s_scale = s_den + G;                                     // [kMergeTile][G]
  float *s_sum = s_scale + kMergeTile * G;                        // [kMergeTile][G] (single-tile form only)
  // A set of at most kMergeTile chunks (every decode step of the benchmark configurations) reads
  // its (max, sum) pairs from memory once, all loads of a thread in flight together; larger
  // sets take three passes over them, tile by tile.
  const bool one_tile = n_chunks <= kMergeTile;
  {
    float mx = -INFINITY;
    if (one_tile) {
#pragma unroll 4
      for (int e = threadIdx.x; e < n_chunks * G; e += kThreads) {
        const float *pp = parts + (size_t)e * kPartStride + kHeadDim;
        const float mk = __ldcg(pp), lk = __ldcg(pp + 1);
        s_scale[e] = mk;
        s_sum[e] = lk;
        mx = fmaxf(mx, mk);
      }
    } else {
      for (int e = threadIdx.x; e < n_chunks * G; e += kThreads)
        mx = fmaxf(mx, __ldcg(parts + (size_t)e * kPartStride + kHeadDim));
    }
    s_red[threadIdx.x] = mx;
    __syncthreads();
    if (threadIdx.x < G) {
      float m_ = -INFINITY;
      for (int i = threadIdx.x; i < kThreads; i += G) m_ = fmaxf(m_, s_red[i]);
      s_mx[threadIdx.x] = m_;
    }
    __syncthreads();
    const float mn = s_mx[threadIdx.x % G];
    float den = 0.f;
    if (one_tile) {
      // a thread's own entries: the chunk's maximum gives way to its weight in place
      for (int e = threadIdx.x; e < n_chunks * G; e += kThreads) {
        const float mk = s_scale[e], w = mk == -INFINITY ? 0.f : exp2f(mk - mn);
        s_scale[e] = w;
        den += mk == -INFINITY ? 0.f : s_sum[e] * w;
      }
    } else {
      for (int e = threadIdx.x; e < n_chunks * G; e += kThreads) {
        const float *pp = parts + (size_t)e * kPartStride;
        const float mk = __ldcg(pp + kHeadDim);
        den += mk == -INFINITY ? 0.f : __ldcg(pp + kHeadDim + 1) * exp2f(mk - mn);
      }
    }
    s_red[threadIdx.x] = den;
    __syncthreads();
    if (threadIdx.x < G) {
      float d_ = 0.f;
      for (int i = threadIdx.x; i < kThreads; i += G) d_ += s_red[i];
      s_den[threadIdx.x] = d_;
    }
  }
  float a_o[G];                                                   // this thread's outputs: e = tid + j * kThreads
#pragma unroll
  for (int j = 0; j < G; ++j) a_o[j] = 0.f;
  for (int k0 = 0; k0 < n_chunks; k0 += kMergeTile) {
    const int kn = min(kMergeTile, n_chunks - k0);
    __syncthreads();                                              // the previous tile's weights have been used (one tile: the weights are all written)
    if (!one_tile) {
      for (int e = threadIdx.x; e < kn * G; e += kThreads) {
        const float mk = __ldcg(parts + ((size_t)k0 * G + e) * kPartStride + kHeadDim);
        s_scale[e] = mk == -INFINITY ? 0.f : exp2f(mk - s_mx[e % G]);
      }
      __syncthreads();
    }
    // a thread's G outputs are channel `threadIdx.x` of every head: the loads of a batch of chunks
    // for all G heads are issued together (their L2 latency is paid once per batch, not once per head)
    const float *pt = parts + (size_t)k0 * G * kPartStride + threadIdx.x;
    // 64 loads in flight per thread; the last batch is padded with its last chunk at weight zero
    // (one loop, no chunk-by-chunk remainder whose loads would each wait for the one before)
    constexpr int kB = G >= 8 ? 8 : G == 4 ? 16 : 32;
#pragma unroll 1
    for (int k = 0; k < kn; k += kB) {
      float v[G][kB];
#pragma unroll
      for (int j = 0; j < G; ++j)
#pragma unroll
        for (int i = 0; i < kB; ++i) v[j][i] = __ldcg(pt + ((size_t)min(k + i, kn - 1) * G + j) * kPartStride);
#pragma unroll
      for (int j = 0; j < G; ++j)
#pragma unroll
        for (int i = 0; i < kB; ++i) {
          const float w = k + i < kn ? s_scale[(k + i) * G + j] : 0.f;
          a_o[j] = fmaf(v[j][i], w, a_o[j]);
        }
    }
  }
#pragma unroll
  for (int j = 0; j < G; ++j) {
    const int e = threadIdx.x + j * kThreads, g = e / kHeadDim, ch = e % kHeadDim;
    const float den = s_den[g];
    out[((size_t)i_req * c.Hq + head * G + g) * kHeadDim + ch] = __float2bfloat16(den > 0.f ? a_o[j] / den : 0.f);
  }
  dbg_ta(b, 15);
}

// The kernel: the CTA's work; one CTA then waits for the kernel before this one.  CTAs that
// go by the per-set flags never wait for the scoring kernel as a whole; with one CTA doing so
// before it exits, this grid cannot complete ahead of that one, and whatever the stream runs
// next (the next step's scoring kernel waits for this grid) comes after all of its writes.
template <int G>
__global__ void __launch_bounds__(kAttnWarps * 32)
k_attn(DevCtx c, Batch bt, const __nv_bfloat16 *__restrict__ q, __nv_bfloat16 *__restrict__ out) {
  extern __shared__ __align__(128) uint8_t smem_pages[];          // [8][8192]
  pdl_launch_next();
  attn_cta<G>(c, bt, q, out, smem_pages);
  if (blockIdx.x == 0 && blockIdx.y == 0) pdl_wait_prev();
}

// Sets whose page list is empty get a zero output (no CTA of k_attn reaches them).
__global__ void k_attn_zero_empty(DevCtx c, __nv_bfloat16 *__restrict__ out, int n_sets) {
  const int b = blockIdx.x;
  if (b >= n_sets || c.n_pages[b] > 0) return;
  const int i_req = b / c.Hkv, head = b % c.Hkv;
  for (int e = threadIdx.x; e < c.G * kHeadDim; e += blockDim.x)
    out[((size_t)i_req * c.Hq + head * c.G) * kHeadDim + e] = __float2bfloat16(0.f);
}

template <int G>
void launch_attn_g(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q, __nv_bfloat16 *out, dim3 grid,
                   cudaStream_t st) {
  static bool configured_dev[kMaxDevices] = {};
  bool &configured = configured_dev[current_device_slot()];
  constexpr int smem = kChunkPages * kPageBytes;
  if (!configured) {
    cudaFuncSetAttribute(k_attn<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaFuncSetAttribute(k_attn<G>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    configured = true;
  }
  launch_pdl(k_attn<G>, grid, dim3(kAttnWarps * 32), (size_t)smem, st, 1, c, b, q, out);
}

}  // namespace

int launch_attention(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q,
                     __nv_bfloat16 *out, int max_pages_hint, bool may_be_empty, cudaStream_t st, Prof *prof) {
  const int n_sets = b.n_req * c.Hkv;
  int chunks = (max_pages_hint + kChunkPages - 1) / kChunkPages;
  if (chunks < 1) chunks = 1;
  if (chunks > c.max_chunks) chunks = c.max_chunks;
  dim3 grid(n_sets, chunks);
  if (b.attn_set_major) grid = dim3(chunks, n_sets);
  int launched = 1;
  if (may_be_empty) { k_attn_zero_empty<<<n_sets, 128, 0, st>>>(c, out, n_sets); ++launched; }
  switch (c.G) {
    case 1: launch_attn_g<1>(c, b, q, out, grid, st); break;
    case 2: launch_attn_g<2>(c, b, q, out, grid, st); break;
    case 4: launch_attn_g<4>(c, b, q, out, grid, st); break;
    default: launch_attn_g<8>(c, b, q, out, grid, st); break;
  }
  prof_mark(prof, st, kProfAttnSplit);
  return launched;
}

}  // namespace spin

// ---------------------------------------------------------------------------------------
// Allocation-free paged attention (see spin_paged_attention_static in spin.h).
//
// The split-K partials and arrival counters of this variant live in a fixed array that is part of the library
// image, so a caller that must not (or cannot) allocate device memory -- code running inside
// someone else's memory budget, a latency-critical loop that may not touch the allocator, a
// plug-in that is only handed its input and output buffers -- can still run the split + merge
// pair.  Every GPU that loads the library carries these 8 MiB until the process exits.
namespace spin {
namespace {
constexpr size_t kStaticPartialFloats = (size_t)2 << 20;                  // 8 MiB of fp32
__device__ __align__(256) static float g_static_partials[kStaticPartialFloats];
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
  // layout of the built-in array: [n_sets] arrival counters (as int32), then the partials
  const size_t counter_floats = ((size_t)n_sets + 63) / 64 * 64;
  const size_t need = counter_floats + (size_t)n_sets * chunks * group * (kHeadDim + 2);
  if (need > kStaticPartialFloats) {
    fprintf(stderr,
            "spin_paged_attention_static: n_sets (%d) x ceil(list_stride/8) (%d) x group (%d) x 130 partial "
            "floats + %zu counters = %zu exceed the built-in %zu; use fewer sets per call or the context API\n",
            n_sets, chunks, group, counter_floats, need, kStaticPartialFloats);
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
  c.n_gpu_pages = 0x7fffffff;                               // the caller vouches for the ids
  c.n_host_pages = 0;
  c.page_src = const_cast<int32_t *>(page_ids);
  c.page_mask = const_cast<uint32_t *>(page_masks);
  c.n_pages = const_cast<int32_t *>(n_pages);
  c.page_fill = nullptr;                                    // every listed page is already in the pool
  c.page_desc = nullptr;                                    // the lists are attended in the order given
  c.ready = nullptr;                                        // plain stream order: no per-set flags
  c.tail_ready = nullptr;
  c.ready1 = nullptr;
  c.n_miss = nullptr;
  c.att_count = reinterpret_cast<int32_t *>(g_static_partials_addr[dev]);
  c.att_part = g_static_partials_addr[dev] + counter_floats;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  // the array still holds the previous call's counters: they are the one thing that must
  // start at zero (a memset of library memory, not an allocation)
  cudaError_t e = cudaMemsetAsync(c.att_count, 0, counter_floats * sizeof(float), st);
  if (e != cudaSuccess) {
    fprintf(stderr, "spin_paged_attention_static: clearing the counters failed: %s\n", cudaGetErrorString(e));
    return SPIN_ERR_CUDA;
  }
  Batch b{};
  b.n_req = n_sets;
  launch_attention(c, b, reinterpret_cast<const __nv_bfloat16 *>(q), reinterpret_cast<__nv_bfloat16 *>(out),
                   list_stride, true, st, nullptr);
  e = cudaGetLastError();
  if (e != cudaSuccess) {
    fprintf(stderr, "spin_paged_attention_static: launch failed: %s\n", cudaGetErrorString(e));
    return SPIN_ERR_CUDA;
  }
  return SPIN_OK;
}

#ifdef SPIN_TIMING
extern "C" __attribute__((visibility("default"))) int spin_debug_timestamps_attn(unsigned long long *out) {
  cudaDeviceSynchronize();
  return (int)cudaMemcpyFromSymbol(out, spin::g_dbg_ta, sizeof(unsigned long long) * 256 * 16);
}
#endif
