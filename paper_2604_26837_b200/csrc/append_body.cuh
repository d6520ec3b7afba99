// Decode-time / edge append of one set, shared by the stand-alone append kernel and by the
// scoring kernel's in-grid append CTAs (Index + Offload, Section 4.1).
#pragma once
#include "spin_dev.cuh"

namespace spin {

// The append body is run by 256 threads that may be part of a larger CTA (the streaming scoring
// kernel has a producer warp besides them): they meet at a named barrier of their own.
__device__ __forceinline__ void sync_256() { asm volatile("bar.sync 1, 256;\n" ::: "memory"); }

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

// Landmark summary (Table 1, ShadowKV's Index: mean(paged_key, dim=dim_page)): per channel the
// 16 keys are added in token order in fp32, scaled by 1/16 (exact) and rounded to bf16
// (nearest even) -- the order and rounding the CPU oracle uses.
__device__ __forceinline__ void write_mean(const DevCtx &c, int set, int part,
                                           const __nv_bfloat16 (*krows)[kHeadDim], int tid) {
  if (tid < kHeadDim) {
    float s = __bfloat162float(krows[0][tid]);
#pragma unroll
    for (int r = 1; r < kPageTokens; ++r) s = s + __bfloat162float(krows[r][tid]);
    uint8_t *dst = summary_at(c, set, part);
    if (!dst) { dev_error(c, 1u); return; }
    reinterpret_cast<__nv_bfloat16 *>(dst)[tid] = __float2bfloat16_rn(s * 0.0625f);
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
  else if (c.kind == kKindPageMean) write_mean(c, set, part, krows, tid);
  else write_token_summaries(c, set, part, krows, tid);
  if (tid == 0) {
    MetaEntry *m = meta_at(c, set, part);
    if (m) { m->tokens = kPageTokens; m->resident = 0; } else dev_error(c, 1u);
    off_mirror_set(c, set, part, part);          // page-sized kinds: partition p starts at page p
  }
}

// The pages at the edges of an append for one set, run by a 256-thread CTA: (1) the old tail
// page, if this call completes it and moves on, is indexed from its HBM copy plus the new rows;
// (2) the newest page receives its new rows in the host tier and in the HBM tail page.  Also
// the only form needed for single-token decode appends.  k, v: [n_req][n_new][Hkv][d]; `i` is
// the request's position in that array.  krows: 16 x 128 bf16 of shared memory.
__device__ __forceinline__ void append_edge_body(const DevCtx &c, int set, int i, int head,
                                                 const __nv_bfloat16 *__restrict__ k,
                                                 const __nv_bfloat16 *__restrict__ v, int n_new,
                                                 int n0_host, int epoch, __nv_bfloat16 (*krows)[kHeadDim]) {
  const int tid = threadIdx.x;
  const int r = tid >> 4, piece = tid & 15;
  SetState st = c.state[set];
  sync_256();            // every thread has read the state before thread 0 rewrites it at the end
  // the host has counted every append; its count is the one used, and a device word that
  // disagrees is reported (it is rewritten below)
  if (threadIdx.x == 0 && st.n_tokens != n0_host) {
    dev_error(c, kErrState);
    if (atomicCAS(&c.counters->dbg[0], 0u, (unsigned)set + 1u) == 0u) {
      c.counters->dbg[1] = (unsigned)st.n_tokens; c.counters->dbg[2] = (unsigned)n0_host; c.counters->dbg[3] = (unsigned)epoch;
    }
  }
  const int n0 = n0_host, n1 = n0 + n_new;
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
    sync_256();
    index_page(c, set, j0, krows, tid);
    sync_256();                                             // tail rows are read before rewritten
  }
  {
    const int lo = max(n0, j_end * kPageTokens) - j_end * kPageTokens;   // first new row
    const int hi = n1 - j_end * kPageTokens;                             // one past last row
    if (r >= lo && r < hi) {
      const int tok = j_end * kPageTokens + r;
      uint4 kk = ld16(kin + in_off(tok)), vv = ld16(vin + in_off(tok));
      const int32_t *hp = cpt_at(c, set, j_end);
      if (hp) {
        const int32_t host_page = *hp;
        uint8_t *dst = c.host_pages + (size_t)host_page * kPageBytes + r * kRowBytes + piece * 16;
        st16(dst, kk);
        st16(dst + kHalfPageBytes, vv);
        if (piece == 0 && r == lo) cpt_mirror_set(c, set, j_end, host_page);
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

}  // namespace spin
