// Retrieve (Section 5.2, lookup steps 1-4) with the bucketed-LRU replacement of Section 5.3.
//
// k_cache: one CTA per set.  It (1) reads the Meta-partition entries of the selected
// partitions (token count -> page count, residency -> hit/miss, page demand); (2) scans the
// set's GPU page table once: pages of hit partitions are promoted to top = min(step, n-1),
// all others are demoted by one once step > n-1, a shared-memory histogram of the updated
// timestamps is built (empty slots in bucket -1, hit pages left out); (3) finds the smallest
// threshold x whose cumulative count meets the demand and evicts every other page with
// ts <= x; (4) admits the missed pages into the free slots in ascending slot order, reads
// their CPU page ids from the pinned Partition Offset / CPU page tables, and queues
// (host page -> GPU page) copies.  It also lays out the page list attention will read
// (selected partitions ascending, pages in order, then the local tail).  Metadata only: the
// bytes move in k_fetch.
//
// k_fetch: persistent warp-per-page copy from pinned host memory into HBM (Section 5.5: one
// warp per page, vectorised 16-byte transactions, pages spread over all warps regardless of
// owner).
#include "spin_dev.cuh"

namespace spin {

namespace {

constexpr int kCacheThreads = 512;
enum : int { kHit = 0, kAdmit = 1, kBypass = 2 };

__device__ __forceinline__ uint32_t block_scan256(uint32_t v, uint32_t *wsum, uint32_t *total) {
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
    uint32_t x = lane < kCacheThreads / 32 ? wsum[lane] : 0, xi = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t t = __shfl_up_sync(0xffffffffu, xi, o);
      if (lane >= o) xi += t;
    }
    wsum[lane] = xi - x;
    if (lane == 31) wsum[32] = xi;
  }
  __syncthreads();
  const uint32_t res = wsum[w] + inc - v;
  *total = wsum[32];
  __syncthreads();
  return res;
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

__global__ void __launch_bounds__(kCacheThreads)
k_cache(DevCtx c, Batch bt) {
  extern __shared__ __align__(16) int32_t smem[];
  int32_t *s_parts = smem;                          // [max_parts]
  int32_t *s_tokens = s_parts + c.max_parts;        // [max_parts]
  int32_t *s_pageoff = s_tokens + c.max_parts;      // [max_parts + 1]
  int32_t *s_missoff = s_pageoff + c.max_parts + 1; // [max_parts] offset into the free list
  int32_t *s_missbefore = s_missoff + c.max_parts;  // [max_parts] missed pages of earlier partitions
  int32_t *s_state = s_missbefore + c.max_parts;    // [max_parts]
  int32_t *s_free = s_state + c.max_parts;          // [max_pages]
  uint32_t *s_hit = reinterpret_cast<uint32_t *>(s_free + c.max_pages);   // [max_slots/32]
  __shared__ uint32_t hist[kMaxBuckets + 2];
  __shared__ uint32_t wsum[33];
  __shared__ int32_t s_hostpage[kCacheThreads];      // CPU page ids of the first missed pages
  __shared__ int sh_x, sh_demand, sh_evicted, sh_qbase, sh_admit_pages,
      sh_bypass_pages;

  const int b = blockIdx.x, i_req = b / c.Hkv, head = b % c.Hkv, tid = threadIdx.x;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  pdl_launch_next();
  pdl_wait_prev();
  const SetState st = c.state[set];
  const int S = st.slots, n = c.n_buckets, t = st.step;
  const int top = min(t, n - 1);
  int np = c.n_parts[b];
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
  for (int base = 0; base < np; base += kCacheThreads) {
    const int r = base + tid;
    uint32_t npg = 0, miss = 0;
    if (r < np) {
      const int p = g_parts[r];
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
    const uint32_t ex_a = block_scan256(npg, wsum, &tot_a);
    const uint32_t ex_m = block_scan256(miss ? npg : 0, wsum, &tot_m);
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
    sh_evicted = 0;
    sh_admit_pages = 0;
    sh_bypass_pages = 0;
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
  for (int i = tid; i < (S + 31) / 32; i += kCacheThreads) s_hit[i] = 0;
  for (int i = tid; i < kMaxBuckets + 2; i += kCacheThreads) hist[i] = 0;
  __syncthreads();

  // Retrieve step 3, started early: the Partition Offset / CPU page table entries of the
  // missed pages live in pinned host memory, two dependent reads over the host link.  They
  // are issued here and consumed after the table scans below, which hides their latency.
  int early_i = 0, early_off = -1, early_host = -1;
  if (tid < demand && np > 0) {
    const int r = owner_of(s_missbefore, np, tid);
    early_i = tid - s_missbefore[r];
    const int32_t *off = off_at(c, set, s_parts[r]);
    if (off) early_off = *off;
  }

  // ---- step 2: one scan of the GPU page table: promote, demote, histogram ---------------
  for (int base = 0; base < S; base += kCacheThreads) {
    const int s = base + tid;
    int bucket = -2;                                  // -2: nothing to count (hit slot or no slot)
    GptEntry *e = s < S ? gpt_at(c, set, s) : nullptr;
    if (s < S && !e) dev_error(c, kErrBounds);
    if (e) {
      const int4 raw = *reinterpret_cast<const int4 *>(e);
      const int part = raw.x, phys = raw.y, pidx = raw.z;
      int ts = raw.w;
      if (c.trace) {
        c.evict_trace[((size_t)set * c.max_slots + s) * 2] = -1;
        c.evict_trace[((size_t)set * c.max_slots + s) * 2 + 1] = -1;
      }
      if (part < 0) {
        bucket = -1;
      } else {
        const int r = find_sorted(s_parts, np, part);
        if (r >= 0) {
          atomicOr(&s_hit[s >> 5], 1u << (s & 31));
          if (ts != top) e->ts = top;
          const int idx = s_pageoff[r] + pidx;
          page_src[idx] = phys;
          page_slot[idx] = s;
        } else {
          if (t > n - 1 && ts > 0) { --ts; e->ts = ts; }
          bucket = ts;
        }
      }
    }
    // slots of one generation share a timestamp: one lane per distinct bucket adds the count
    const uint32_t same = __match_any_sync(0xffffffffu, bucket);
    if (bucket >= -1 && (tid & 31) == __ffs(same) - 1) atomicAdd(&hist[bucket + 1], (uint32_t)__popc(same));
  }
  __syncthreads();

  if (early_off >= 0) {
    const int32_t *hp = cpt_at(c, set, early_off + early_i);
    if (hp) early_host = *hp;
  }

  // ---- step 3: threshold and eviction; free slots in ascending order --------------------
  if (tid == 0) {
    int x = -2;                                   // nothing is <= -2: no eviction
    if (demand > 0) {
      x = n - 1;
      uint32_t cum = 0;
      for (int bk = -1; bk < n; ++bk) {
        cum += hist[bk + 1];
        if ((int)cum >= demand) { x = bk; break; }
      }
    }
    sh_x = x;
  }
  __syncthreads();
  const int x = sh_x;
  uint32_t run_free = 0;
  if (demand > 0) {
    for (int base = 0; base < S; base += kCacheThreads) {
      const int s = base + tid;
      uint32_t fr = 0;
      if (s < S) {
        GptEntry *e = gpt_at(c, set, s);
        if (e) {
          const int part = e->partition;
          if (part < 0) fr = 1;
          else if (!((s_hit[s >> 5] >> (s & 31)) & 1u) && e->ts <= x) {
            MetaEntry *m = meta_at(c, set, part);
            if (m) m->resident = 0;
            if (c.trace) {
              c.evict_trace[((size_t)set * c.max_slots + s) * 2] = part;
              c.evict_trace[((size_t)set * c.max_slots + s) * 2 + 1] = e->page_idx;
            }
            e->partition = -1;
            e->page_idx = 0;
            e->ts = -1;
            atomicAdd(&sh_evicted, 1);
            fr = 1;
          }
        }
      }
      uint32_t tot;
      const uint32_t ex = block_scan256(fr, wsum, &tot);
      if (fr && run_free + ex < (uint32_t)c.max_pages) s_free[run_free + ex] = s;
      run_free += tot;
    }
  }
  __syncthreads();

  s_hostpage[tid] = early_host;

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
      sh_demand = used;
    }
  } else if (tid == 0) sh_demand = demand;
  __syncthreads();
  if (tid == 0) sh_qbase = (sh_demand > 0 && c.fetch_mode != 0) ? atomicAdd(c.fetch_count, sh_demand) : 0;
  __syncthreads();
  const int qbase = sh_qbase;

  for (int r = tid; r < np; r += kCacheThreads) {
    c.part_state[(size_t)b * c.max_parts + r] = s_state[r];
    if (s_state[r] == kAdmit) {
      MetaEntry *m = meta_at(c, set, s_parts[r]);
      if (m) m->resident = 1;
    }
  }
  int my_admit = 0, my_bypass = 0;
  for (int idx = tid; idx < total_pages; idx += kCacheThreads) {
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
    int host_page = mi < kCacheThreads ? s_hostpage[mi] : -1;
    const int32_t *hp = &host_page;
    if (host_page < 0) {                       // beyond the early batch (or it failed): look up now
      const int32_t *off = off_at(c, set, p);
      hp = off ? cpt_at(c, set, *off + i) : nullptr;
      if (hp) host_page = *hp;
    }
    if (!hp) { dev_error(c, kErrBounds); page_src[idx] = 0; page_mask[idx] = 0; page_desc[pos] = make_int4(0, -1, 0, idx); continue; }
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
        page_fill[idx] = host_page;               // the attention kernel brings it in
      } else {
        const int qi = qbase + s_missoff[r] + i;
        if (qi < c.fetch_cap) c.fetch_queue[qi] = FetchItem{host_page, phys};
        else dev_error(c, kErrBounds);
      }
      page_desc[pos] = make_int4(phys, page_fill[idx], (int)page_mask[idx], idx);
      ++my_admit;
    } else {
      page_src[idx] = ~host_page;
      page_slot[idx] = -1;
      page_desc[pos] = make_int4(~host_page, -1, (int)page_mask[idx], idx);
      ++my_bypass;
    }
  }
  if (my_admit) atomicAdd(&sh_admit_pages, my_admit);
  if (my_bypass) atomicAdd(&sh_bypass_pages, my_bypass);

  // ---- local tail: always attended -------------------------------------------------------
  for (int j = tid; j < st.tail_pages; j += kCacheThreads) {
    const int idx = total_pages + j;
    page_src[idx] = c.tail_phys[(size_t)set * c.tail_cap + j];
    page_mask[idx] = j == st.tail_pages - 1 ? ((1u << st.tail_len) - 1u) : 0xffffu;
    page_slot[idx] = -2;
    page_fill[idx] = -1;
    page_desc[idx] = make_int4(page_src[idx], -1, (int)page_mask[idx], idx);
    page_part[idx] = -1;
    page_pidx[idx] = j;
  }
  __syncthreads();
  if (tid == 0) {
    c.n_pages[b] = total_pages + st.tail_pages;
    c.n_parts[b] = np;
    c.state[set].step = t + 1;
    Counters *k = c.counters;
    const int miss_pages = sh_admit_pages + sh_bypass_pages;
    atomicAdd(&k->set_steps, 1ull);
    atomicAdd(&k->selected_partitions, (unsigned long long)np);
    atomicAdd(&k->selected_pages, (unsigned long long)total_pages);
    atomicAdd(&k->tail_pages, (unsigned long long)st.tail_pages);
    atomicAdd(&k->hit_pages, (unsigned long long)(total_pages - miss_pages));
    atomicAdd(&k->miss_pages, (unsigned long long)miss_pages);
    atomicAdd(&k->evicted_pages, (unsigned long long)sh_evicted);
    atomicAdd(&k->bypass_pages, (unsigned long long)sh_bypass_pages);
  }
}

// One warp per missed page: 8 KiB = 16 x (32 lanes x 16 B), all loads issued before the
// stores so that a warp keeps a whole page in flight on the host link.
__global__ void __launch_bounds__(256)
k_fetch(DevCtx c) {
  const int n = min(*c.fetch_count, c.fetch_cap);
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (blockDim.x >> 5);
  for (int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < n; i += warps) {
    const FetchItem it = c.fetch_queue[i];
    const uint4 *src = reinterpret_cast<const uint4 *>(c.host_pages + (size_t)it.host_page * kPageBytes) + lane;
    uint4 *dst = reinterpret_cast<uint4 *>(c.gpu_pages + (size_t)it.gpu_page * kPageBytes) + lane;
    uint4 buf[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) buf[j] = __ldcs(src + j * 32);
#pragma unroll
    for (int j = 0; j < 16; ++j) dst[j * 32] = buf[j];
  }
}

}  // namespace

size_t cache_smem_bytes(const DevCtx &c) {
  return (size_t)(6 * c.max_parts + 1 + c.max_pages) * 4 + (size_t)((c.max_slots + 31) / 32) * 4 + 16;
}

int launch_cache(const DevCtx &c, const Batch &b, cudaStream_t st, int sm_count, Prof *prof) {
  static size_t configured = 0;
  const size_t smem = cache_smem_bytes(c);
  if (smem > configured) {
    cudaFuncSetAttribute(k_cache, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = smem;
  }
  launch_pdl(k_cache, dim3(b.n_req * c.Hkv), dim3(kCacheThreads), smem, st, 1, c, b);
  prof_mark(prof, st, kProfCache);
  if (c.fetch_mode == 0) return 1;
  k_fetch<<<sm_count * 4, 256, 0, st>>>(c);
  prof_mark(prof, st, kProfFetch);
  return 2;
}

}  // namespace spin
