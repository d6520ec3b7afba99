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
#define SPIN_FILE_ID 3
#include "stages.cuh"

namespace spin {

namespace {

constexpr int kCacheThreads = 512;

// Stand-alone cache manager: one CTA per set (used when top-k ran as its own cluster kernel).
// fast != 0: every set of the batch has at most kFastSlots slots and the shared-memory layout
// fits, so the page table is staged in shared memory (cache_fast); else it is worked on in
// global memory (cache_stage).
__global__ void __launch_bounds__(kCacheThreads)
k_cache(DevCtx c, Batch bt, int fast, int tbl_cap) {
  extern __shared__ __align__(16) uint8_t dyn_smem[];
  __shared__ union { CacheShared staged; FastShared fast; } shm;
  const int b = blockIdx.x, i_req = b / c.Hkv, head = b % c.Hkv, tid = threadIdx.x;
  const int set = set_index(c, bt.req[i_req], bt.layer, head);
  pdl_launch_next();
  pdl_wait_prev();
  const int np = c.n_parts[b];
  if (!fast) {
    cache_stage<kCacheThreads>(c, b, set, np, bt.tail_pages[i_req], bt.tail_len[i_req], bt.epoch,
                               reinterpret_cast<int32_t *>(dyn_smem), shm.staged);
    return;
  }
  const int S = bt.slots[i_req];
  const FastLayout L = fast_layout(c, dyn_smem, 0, S, tbl_cap);
  fast_prefetch_dirs<kCacheThreads>(c, L, set, S);
  const int32_t *g_parts = c.parts + (size_t)b * c.max_parts;
  for (int r = tid; r < np; r += kCacheThreads) L.s_parts[r] = g_parts[r];
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  __syncthreads();
  fast_prefetch_gpt<kCacheThreads>(c, L, S);
  fast_prefetch_tables<kCacheThreads>(c, L, bt.n_partitions[i_req]);
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
  __syncthreads();
  cache_fast<kCacheThreads>(c, bt, b, i_req, set, L, np, shm.fast);
}

// Buffer elasticity (Section 5.3): shrink a request's sets from old_S to new_S slots by
// reclaiming the tail of the GPU page table.  A partition with a page in the reclaimed tail
// becomes non-resident as a whole, so its pages below the cut are cleared as well.
// One CTA per (layer, kv head) set of the request.
__global__ void __launch_bounds__(256)
k_shrink(DevCtx c, int req, int old_S, int new_S) {
  const int set = req * c.num_layers * c.Hkv + blockIdx.x, tid = threadIdx.x;
  for (int s = new_S + tid; s < old_S; s += 256) {
    const GptEntry *e = gpt_at(c, set, s);
    if (!e) { dev_error(c, kErrBounds); continue; }
    if (e->partition >= 0) {
      MetaEntry *m = meta_at(c, set, e->partition);
      if (m) m->resident = 0;
    }
  }
  __threadfence();
  __syncthreads();
  for (int s = tid; s < old_S; s += 256) {
    GptEntry *e = gpt_at(c, set, s);
    if (!e) continue;
    const int part = e->partition;
    if (part < 0) continue;
    const MetaEntry *m = meta_at(c, set, part);
    if (s >= new_S || (m && m->resident == 0)) { e->partition = -1; e->page_idx = 0; e->ts = -1; }
  }
  if (tid == 0) c.state[set].slots = new_S;
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

size_t cache_smem_bytes(const DevCtx &c) { return cache_stage_smem_bytes(c.max_parts, c.max_pages, c.max_slots); }

int launch_cache(const DevCtx &c, const Batch &b, cudaStream_t st, Prof *prof) {
  static size_t configured_dev[kMaxDevices] = {};
  size_t &configured = configured_dev[current_device_slot()];
  int tbl_cap = 0;
  size_t smem = 0;
  // one CTA per set: the snapshot of the partition tables may take what shared memory is left
  const int fast = plan_cache_fast(c, b, 200 * 1024, &tbl_cap, &smem) ? 1 : 0;
  if (!fast) smem = cache_smem_bytes(c);
  if (smem > configured) {
    cudaFuncSetAttribute(k_cache, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured = smem;
  }
  launch_pdl(k_cache, dim3(b.n_req * c.Hkv), dim3(kCacheThreads), smem, st, 1, c, b, fast, tbl_cap);
  prof_mark(prof, st, kProfCache);
  return 1;
}

// One warp waits, with the given poll limit, for a value that no kernel ever publishes (a
// negative call number) in the first set's `scored` word: the wait runs out, the timeout bit is
// set and the kernel returns.  This is how the bounded-wait path is exercised without any
// other kernel misbehaving.
__global__ void k_wait_probe(DevCtx c, int max_polls) {
  if (threadIdx.x == 0) flag_wait(c, c.scored, -1, max_polls);
}

// What the host link gives a kernel: every warp of a grid that fills the GPU reads whole pages of
// the pinned host tier (16 x 512 bytes in flight per warp, as the page fetch does) and keeps
// only a checksum.  The caller times it; nothing else is touched.
__global__ void __launch_bounds__(256)
k_link_probe(DevCtx c, int n_pages, unsigned *sink) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int n_warps = (gridDim.x * blockDim.x) >> 5;
  unsigned acc = 0;
  for (int i = warp; i < n_pages; i += n_warps) {
    const uint4 *src = reinterpret_cast<const uint4 *>(c.host_pages + (size_t)(i % c.n_host_pages) * kPageBytes) + lane;
    uint4 buf[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) buf[j] = __ldcs(src + j * 32);
#pragma unroll
    for (int j = 0; j < 16; ++j) acc ^= buf[j].x ^ buf[j].y ^ buf[j].z ^ buf[j].w;
  }
  if (acc == 0x9e3779b9u) *sink = acc;             // keeps the loads alive; practically never taken
}

int launch_link_probe(const DevCtx &c, int n_pages, cudaStream_t st, int sm_count) {
  k_link_probe<<<sm_count * 4, 256, 0, st>>>(c, n_pages, reinterpret_cast<unsigned *>(c.fetch_count));
  return 1;
}

// The least a decode step of this design can take: its two launches, chained by programmatic
// stream serialization like the step's kernels, with one flag handed from the first to the
// second and nothing else to do.
__global__ void k_floor_first(DevCtx c, int token) {
  pdl_launch_next();
  pdl_wait_prev();
  if (threadIdx.x == 0) flag_publish(c.score_done, token);
}
__global__ void k_floor_second(DevCtx c, int token) {
  pdl_launch_next();
  if (threadIdx.x == 0) {
    flag_wait(c, c.score_done, token);
    pdl_wait_prev();                                // not to complete ahead of the kernel before it
    *c.score_done = 0;                              // as the scoring kernel expects to find it
  }
}

int launch_floor(const DevCtx &c, int token, cudaStream_t st) {
  launch_pdl(k_floor_first, dim3(1), dim3(32), 0, st, 1, c, token);
  launch_pdl(k_floor_second, dim3(1), dim3(32), 0, st, 1, c, token);
  return 2;
}

int launch_wait_probe(const DevCtx &c, int max_polls, cudaStream_t st) {
  k_wait_probe<<<1, 32, 0, st>>>(c, max_polls);
  return 1;
}

int launch_shrink(const DevCtx &c, int req, int old_S, int new_S, cudaStream_t st) {
  k_shrink<<<c.num_layers * c.Hkv, 256, 0, st>>>(c, req, old_S, new_S);
  return 1;
}

int launch_fetch(const DevCtx &c, cudaStream_t st, int sm_count, Prof *prof) {
  if (c.fetch_mode == 0) return 0;
  k_fetch<<<sm_count * 4, 256, 0, st>>>(c);
  prof_mark(prof, st, kProfFetch);
  return 1;
}

}  // namespace spin
