// Device-side data layout shared by the kernels and the host runtime.
//
// A "set" is one (request, layer, kv head).  Everything a set owns in HBM is reached from
// its SetState and its five directories (two-level indexing, Section 5.4): a directory entry
// names a fixed-size second-level segment in a shared pool; segments are mapped on demand by
// the host runtime's bitmap allocators, so metadata grows with the mapped pages.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spin {

constexpr int kHeadDim = 128;
constexpr int kPageTokens = 16;
constexpr int kRowBytes = kHeadDim * 2;                     // one K or V row, bf16
constexpr int kHalfPageBytes = kPageTokens * kRowBytes;     // K half or V half: 4 KiB
constexpr int kPageBytes = 2 * kHalfPageBytes;              // K rows then V rows: 8 KiB
constexpr int kMaxBatch = 256;                              // requests per decode step
constexpr int kMaxBuckets = 64;

enum : int { kKindPage = 0, kKindToken = 1, kKindCluster = 2, kKindPageMean = 3 };
// sticky device error bits (same values as SPIN_DEV_ERR_* of the public header)
constexpr unsigned kErrBounds = 1u, kErrPageList = 2u, kErrTimeout = 4u, kErrState = 8u;
constexpr int kChunkPages = 8;                              // pages per attention split

// Per-set scalars (device resident, updated only by kernels).
struct SetState {
  int32_t n_tokens;       // tokens appended
  int32_t n_partitions;   // indexed partitions = rows of the Meta-partition table
  int32_t n_host_pages;   // entries of the set's CPU page table
  int32_t tail_first;     // CPU-page-table index of the first tail page
  int32_t tail_pages;     // tail pages (0/1 for the page-sized kinds)
  int32_t tail_len;       // tokens in the newest tail page
  int32_t step;           // decode steps done
  int32_t slots;          // S: GPU page table entries
};

// Meta-partition table entry (GPU): token count + residency (Section 5.2).
struct MetaEntry { int32_t tokens; int32_t resident; };
// GPU page table entry: page-centric (slot -> owner) with the recency timestamp.
struct GptEntry { int32_t partition; int32_t phys; int32_t page_idx; int32_t ts; };

struct Counters {
  unsigned long long set_steps, selected_partitions, selected_pages, tail_pages, hit_pages,
      miss_pages, evicted_pages, bypass_pages, candidates_scored;
  unsigned int error_bits;
  unsigned int first_site;   // where the first device-side error was raised (file id * 100000 + line)
  unsigned int dbg[4];       // payload of the first state mismatch: set, device value, host value, epoch
};

struct FetchItem { int32_t host_page; int32_t gpu_page; };

// Everything a kernel needs to find its data; passed by value (fits the 4 KiB param space
// together with a Batch).
struct DevCtx {
  // geometry
  int32_t num_layers, Hq, Hkv, G, kind, topk, n_buckets, trace;
  int32_t seg_shift;            // log2(entries per metadata segment)
  int32_t sum_shift;            // log2(entries per summary segment)
  int32_t sum_entry_bytes;      // 512 (min+max) or 256 (key / centroid)
  int32_t dir_part, dir_slot, dir_page, dir_sum;   // directory lengths per set
  int32_t max_sel, max_parts, max_pages, tail_cap; // scratch strides per batch set
  int32_t max_cand;             // score stride per batch set
  float sm_scale;
  // pools
  int32_t n_gpu_pages, n_host_pages;   // pool sizes, for range checks
  uint8_t *gpu_pages;           // HBM KV pages (cache slots + tails)
  uint8_t *host_pages;          // pinned host KV pages (device-visible address)
  uint8_t *summaries;           // summary segments (64 KiB each)
  MetaEntry *meta_pool;         // GPU
  GptEntry *gpt_pool;           // GPU
  int32_t *off_pool;            // pinned host: Partition Offset table segments
  int32_t *cpt_pool;            // pinned host: CPU page table segments
  int32_t *off_mirror;          // HBM copies of the two host tables (same segment layout), or null:
  int32_t *cpt_mirror;          //   what the decode kernels read, kept up to date by the append kernels
  // per set
  SetState *state;
  int32_t *dir_meta, *dir_gpt, *dir_off, *dir_cpt, *dir_sumseg;
  int32_t *tail_phys;           // [set][tail_cap] GPU pages of the tail
  int32_t *evict_trace;         // [set][max_slots][2] (trace only)
  int32_t max_slots;
  // per-step scratch, indexed by batch set b = i_req * Hkv + head
  float *scores;                // [b][max_cand]
  float *score_xfer;            // [b][max_cand] hand-over buffer of the streaming scoring kernel: all words hold the
                                //   "not written" pattern between steps; the set's selection takes a score out
                                //   (into `scores`) and puts the pattern back
  int32_t *sel_ids;             // [b][max_sel]   chosen candidates, ascending
  int32_t *n_sel;               // [b]
  int32_t *parts;               // [b][max_parts] partitions for the cache manager
  uint32_t *part_mask;          // [b][max_parts] token masks (token kind)
  int32_t *part_state;          // [b][max_parts] 0 hit / 1 admitted / 2 bypassed
  int32_t *n_parts;             // [b]
  int32_t *page_src;            // [b][max_pages+tail_cap] >=0 GPU page, <0 ~host page
  uint32_t *page_mask;          // [b][...]
  int32_t *page_fill;           // [b][...] host page to copy into page_src first, or -1
  int4 *page_desc;              // [b][...] attention's work list, misses first: {page_src, page_fill, mask, list index}
  int32_t *page_slot;           // [b][...] set-local slot / -1 bypass / -2 tail
  int32_t *page_part;           // [b][...] owning partition (-1 tail)
  int32_t *page_pidx;           // [b][...]
  int32_t *n_pages;             // [b]
  FetchItem *fetch_queue;       // misses of the whole batch
  int32_t *fetch_count;
  int32_t fetch_cap;
  float *att_part;              // split-K partials [b][max_chunks][G][kHeadDim + 2]
  int32_t *att_count;           // [b] chunks of the set that have finished (zero before attention)
  int32_t *sel_count;           // [b] scoring CTAs of the set that have finished (zero between steps)
  int32_t *score_queue;         // next work item of the resident scoring grid (zero between steps)
  int32_t *score_done;          // CTAs of that grid that have left (zero between steps)
  int32_t *scored;              // [b] epoch of the last step whose scores are complete (stand-alone top-k waits on it)
  int32_t *ready;               // [b] epoch of the last step whose page list is complete
  int32_t *tail_ready;          // [b] epoch of the last step whose appended rows are in the tail page
  int32_t *ready1;              // [b] epoch of the last step whose missed pages are listed (before their slots are known)
  int32_t *n_miss;              // [b] leading descriptors of the page list that may be followed once ready1 is set
  int32_t max_chunks;
  int32_t fetch_mode;           // 0: misses are fetched by the attention kernel; 1: by k_fetch
  int32_t evict_exact;          // 1: exact-demand eviction variant (see spin_config)
  int32_t resident_scoring;     // 0 automatic, 1 always, -1 never (see spin_config)
  Counters *counters;
};

struct Batch {
  int32_t n_req;
  int32_t layer;
  int32_t req[kMaxBatch];
  // local tail of each request after this step's append, as the host has counted it: lets
  // the cache manager lay out the page list without waiting for the append kernel
  int16_t tail_pages[kMaxBatch];
  int16_t tail_len[kMaxBatch];
  // what the host knows of every request's sets without asking the device (all kv heads of a
  // request and layer agree): GPU slots, decode steps done, indexed partitions
  int32_t slots[kMaxBatch];
  int32_t step[kMaxBatch];
  int32_t n_partitions[kMaxBatch];
  int32_t n_tokens[kMaxBatch];   // tokens before this step's append
  int32_t epoch;            // number of this decode call: value of the ready flags it sets
  int32_t append_in_grid;   // the scoring kernel's tail CTAs append this step's tokens
  int32_t attn_set_major;   // attention CTAs ordered set by set (sets become ready one after the
                            // other over a long scoring phase) instead of chunk 0 of every set first
};

__host__ __device__ inline int set_index(const DevCtx &c, int req, int layer, int head) {
  return (req * c.num_layers + layer) * c.Hkv + head;
}

#ifdef __CUDACC__
// Records the error bits and, for the first error only, where it was raised (source file id *
// 100000 + line), so that a sticky bit can be traced to its check.
__device__ __forceinline__ void dev_error_site(const DevCtx &c, unsigned bits, unsigned site) {
  if (!c.counters) return;                       // a caller without a context has no status words
  atomicOr(&c.counters->error_bits, bits);
  atomicCAS(&c.counters->first_site, 0u, site);
}
#ifndef SPIN_FILE_ID
#define SPIN_FILE_ID 0
#endif
#define dev_error(c, bits) dev_error_site((c), (bits), (unsigned)(SPIN_FILE_ID * 100000 + __LINE__))
// Two-level lookups.  A negative directory entry means "not mapped": the caller gets nullptr
// and records a bounds error instead of touching memory.
__device__ __forceinline__ MetaEntry *meta_at(const DevCtx &c, int set, int p) {
  int seg = c.dir_meta[(size_t)set * c.dir_part + (p >> c.seg_shift)];
  return seg < 0 ? nullptr : c.meta_pool + ((size_t)seg << c.seg_shift) + (p & ((1 << c.seg_shift) - 1));
}
__device__ __forceinline__ GptEntry *gpt_at(const DevCtx &c, int set, int s) {
  int seg = c.dir_gpt[(size_t)set * c.dir_slot + (s >> c.seg_shift)];
  return seg < 0 ? nullptr : c.gpt_pool + ((size_t)seg << c.seg_shift) + (s & ((1 << c.seg_shift) - 1));
}
__device__ __forceinline__ int32_t *off_at(const DevCtx &c, int set, int p) {
  int seg = c.dir_off[(size_t)set * c.dir_part + (p >> c.seg_shift)];
  return seg < 0 ? nullptr : c.off_pool + ((size_t)seg << c.seg_shift) + (p & ((1 << c.seg_shift) - 1));
}
__device__ __forceinline__ int32_t *cpt_at(const DevCtx &c, int set, int i) {
  int seg = c.dir_cpt[(size_t)set * c.dir_page + (i >> c.seg_shift)];
  return seg < 0 ? nullptr : c.cpt_pool + ((size_t)seg << c.seg_shift) + (i & ((1 << c.seg_shift) - 1));
}
// Lookups for the decode path: the HBM mirror when there is one, else the pinned host table.
__device__ __forceinline__ const int32_t *off_lookup(const DevCtx &c, int set, int p) {
  int seg = c.dir_off[(size_t)set * c.dir_part + (p >> c.seg_shift)];
  if (seg < 0) return nullptr;
  return (c.off_mirror ? c.off_mirror : c.off_pool) + ((size_t)seg << c.seg_shift) + (p & ((1 << c.seg_shift) - 1));
}
__device__ __forceinline__ const int32_t *cpt_lookup(const DevCtx &c, int set, int i) {
  int seg = c.dir_cpt[(size_t)set * c.dir_page + (i >> c.seg_shift)];
  if (seg < 0) return nullptr;
  return (c.cpt_mirror ? c.cpt_mirror : c.cpt_pool) + ((size_t)seg << c.seg_shift) + (i & ((1 << c.seg_shift) - 1));
}
// Append-side helpers: record an entry of a host table in its HBM mirror.
__device__ __forceinline__ void off_mirror_set(const DevCtx &c, int set, int p, int32_t v) {
  if (!c.off_mirror) return;
  int seg = c.dir_off[(size_t)set * c.dir_part + (p >> c.seg_shift)];
  if (seg >= 0) c.off_mirror[((size_t)seg << c.seg_shift) + (p & ((1 << c.seg_shift) - 1))] = v;
}
__device__ __forceinline__ void cpt_mirror_set(const DevCtx &c, int set, int i, int32_t v) {
  if (!c.cpt_mirror) return;
  int seg = c.dir_cpt[(size_t)set * c.dir_page + (i >> c.seg_shift)];
  if (seg >= 0) c.cpt_mirror[((size_t)seg << c.seg_shift) + (i & ((1 << c.seg_shift) - 1))] = v;
}
__device__ __forceinline__ uint8_t *summary_at(const DevCtx &c, int set, int e) {
  int seg = c.dir_sumseg[(size_t)set * c.dir_sum + (e >> c.sum_shift)];
  return seg < 0 ? nullptr
                 : c.summaries + (((size_t)seg << c.sum_shift) + (e & ((1 << c.sum_shift) - 1))) *
                                     (size_t)c.sum_entry_bytes;
}
// Programmatic dependent launch: the kernels of a decode step are launched back to back with
// the "programmatic stream serialization" attribute, so a kernel's CTAs may become resident
// while the previous kernel drains.  pdl_launch_next() lets the next kernel start launching;
// pdl_wait_prev() blocks until the previous kernel has completed and its writes are visible.
// Every kernel launched this way calls pdl_wait_prev() before it reads or writes anything
// another kernel touches.
__device__ __forceinline__ void pdl_launch_next() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait_prev() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Per-set flags that let the attention kernel start on a set as soon as that set's page list
// is complete, while the scoring kernel is still working on other sets.  The producer is
// always resident before a consumer can exist (the consumer kernel is launched with
// programmatic stream serialization after every producer CTA has started), so a consumer only
// ever waits for work that is already running.  The wait is bounded all the same: it gives up
// after ~0.1 s, reports SPIN_DEV_ERR_TIMEOUT and the CTA returns without touching the set.
__device__ __forceinline__ void flag_publish(int32_t *flag, int32_t value) {
  // a release store: everything this thread has written or observed (through the CTA barrier
  // before the call: the other threads' writes too) is visible to whoever acquires the flag
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(value) : "memory");
}
constexpr int kFlagWaitPolls = 1 << 19;          // ~0.1 s of polls at the capped back-off
__device__ __forceinline__ bool flag_wait(const DevCtx &c, const int32_t *flag, int32_t value,
                                          int max_polls = kFlagWaitPolls) {
  // polls back off from 32 ns to 256 ns: hundreds of waiting CTAs should not keep the L2
  // lines of the flags busy, and a raised flag should still be seen within a fraction of a
  // microsecond
  unsigned pause = 32;
  for (int spin = 0; spin < max_polls; ++spin) {
    int32_t v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(flag) : "memory");
    if (v == value) return true;
    __nanosleep(pause);
    if (pause < 256) pause <<= 1;
  }
  dev_error(c, kErrTimeout);
  return false;
}

// Scores handed from the streaming scoring kernel to a set's selection without a fence: a score
// is one naturally aligned 4-byte store, so the word itself says whether it has arrived.  The
// buffer holds kScoreUnset (a NaN pattern no finite computation produces) in every word between
// steps; the reader polls a word until it differs (bounded), copies it and restores the pattern.
constexpr uint32_t kScoreUnset = 0xffffffffu;
__device__ __forceinline__ float take_score(const DevCtx &c, float *xfer) {
  uint32_t v = kScoreUnset;
  for (int spin = 0; spin < (1 << 20); ++spin) {
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(xfer) : "memory");
    if (v != kScoreUnset) break;
    __nanosleep(64);
  }
  if (v == kScoreUnset) { dev_error(c, kErrTimeout); v = 0u; }
  *reinterpret_cast<uint32_t *>(xfer) = kScoreUnset;
  return __uint_as_float(v);
}

__device__ __forceinline__ const uint8_t *page_ptr(const DevCtx &c, int src) {
  return src >= 0 ? c.gpu_pages + (size_t)src * kPageBytes : c.host_pages + (size_t)(~src) * kPageBytes;
}
#endif

// Function attributes (opt-in shared memory), occupancy and SM counts are properties of a device:
// what a launcher remembers about them is kept per device ordinal (the current device, which a
// launcher's caller has made the stream's device).
constexpr int kMaxDevices = 64;
inline int current_device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
  return dev % kMaxDevices;
}

// Optional per-kernel timing: an event after every launch; durations are read afterwards.
enum : int { kProfAppend = 0, kProfScore, kProfTopk, kProfCache, kProfFetch, kProfAttnSplit,
             kProfAttnMerge, kProfKernels };
struct Prof {
  bool on = false;
  static constexpr size_t kMaxMarks = 1 << 15;
  cudaEvent_t *ev = nullptr;       // kMaxMarks events, created on first use
  int *id = nullptr;               // kernel that ended at mark i (-1 = start of a sequence)
  size_t used = 0;
  void mark(cudaStream_t st, int kernel);
};
inline void prof_mark(Prof *p, cudaStream_t st, int kernel) { if (p && p->on) p->mark(st, kernel); }

// Launch with programmatic stream serialization (and optionally a cluster size).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              int cluster_x, Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[na].val.programmaticStreamSerializationAllowed = 1;
  ++na;
  if (cluster_x > 1) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = cluster_x;
    attr[na].val.clusterDim.y = 1;
    attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = attr;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- kernel launchers (each returns the number of kernels it launched) -----------------
struct AppendEdgeArgs {     // one (request) per entry; all its kv heads are processed
  int32_t n_req, layer;
  int32_t req[kMaxBatch];
  int32_t n_tokens[kMaxBatch];   // tokens of the request before this append, as the host has counted them
};
int launch_append_bulk(const DevCtx &c, int req, int layer, const __nv_bfloat16 *k,
                       const __nv_bfloat16 *v, int first_page, int n_pages, int first_token_of_call,
                       cudaStream_t st, Prof *prof, uint8_t *stage = nullptr, const int32_t *stage_hp = nullptr);
int launch_append_edge(const DevCtx &c, const AppendEdgeArgs &a, const __nv_bfloat16 *k,
                       const __nv_bfloat16 *v, int n_new, cudaStream_t st, Prof *prof);
int launch_cluster_scatter(const DevCtx &c, int req, int layer, const __nv_bfloat16 *k,
                           const __nv_bfloat16 *v, const int64_t *dest_row, int n_tokens,
                           cudaStream_t st);
int launch_cluster_scatter_staged(const DevCtx &c, const __nv_bfloat16 *k, const __nv_bfloat16 *v, const int32_t *lrow,
                                  int n_tokens, int p0, int m, uint8_t *stage, cudaStream_t st);
int launch_stage_in(void *dq, const void *sq, size_t q_bytes, void *dk, const void *sk, void *dv, const void *sv,
                    size_t kv_bytes, cudaStream_t st);
int launch_copy_centroids(const DevCtx &c, int req, int layer, const __nv_bfloat16 *cen,
                          int n_clusters, cudaStream_t st);
int launch_select(const DevCtx &c, Batch &b, const __nv_bfloat16 *q, const __nv_bfloat16 *k_new,
                  const __nv_bfloat16 *v_new, int max_cand, cudaStream_t st, Prof *prof);
int launch_cache(const DevCtx &c, const Batch &b, cudaStream_t st, Prof *prof);
int launch_fetch(const DevCtx &c, cudaStream_t st, int sm_count, Prof *prof);
int launch_shrink(const DevCtx &c, int req, int old_S, int new_S, cudaStream_t st);
int launch_wait_probe(const DevCtx &c, int max_polls, cudaStream_t st);
int launch_floor(const DevCtx &c, int token, cudaStream_t st);
int launch_link_probe(const DevCtx &c, int n_pages, cudaStream_t st, int sm_count);
int launch_assign(const DevCtx &c, int req, int layer, int n_clusters, int n_tokens, int32_t *assign, cudaStream_t st);
int launch_move_rows(const DevCtx &c, int req, int layer, const int64_t *dest, int n_tokens, cudaStream_t st);
int launch_reindex_apply(const DevCtx &c, int req, int layer, int n_clusters, int n_folded_pages, int tail_first,
                         int tail_pages, int tail_len, int n_host_pages, const int32_t *new_tokens,
                         const uint32_t *touched, cudaStream_t st);
size_t cache_smem_bytes(const DevCtx &c);
int launch_attention(const DevCtx &c, const Batch &b, const __nv_bfloat16 *q,
                     __nv_bfloat16 *out, int max_pages_hint, bool may_be_empty, cudaStream_t st, Prof *prof);

}  // namespace spin
