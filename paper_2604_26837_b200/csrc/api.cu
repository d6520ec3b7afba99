// Host runtime behind the C ABI: context, bitmap-allocated pools (GPU pages, host pages, the
// second-level segments of the four mapping tables, summary segments), the host-side part of
// Index/Offload (which pages and segments an append touches) and the per-step launch sequence.
// All decisions that need the tables' contents are taken on the GPU; the host only tracks
// counts it can derive from the calls it has seen, so no call in the decode loop synchronises.
#define SPIN_FILE_ID 5
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "../../include/spin.h"
#include "spin_dev.cuh"

using namespace spin;

namespace {

// Lowest-free-bit-first bitmap allocator (Section 5.4: "lightweight bitmap allocator").
struct BitmapPool {
  std::vector<uint64_t> bits;
  int64_t n = 0, in_use = 0, hint = 0;
  void init(int64_t count) { n = count; bits.assign((size_t)((count + 63) / 64), 0); in_use = 0; hint = 0; }
  int64_t alloc() {
    for (int64_t w = hint; w < (int64_t)bits.size(); ++w) {
      if (bits[(size_t)w] != ~0ull) {
        int b = __builtin_ctzll(~bits[(size_t)w]);
        int64_t id = w * 64 + b;
        if (id >= n) return -1;
        bits[(size_t)w] |= 1ull << b;
        ++in_use;
        hint = w;
        return id;
      }
    }
    return -1;
  }
  void release(int64_t id) {
    if (id < 0 || id >= n) return;
    uint64_t m = 1ull << (id & 63);
    if (bits[(size_t)(id >> 6)] & m) { bits[(size_t)(id >> 6)] &= ~m; --in_use; }
    if ((id >> 6) < hint) hint = id >> 6;
  }
  int64_t available() const { return n - in_use; }
};

struct SetHost {                     // host mirror of one (request, layer, kv head)
  std::vector<int32_t> dir_meta, dir_gpt, dir_off, dir_cpt, dir_sum;
  std::vector<int32_t> gpu_pages;    // physical pages behind the slots
  std::vector<int32_t> host_pages;   // CPU page table mirror (logical page -> host page)
  std::vector<int32_t> cl_tokens;    // cluster granularity: tokens of every cluster
};

struct LayerHost {                   // counts shared by the kv-head sets of (request, layer)
  int64_t n_tokens = 0;
  int32_t steps = 0;                 // decode steps done
  int32_t n_partitions = 0, n_host_pages = 0, tail_first = 0, tail_pages = 0, tail_len = 0;
  bool clustered = false;
  int32_t last_batch_pos = -1;
};

struct RequestHost {
  bool open = false;
  int64_t slots = 0;
  std::vector<LayerHost> layers;
};

struct Geometry {
  int64_t n_sets, pages_per_set, parts_per_set, max_slots, max_cand;
  int32_t seg, seg_shift, sum_entries, sum_shift, sum_entry_bytes;
  int32_t dir_part, dir_slot, dir_page, dir_sum;
  int32_t max_sel, max_parts, max_pages, tail_cap, max_chunks, max_batch_sets;
  int64_t n_gpu_pages_total, n_gpt_segs, n_meta_segs, n_off_segs, n_cpt_segs, n_sum_segs;
  int64_t fetch_cap, stage_tokens;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ilog2(int64_t x) { int s = 0; while ((1ll << s) < x) ++s; return s; }

int compute_geometry(const spin_config &cfg, Geometry &g, std::string &err) {
  auto bad = [&](const char *m) { err = m; return (int)SPIN_ERR_INVALID; };
  if (cfg.struct_size != sizeof(spin_config)) return bad("spin_config.struct_size mismatch");
  if (cfg.head_dim != kHeadDim) return bad("head_dim must be 128");
  if (cfg.page_tokens != kPageTokens) return bad("page_tokens must be 16");
  if (cfg.num_layers < 1 || cfg.num_kv_heads < 1 || cfg.num_q_heads < 1) return bad("bad head/layer counts");
  if (cfg.num_q_heads % cfg.num_kv_heads) return bad("num_q_heads must be a multiple of num_kv_heads");
  const int G = cfg.num_q_heads / cfg.num_kv_heads;
  if (G != 1 && G != 2 && G != 4 && G != 8) return bad("group size must be 1, 2, 4 or 8");
  if (cfg.max_requests < 1 || cfg.max_requests > kMaxBatch) return bad("max_requests must be 1..256");
  if (cfg.max_context_tokens < 1 || cfg.max_context_tokens > (1ll << 26)) return bad("bad max_context_tokens");
  if (cfg.partition_kind < 0 || cfg.partition_kind > 3) return bad("bad partition_kind");
  if (cfg.topk < 1 || cfg.topk > 4096) return bad("topk must be 1..4096");
  if (cfg.lru_buckets < 1 || cfg.lru_buckets > kMaxBuckets) return bad("lru_buckets must be 1..64");
  if (cfg.gpu_cache_pages < 0 || cfg.host_pages < 1) return bad("bad page counts");
  if (cfg.offload_stage_bytes < 0 || (cfg.offload_stage_bytes > 0 &&
      cfg.offload_stage_bytes / 4 / kPageBytes < cfg.num_kv_heads))
    return bad("offload_stage_bytes must be 0 or hold at least 4 pages of every kv head");
  const bool cluster = cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID;
  if (cluster && cfg.num_clusters < 1) return bad("num_clusters must be >= 1 for the cluster kind");
  g.seg = cfg.segment_entries ? cfg.segment_entries : 256;
  if (g.seg < 16 || g.seg > 65536 || (g.seg & (g.seg - 1))) return bad("segment_entries must be a power of two in 16..65536");
  g.seg_shift = ilog2(g.seg);
  g.n_sets = (int64_t)cfg.max_requests * cfg.num_layers * cfg.num_kv_heads;
  const int64_t ctx_pages = (cfg.max_context_tokens + kPageTokens - 1) / kPageTokens;
  g.tail_cap = cluster ? (int32_t)std::max<int64_t>(1, (cfg.max_tail_tokens + kPageTokens - 1) / kPageTokens) : 1;
  g.pages_per_set = cluster ? ctx_pages + cfg.num_clusters + g.tail_cap + 1 : ctx_pages + 1;
  g.parts_per_set = cluster ? cfg.num_clusters : g.pages_per_set;
  // a budget beyond the set's own page count is never useful, but small sets may ask for it
  g.max_slots = std::max<int64_t>(1, std::min<int64_t>(std::max<int64_t>(g.pages_per_set, 256), cfg.gpu_cache_pages));
  g.sum_entries = cfg.partition_kind == SPIN_PART_PAGE_MINMAX ? 128 : 256;
  g.sum_shift = ilog2(g.sum_entries);
  g.sum_entry_bytes = cfg.partition_kind == SPIN_PART_PAGE_MINMAX ? 2 * kRowBytes : kRowBytes;
  int64_t cand = cfg.partition_kind == SPIN_PART_TOKEN_DOT ? g.pages_per_set * kPageTokens : g.parts_per_set;
  g.max_cand = (cand + g.sum_entries - 1) / g.sum_entries * g.sum_entries;
  g.dir_part = (int32_t)((g.parts_per_set + g.seg - 1) / g.seg);
  g.dir_slot = (int32_t)((g.max_slots + g.seg - 1) / g.seg);
  g.dir_page = (int32_t)((g.pages_per_set + g.seg - 1) / g.seg);
  g.dir_sum = (int32_t)(g.max_cand / g.sum_entries);
  g.max_sel = cfg.topk;
  g.max_parts = cfg.topk;
  g.max_pages = cluster ? (cfg.max_selected_pages > 0 ? cfg.max_selected_pages : cfg.topk * 16) : cfg.topk;
  g.max_chunks = (g.max_pages + g.tail_cap + kChunkPages - 1) / kChunkPages;
  g.max_batch_sets = cfg.max_requests * cfg.num_kv_heads;
  g.n_gpu_pages_total = cfg.gpu_cache_pages + g.n_sets * g.tail_cap;
  g.n_gpt_segs = (cfg.gpu_cache_pages + g.seg - 1) / g.seg + g.n_sets;
  if (cluster) {
    g.n_meta_segs = g.n_sets * g.dir_part;
    g.n_sum_segs = g.n_sets * g.dir_sum;
  } else {
    g.n_meta_segs = (cfg.host_pages + g.seg - 1) / g.seg + g.n_sets;
    int64_t entries = cfg.partition_kind == SPIN_PART_TOKEN_DOT ? cfg.host_pages * kPageTokens : cfg.host_pages;
    g.n_sum_segs = (entries + g.sum_entries - 1) / g.sum_entries + g.n_sets;
  }
  g.n_off_segs = g.n_meta_segs;
  g.n_cpt_segs = (cfg.host_pages + g.seg - 1) / g.seg + g.n_sets;
  g.fetch_cap = (int64_t)g.max_batch_sets * g.max_pages;
  g.stage_tokens = 2048;
  if ((size_t)(6 * g.max_parts + 1 + g.max_pages) * 4 + (size_t)((g.max_slots + 31) / 32) * 4 > 200 * 1024)
    return bad("topk / max_selected_pages / budget too large for the cache kernel's shared memory");
  return SPIN_OK;
}

struct Arena {                       // carves the caller's hbm_pool; with base == nullptr it only sizes
  uint8_t *base = nullptr;
  size_t off = 0;
  template <typename T> T *take(size_t count) {
    off = align_up(off, 256);
    T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
    off += count * sizeof(T);
    return p;
  }
};

}  // namespace

struct spin_ctx {
  spin_config cfg{};
  Geometry g{};
  DevCtx d{};
  std::string err;
  BitmapPool gpu_page_pool, host_page_pool, gpt_segs, meta_segs, off_segs, cpt_segs, sum_segs;
  std::vector<RequestHost> reqs;
  std::vector<SetHost> sets;
  uint8_t *host_base = nullptr;      // pinned allocation
  size_t host_bytes = 0;
  int32_t *h_off_pool = nullptr, *h_cpt_pool = nullptr;   // host views of the pinned tables
  uint8_t *h_pages = nullptr;
  // staging for host-pointer arguments
  __nv_bfloat16 *stage_q = nullptr, *stage_out = nullptr, *stage_k = nullptr, *stage_v = nullptr;
  int64_t *stage_dest = nullptr;
  int sm_count = 148;
  uint64_t launches = 0;
  size_t dir_bytes_in_use = 0;
  Prof prof;
  int32_t epoch = 0;                 // decode calls so far (value of the per-set ready flags)
  uint32_t floor_calls = 0;          // spin_debug_launch_floor calls (their flag values)
  // asynchronous offload: a ring of kOffloadSlots staging slots in HBM, drained by copy-engine
  // transfers on offload_stream; slot i is free again once ev_done[i] has happened
  static constexpr int kOffloadSlots = 4;
  uint8_t *offload_stage = nullptr;
  int32_t *offload_hp = nullptr;     // per staged unit: its host page id (what the kernel records in the mirror)
  int32_t *offload_lrow = nullptr;   // cluster prefill: row places of one prefill's tokens (see prefill_clustered)
  int64_t offload_slot_units = 0;    // (page, kv head) units of 8 KiB per slot; 0 = write-through
  cudaStream_t offload_stream = nullptr;
  cudaEvent_t ev_staged[kOffloadSlots] = {}, ev_done[kOffloadSlots] = {};
  bool slot_used[kOffloadSlots] = {};
  int offload_next = 0, offload_last = -1;
  uint64_t offload_gen = 0, offload_waited_gen = 0;
  cudaStream_t offload_waited_stream = nullptr;
};

namespace {

int fail(spin_ctx *c, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (c) c->err = buf;
  return code;
}

#define CK(call)                                                                         \
  do {                                                                                   \
    cudaError_t e_ = (call);                                                             \
    if (e_ != cudaSuccess)                                                               \
      return fail(ctx, SPIN_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));  \
  } while (0)

void carve(Arena &a, const spin_config &cfg, const Geometry &g, DevCtx &d, spin_ctx *ctx) {
  const int G = cfg.num_q_heads / cfg.num_kv_heads;
  d.gpu_pages = a.take<uint8_t>((size_t)g.n_gpu_pages_total * kPageBytes);
  d.summaries = a.take<uint8_t>((size_t)g.n_sum_segs * g.sum_entries * g.sum_entry_bytes);
  d.meta_pool = a.take<MetaEntry>((size_t)g.n_meta_segs * g.seg);
  d.gpt_pool = a.take<GptEntry>((size_t)g.n_gpt_segs * g.seg);
  if (!cfg.host_tables_only) {
    d.off_mirror = a.take<int32_t>((size_t)g.n_off_segs * g.seg);
    d.cpt_mirror = a.take<int32_t>((size_t)g.n_cpt_segs * g.seg);
  }
  d.state = a.take<SetState>((size_t)g.n_sets);
  d.dir_meta = a.take<int32_t>((size_t)g.n_sets * g.dir_part);
  d.dir_off = a.take<int32_t>((size_t)g.n_sets * g.dir_part);
  d.dir_gpt = a.take<int32_t>((size_t)g.n_sets * g.dir_slot);
  d.dir_cpt = a.take<int32_t>((size_t)g.n_sets * g.dir_page);
  d.dir_sumseg = a.take<int32_t>((size_t)g.n_sets * g.dir_sum);
  d.tail_phys = a.take<int32_t>((size_t)g.n_sets * g.tail_cap);
  d.evict_trace = cfg.trace ? a.take<int32_t>((size_t)g.n_sets * g.max_slots * 2) : nullptr;
  const size_t B = (size_t)g.max_batch_sets, PL = (size_t)(g.max_pages + g.tail_cap);
  d.scores = a.take<float>(B * g.max_cand);
  d.score_xfer = a.take<float>(B * g.max_cand);
  d.sel_ids = a.take<int32_t>(B * g.max_sel);
  d.n_sel = a.take<int32_t>(B);
  d.parts = a.take<int32_t>(B * g.max_parts);
  d.part_mask = a.take<uint32_t>(B * g.max_parts);
  d.part_state = a.take<int32_t>(B * g.max_parts);
  d.n_parts = a.take<int32_t>(B);
  d.page_src = a.take<int32_t>(B * PL);
  d.page_mask = a.take<uint32_t>(B * PL);
  d.page_fill = a.take<int32_t>(B * PL);
  d.page_desc = a.take<int4>(B * PL);
  d.page_slot = a.take<int32_t>(B * PL);
  d.page_part = a.take<int32_t>(B * PL);
  d.page_pidx = a.take<int32_t>(B * PL);
  d.n_pages = a.take<int32_t>(B);
  d.fetch_queue = a.take<FetchItem>((size_t)g.fetch_cap);
  d.fetch_count = a.take<int32_t>(1);
  d.att_part = a.take<float>(B * g.max_chunks * G * (kHeadDim + 2));
  d.att_count = a.take<int32_t>(B);
  d.sel_count = a.take<int32_t>(B);
  d.score_queue = a.take<int32_t>(1);
  d.score_done = a.take<int32_t>(1);
  d.scored = a.take<int32_t>(B);
  d.ready = a.take<int32_t>(B);
  d.tail_ready = a.take<int32_t>(B);
  d.ready1 = a.take<int32_t>(B);
  d.n_miss = a.take<int32_t>(B);
  d.counters = a.take<Counters>(1);
  __nv_bfloat16 *sq = a.take<__nv_bfloat16>((size_t)cfg.max_requests * cfg.num_q_heads * kHeadDim);
  __nv_bfloat16 *so = a.take<__nv_bfloat16>((size_t)cfg.max_requests * cfg.num_q_heads * kHeadDim);
  const size_t stage_rows = (size_t)std::max<int64_t>(g.stage_tokens, cfg.max_requests) * cfg.num_kv_heads;
  __nv_bfloat16 *sk = a.take<__nv_bfloat16>(stage_rows * kHeadDim);
  __nv_bfloat16 *sv = a.take<__nv_bfloat16>(stage_rows * kHeadDim);
  int64_t *sd = a.take<int64_t>(stage_rows);
  if (ctx) { ctx->stage_q = sq; ctx->stage_out = so; ctx->stage_k = sk; ctx->stage_v = sv; ctx->stage_dest = sd; }
  if (cfg.offload_stage_bytes > 0) {
    const int64_t units = cfg.offload_stage_bytes / spin_ctx::kOffloadSlots / kPageBytes;
    uint8_t *os = a.take<uint8_t>((size_t)units * spin_ctx::kOffloadSlots * kPageBytes);
    int32_t *oh = a.take<int32_t>((size_t)units * spin_ctx::kOffloadSlots);
    // cluster granularity: where every (token, head) row of a prefill goes in its set's page order
    int32_t *ol = cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID
                      ? a.take<int32_t>((size_t)cfg.max_context_tokens * cfg.num_kv_heads) : nullptr;
    if (ctx) { ctx->offload_stage = os; ctx->offload_hp = oh; ctx->offload_slot_units = units; ctx->offload_lrow = ol; }
  }
}

size_t host_bytes_needed(const Geometry &g, const spin_config &cfg) {
  size_t b = align_up((size_t)cfg.host_pages * kPageBytes, 4096);
  b += align_up((size_t)g.n_off_segs * g.seg * 4, 4096);
  b += align_up((size_t)g.n_cpt_segs * g.seg * 4, 4096);
  return b;
}

// 0: device memory; 1: pinned (or registered) host memory, *alias = the address kernels can use;
// 2: ordinary host memory
int classify_ptr(const void *p, const void **alias) {
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return 2; }
  if (at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged) { if (alias) *alias = p; return 0; }
  if (at.type == cudaMemoryTypeHost && at.devicePointer) { if (alias) *alias = at.devicePointer; return 1; }
  return 2;
}

bool is_device_ptr(const void *p) {
  cudaPointerAttributes at{};
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return false; }
  return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

inline SetHost &set_of(spin_ctx *ctx, int req, int layer, int head) {
  return ctx->sets[(size_t)set_index(ctx->d, req, layer, head)];
}

// Map the second-level segment holding entry `idx` of one table if it is not mapped yet, and
// push the directory entry to the device (stream ordered).  Returns the segment or -1.
int ensure_seg(spin_ctx *ctx, BitmapPool &pool, std::vector<int32_t> &dir, int32_t *dev_dir_row,
               int64_t idx, int shift, cudaStream_t st) {
  const size_t di = (size_t)(idx >> shift);
  if (di >= dir.size()) return -1;
  if (dir[di] < 0) {
    int64_t s = pool.alloc();
    if (s < 0) return -1;
    dir[di] = (int32_t)s;
    ctx->dir_bytes_in_use += 4;
    if (cudaMemcpyAsync(dev_dir_row + di, &dir[di], 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return -1;
  }
  return dir[di];
}

int validate_req_layer(spin_ctx *ctx, int req, int layer) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (req < 0 || req >= ctx->cfg.max_requests) return fail(ctx, SPIN_ERR_INVALID, "request id %d out of range", req);
  if (!ctx->reqs[(size_t)req].open) return fail(ctx, SPIN_ERR_STATE, "request %d is not open", req);
  if (layer < 0 || layer >= ctx->cfg.num_layers) return fail(ctx, SPIN_ERR_INVALID, "layer %d out of range", layer);
  return SPIN_OK;
}

// Host-side Index/Offload bookkeeping of the page-sized kinds for one (request, layer) that
// grows from n0 to n1 tokens: allocate host pages, fill CPU page table / Partition Offset
// entries, map the segments the kernels will write.
int grow_paged(spin_ctx *ctx, int req, int layer, int64_t n1, cudaStream_t st) {
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  const int64_t n0 = L.n_tokens;
  if (n1 > ctx->cfg.max_context_tokens) return fail(ctx, SPIN_ERR_INVALID, "request %d exceeds max_context_tokens", req);
  const int64_t first_new_page = n0 == 0 ? 0 : (n0 - 1) / kPageTokens + 1;
  const int64_t j_end = (n1 - 1) / kPageTokens;
  const int64_t new_pages = j_end - first_new_page + 1;
  if (new_pages > 0 && ctx->host_page_pool.available() < new_pages * ctx->cfg.num_kv_heads)
    return fail(ctx, SPIN_ERR_OOM_HOST, "out of host pages");
  for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
    const int set = set_index(d, req, layer, h);
    SetHost &S = ctx->sets[(size_t)set];
    for (int64_t j = first_new_page; j <= j_end; ++j) {
      int seg = ensure_seg(ctx, ctx->cpt_segs, S.dir_cpt, d.dir_cpt + (size_t)set * g.dir_page, j, g.seg_shift, st);
      if (seg < 0) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
      const int64_t hp = ctx->host_page_pool.alloc();
      ctx->h_cpt_pool[((size_t)seg << g.seg_shift) + (j & (g.seg - 1))] = (int32_t)hp;
      S.host_pages.push_back((int32_t)hp);
    }
    // partitions L.n_partitions .. j_end-1 get indexed by this call
    for (int64_t p = L.n_partitions; p < j_end; ++p) {
      if (ensure_seg(ctx, ctx->meta_segs, S.dir_meta, d.dir_meta + (size_t)set * g.dir_part, p, g.seg_shift, st) < 0)
        return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of Meta-partition segments");
      int seg = ensure_seg(ctx, ctx->off_segs, S.dir_off, d.dir_off + (size_t)set * g.dir_part, p, g.seg_shift, st);
      if (seg < 0) return fail(ctx, SPIN_ERR_OOM_HOST, "out of Partition Offset segments");
      ctx->h_off_pool[((size_t)seg << g.seg_shift) + (p & (g.seg - 1))] = (int32_t)p;
      const int64_t e = ctx->cfg.partition_kind == SPIN_PART_TOKEN_DOT ? p * kPageTokens : p;
      if (ensure_seg(ctx, ctx->sum_segs, S.dir_sum, d.dir_sumseg + (size_t)set * g.dir_sum, e, g.sum_shift, st) < 0)
        return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of summary segments");
    }
  }
  L.n_tokens = n1;
  L.n_partitions = (int32_t)j_end;
  L.n_host_pages = (int32_t)j_end + 1;
  L.tail_first = (int32_t)j_end;
  L.tail_pages = 1;
  L.tail_len = (int32_t)(n1 - j_end * kPageTokens);
  return SPIN_OK;
}

// Decode tokens of a clustered (request, layer): they extend the tail.
int grow_cluster_tail(spin_ctx *ctx, int req, int layer, int64_t n_new, cudaStream_t st) {
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  if (L.n_tokens + n_new > ctx->cfg.max_context_tokens) return fail(ctx, SPIN_ERR_INVALID, "request %d exceeds max_context_tokens", req);
  for (int64_t i = 0; i < n_new; ++i) {
    if (L.tail_pages == 0 || L.tail_len == kPageTokens) {
      if (L.tail_pages + 1 > g.tail_cap) return fail(ctx, SPIN_ERR_INVALID, "request %d exceeds max_tail_tokens", req);
      if (ctx->host_page_pool.available() < ctx->cfg.num_kv_heads) return fail(ctx, SPIN_ERR_OOM_HOST, "out of host pages");
      for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
        const int set = set_index(d, req, layer, h);
        SetHost &S = ctx->sets[(size_t)set];
        const int64_t j = L.tail_first + L.tail_pages;
        int seg = ensure_seg(ctx, ctx->cpt_segs, S.dir_cpt, d.dir_cpt + (size_t)set * g.dir_page, j, g.seg_shift, st);
        if (seg < 0) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
        const int64_t hp = ctx->host_page_pool.alloc();
        ctx->h_cpt_pool[((size_t)seg << g.seg_shift) + (j & (g.seg - 1))] = (int32_t)hp;
        S.host_pages.push_back((int32_t)hp);
      }
      ++L.tail_pages;
      L.tail_len = 0;
    }
    ++L.tail_len;
    ++L.n_tokens;
  }
  L.n_host_pages = L.tail_first + L.tail_pages;
  return SPIN_OK;
}

// Pages still on their way to host memory must have arrived before `st` reads the host tier
// (a decode step's fetch) or hands host pages back (request close).  The library's stream is
// in order, so the newest drain event covers all earlier ones.
int wait_for_offload(spin_ctx *ctx, cudaStream_t st) {
  if (ctx->offload_last < 0) return SPIN_OK;
  if (ctx->offload_gen == ctx->offload_waited_gen && st == ctx->offload_waited_stream) return SPIN_OK;
  CK(cudaStreamWaitEvent(st, ctx->ev_done[ctx->offload_last], 0));
  ctx->offload_waited_gen = ctx->offload_gen;
  ctx->offload_waited_stream = st;
  return SPIN_OK;
}

// One more token for each listed request of one layer: everything that could make grow_paged /
// grow_cluster_tail fail is checked here for the whole batch, before any of them runs, so that
// a refused call leaves the host's counts (and with them the device's) untouched.
int precheck_append_one(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req) {
  const Geometry &g = ctx->g;
  const bool cluster = ctx->cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID;
  int64_t new_pages = 0, cpt = 0, meta = 0, off = 0, sum = 0;      // host pages and table segments the batch needs
  auto unmapped = [](const std::vector<int32_t> &dir, int64_t idx, int shift) {
    const size_t di = (size_t)(idx >> shift);
    return di < dir.size() && dir[di] < 0 ? 1 : 0;
  };
  for (int i = 0; i < n_req; ++i) {
    const LayerHost &L = ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer];
    if (cluster && !L.clustered) return fail(ctx, SPIN_ERR_STATE, "request %d has no cluster prefill yet", req_ids[i]);
    if (L.n_tokens + 1 > ctx->cfg.max_context_tokens)
      return fail(ctx, SPIN_ERR_INVALID, "request %d exceeds max_context_tokens", req_ids[i]);
    const bool page_starts = cluster ? (L.tail_pages == 0 || L.tail_len == kPageTokens) : L.n_tokens % kPageTokens == 0;
    if (!page_starts) continue;
    if (cluster && L.tail_pages + 1 > g.tail_cap) return fail(ctx, SPIN_ERR_INVALID, "request %d exceeds max_tail_tokens", req_ids[i]);
    new_pages += ctx->cfg.num_kv_heads;
    for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
      const SetHost &S = set_of(ctx, req_ids[i], layer, h);
      const int64_t j = cluster ? (int64_t)L.tail_first + L.tail_pages : L.n_tokens / kPageTokens;   // the new page
      cpt += unmapped(S.dir_cpt, j, g.seg_shift);
      if (!cluster && j > L.n_partitions) {
        // the page before it becomes a candidate: one entry in the partition tables, its summaries
        const int64_t p = j - 1;
        meta += unmapped(S.dir_meta, p, g.seg_shift);
        off += unmapped(S.dir_off, p, g.seg_shift);
        sum += unmapped(S.dir_sum, ctx->cfg.partition_kind == SPIN_PART_TOKEN_DOT ? p * kPageTokens : p, g.sum_shift);
      }
    }
  }
  if (ctx->host_page_pool.available() < new_pages) return fail(ctx, SPIN_ERR_OOM_HOST, "out of host pages");
  if (ctx->cpt_segs.available() < cpt) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
  if (ctx->off_segs.available() < off) return fail(ctx, SPIN_ERR_OOM_HOST, "out of Partition Offset segments");
  if (ctx->meta_segs.available() < meta) return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of Meta-partition segments");
  if (ctx->sum_segs.available() < sum) return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of summary segments");
  return SPIN_OK;
}

int append_paged_device(spin_ctx *ctx, int req, int layer, const __nv_bfloat16 *k, const __nv_bfloat16 *v,
                        int64_t n, cudaStream_t st) {
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  const int64_t n0 = L.n_tokens;
  const int64_t j0 = n0 > 0 ? (n0 - 1) / kPageTokens : -1;
  int rc = grow_paged(ctx, req, layer, n0 + n, st);
  if (rc) return rc;
  const int64_t j_end = (n0 + n - 1) / kPageTokens;
  // pages strictly between the old tail page and the newest page: complete, all rows new
  const int64_t first = j0 + 1, nb = j_end - first;
  if (ctx->offload_slot_units > 0 && nb > 0) {
    // asynchronous offload: slot by slot through the staging ring (see spin_ctx)
    const int64_t per = ctx->offload_slot_units / ctx->cfg.num_kv_heads;
    for (int64_t p = 0; p < nb; p += per) {
      const int m = (int)std::min<int64_t>(per, nb - p), slot = ctx->offload_next;
      ctx->offload_next = (slot + 1) % spin_ctx::kOffloadSlots;
      if (ctx->slot_used[slot]) CK(cudaStreamWaitEvent(st, ctx->ev_done[slot], 0));     // ring full: wait for the drain
      uint8_t *stage = ctx->offload_stage + (size_t)slot * ctx->offload_slot_units * kPageBytes;
      int32_t *hp = ctx->offload_hp + (size_t)slot * ctx->offload_slot_units;
      {
        // the pages' host ids come with the call (head-major like the slot): while copy-engine
        // transfers own the host link, a kernel's small reads of the pinned CPU page table
        // would wait behind them
        std::vector<int32_t> ids((size_t)m * ctx->cfg.num_kv_heads);
        for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
          const std::vector<int32_t> &hpv = set_of(ctx, req, layer, h).host_pages;
          for (int i = 0; i < m; ++i) ids[(size_t)h * m + i] = hpv[(size_t)(first + p + i)];
        }
        CK(cudaMemcpyAsync(hp, ids.data(), ids.size() * 4, cudaMemcpyHostToDevice, st));   // pageable source: staged before the call returns
      }
      ctx->launches += launch_append_bulk(ctx->d, req, layer, k, v, (int)(first + p), m, (int)n0, st, &ctx->prof, stage, hp);
      CK(cudaEventRecord(ctx->ev_staged[slot], st));
      CK(cudaStreamWaitEvent(ctx->offload_stream, ctx->ev_staged[slot], 0));
      // The slot is laid out head-major, the order in which host pages were handed out, so a
      // head's pages are as a rule one run of consecutive host pages: one copy-engine transfer
      // per run, no SM involved (a fragmented host pool means more and shorter transfers).
      const int H = ctx->cfg.num_kv_heads;
      for (int h = 0; h < H; ++h) {
        const std::vector<int32_t> &hpv = set_of(ctx, req, layer, h).host_pages;
        for (int i = 0; i < m;) {
          int len = 1;
          while (i + len < m && hpv[(size_t)(first + p + i + len)] == hpv[(size_t)(first + p + i)] + len) ++len;
          CK(cudaMemcpyAsync(ctx->h_pages + (size_t)hpv[(size_t)(first + p + i)] * kPageBytes,
                             stage + ((size_t)h * m + i) * kPageBytes, (size_t)len * kPageBytes,
                             cudaMemcpyDeviceToHost, ctx->offload_stream));
          i += len;
        }
      }
      CK(cudaEventRecord(ctx->ev_done[slot], ctx->offload_stream));
      ctx->slot_used[slot] = true;
      ctx->offload_last = slot;
      ++ctx->offload_gen;
    }
  } else {
    ctx->launches += launch_append_bulk(ctx->d, req, layer, k, v, (int)first, (int)nb, (int)n0, st, &ctx->prof);
  }
  AppendEdgeArgs a{};
  a.n_req = 1;
  a.layer = layer;
  a.req[0] = req;
  a.n_tokens[0] = (int32_t)n0;
  ctx->launches += launch_append_edge(ctx->d, a, k, v, (int)n, st, &ctx->prof);
  return SPIN_OK;
}

int prefill_clustered(spin_ctx *ctx, int req, int layer, const void *k, const void *v, int64_t n,
                      const int32_t *token_partition, const void *centroids, cudaStream_t st) {
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  const int H = ctx->cfg.num_kv_heads, C = ctx->cfg.num_clusters;
  if (L.n_tokens != 0) return fail(ctx, SPIN_ERR_STATE, "cluster prefill must be the first append of (request, layer)");
  if (n > ctx->cfg.max_context_tokens) return fail(ctx, SPIN_ERR_INVALID, "prefill exceeds max_context_tokens");
  CK(cudaStreamSynchronize(st));
  // partition specification on the host
  std::vector<int32_t> tp((size_t)n * H);
  CK(cudaMemcpy(tp.data(), token_partition, tp.size() * 4, cudaMemcpyDefault));
  std::vector<int32_t> count((size_t)H * C, 0);
  for (int64_t t = 0; t < n; ++t)
    for (int h = 0; h < H; ++h) {
      const int32_t c = tp[(size_t)t * H + h];
      if (c < 0 || c >= C) return fail(ctx, SPIN_ERR_INVALID, "token_partition[%lld][%d] = %d out of range", (long long)t, h, c);
      ++count[(size_t)h * C + c];
    }
  int64_t pages_needed = 0;
  for (size_t i = 0; i < count.size(); ++i) pages_needed += (count[i] + kPageTokens - 1) / kPageTokens;
  if (ctx->host_page_pool.available() < pages_needed) return fail(ctx, SPIN_ERR_OOM_HOST, "out of host pages");
  std::vector<int32_t> first_row_page((size_t)H * C);       // CPU-page-table offset of each cluster
  std::vector<MetaEntry> meta((size_t)C);
  int32_t total_pages_max = 0;
  for (int h = 0; h < H; ++h) {
    const int set = set_index(d, req, layer, h);
    SetHost &S = ctx->sets[(size_t)set];
    int32_t off = 0;
    for (int c = 0; c < C; ++c) {
      const int32_t m = count[(size_t)h * C + c], npg = (m + kPageTokens - 1) / kPageTokens;
      first_row_page[(size_t)h * C + c] = off;
      meta[(size_t)c] = MetaEntry{m, 0};
      int seg = ensure_seg(ctx, ctx->off_segs, S.dir_off, d.dir_off + (size_t)set * g.dir_part, c, g.seg_shift, st);
      if (seg < 0) return fail(ctx, SPIN_ERR_OOM_HOST, "out of Partition Offset segments");
      ctx->h_off_pool[((size_t)seg << g.seg_shift) + (c & (g.seg - 1))] = off;
      if (ensure_seg(ctx, ctx->meta_segs, S.dir_meta, d.dir_meta + (size_t)set * g.dir_part, c, g.seg_shift, st) < 0)
        return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of Meta-partition segments");
      if (ensure_seg(ctx, ctx->sum_segs, S.dir_sum, d.dir_sumseg + (size_t)set * g.dir_sum, c, g.sum_shift, st) < 0)
        return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of summary segments");
      for (int i = 0; i < npg; ++i) {
        const int64_t j = off + i;
        int cs = ensure_seg(ctx, ctx->cpt_segs, S.dir_cpt, d.dir_cpt + (size_t)set * g.dir_page, j, g.seg_shift, st);
        if (cs < 0) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
        const int64_t hp = ctx->host_page_pool.alloc();
        ctx->h_cpt_pool[((size_t)cs << g.seg_shift) + (j & (g.seg - 1))] = (int32_t)hp;
        S.host_pages.push_back((int32_t)hp);
      }
      off += npg;
    }
    total_pages_max = std::max(total_pages_max, off);
    S.cl_tokens.assign(count.begin() + (size_t)h * C, count.begin() + (size_t)(h + 1) * C);
    // Meta-partition entries, segment by segment
    for (int c0 = 0; c0 < C; c0 += g.seg) {
      const int cnt = std::min(g.seg, C - c0);
      CK(cudaMemcpyAsync(d.meta_pool + ((size_t)S.dir_meta[(size_t)(c0 >> g.seg_shift)] << g.seg_shift),
                         meta.data() + c0, (size_t)cnt * sizeof(MetaEntry), cudaMemcpyHostToDevice, st));
      CK(cudaStreamSynchronize(st));
    }
    SetState s{};
    s.n_tokens = (int32_t)n;
    s.n_partitions = C;
    s.n_host_pages = off;
    s.tail_first = off;
    s.slots = (int32_t)ctx->reqs[(size_t)req].slots;
    SetState cur{};
    CK(cudaMemcpy(&cur, d.state + set, sizeof cur, cudaMemcpyDeviceToHost));
    s.step = cur.step;
    CK(cudaMemcpy(d.state + set, &s, sizeof s, cudaMemcpyHostToDevice));
  }
  // all heads of a (request, layer) share one tail position: use the largest page count so
  // that tail pages never collide with cluster pages of any head
  for (int h = 0; h < H; ++h) {
    const int set = set_index(d, req, layer, h);
    SetHost &S = ctx->sets[(size_t)set];
    while ((int32_t)S.host_pages.size() < total_pages_max) S.host_pages.push_back(-1);
    SetState s{};
    CK(cudaMemcpy(&s, d.state + set, sizeof s, cudaMemcpyDeviceToHost));
    s.tail_first = total_pages_max;
    s.n_host_pages = total_pages_max;
    CK(cudaMemcpy(d.state + set, &s, sizeof s, cudaMemcpyHostToDevice));
  }
  // the decode kernels read the two host tables through their HBM mirror
  if (d.off_mirror) {
    for (int h = 0; h < H; ++h) {
      const SetHost &S = set_of(ctx, req, layer, h);
      for (int32_t seg : S.dir_off)
        if (seg >= 0) CK(cudaMemcpyAsync(d.off_mirror + ((size_t)seg << g.seg_shift), ctx->h_off_pool + ((size_t)seg << g.seg_shift), (size_t)g.seg * 4, cudaMemcpyHostToDevice, st));
      for (int32_t seg : S.dir_cpt)
        if (seg >= 0) CK(cudaMemcpyAsync(d.cpt_mirror + ((size_t)seg << g.seg_shift), ctx->h_cpt_pool + ((size_t)seg << g.seg_shift), (size_t)g.seg * 4, cudaMemcpyHostToDevice, st));
    }
  }
  // destination row of every (token, head): clusters keep their tokens in arrival order
  std::vector<int32_t> filled((size_t)H * C, 0);
  std::vector<int64_t> dest((size_t)n * H);
  for (int64_t t = 0; t < n; ++t)
    for (int h = 0; h < H; ++h) {
      const int32_t c = tp[(size_t)t * H + h];
      const int32_t r = filled[(size_t)h * C + c]++;
      const SetHost &S = set_of(ctx, req, layer, h);
      const int32_t hp = S.host_pages[(size_t)(first_row_page[(size_t)h * C + c] + r / kPageTokens)];
      dest[(size_t)t * H + h] = (int64_t)hp * kPageTokens + r % kPageTokens;
    }
  // centroids -> summary segments
  const __nv_bfloat16 *cen = reinterpret_cast<const __nv_bfloat16 *>(centroids);
  void *cen_tmp = nullptr;
  if (!is_device_ptr(centroids)) {
    CK(cudaMalloc(&cen_tmp, (size_t)C * H * kRowBytes));
    CK(cudaMemcpy(cen_tmp, centroids, (size_t)C * H * kRowBytes, cudaMemcpyHostToDevice));
    cen = reinterpret_cast<const __nv_bfloat16 *>(cen_tmp);
  }
  ctx->launches += launch_copy_centroids(d, req, layer, cen, C, st);
  const bool dev_kv = is_device_ptr(k);
  if (dev_kv && ctx->offload_slot_units > 0) {
    // Asynchronous offload (Section 4.1): the rows are packed into pages in HBM staging slots on
    // the caller's stream, at HBM speed, range by range of the sets' logical pages; each slot
    // then moves to host memory by copy-engine transfers (one per run of consecutive host
    // pages) on the library's stream, behind this call.
    std::vector<int32_t> lrow((size_t)n * H);
    std::fill(filled.begin(), filled.end(), 0);
    for (int64_t t = 0; t < n; ++t)
      for (int h = 0; h < H; ++h) {
        const int32_t c = tp[(size_t)t * H + h];
        const int32_t r = filled[(size_t)h * C + c]++;
        lrow[(size_t)t * H + h] = (first_row_page[(size_t)h * C + c] + r / kPageTokens) * kPageTokens + r % kPageTokens;
      }
    int32_t *d_lrow = ctx->offload_lrow;                    // this call ends with the stream idle: no earlier prefill still reads it
    CK(cudaMemcpyAsync(d_lrow, lrow.data(), lrow.size() * 4, cudaMemcpyHostToDevice, st));
    const int64_t per = ctx->offload_slot_units / H;
    for (int64_t p0 = 0; p0 < total_pages_max; p0 += per) {
      const int m = (int)std::min<int64_t>(per, total_pages_max - p0), slot = ctx->offload_next;
      ctx->offload_next = (slot + 1) % spin_ctx::kOffloadSlots;
      if (ctx->slot_used[slot]) CK(cudaStreamWaitEvent(st, ctx->ev_done[slot], 0));     // ring full: wait for the drain
      uint8_t *stage = ctx->offload_stage + (size_t)slot * ctx->offload_slot_units * kPageBytes;
      CK(cudaMemsetAsync(stage, 0, (size_t)H * m * kPageBytes, st));                   // rows past a cluster's last token stay zero
      ctx->launches += launch_cluster_scatter_staged(d, reinterpret_cast<const __nv_bfloat16 *>(k),
                                                     reinterpret_cast<const __nv_bfloat16 *>(v), d_lrow, (int)n, (int)p0, m, stage, st);
      CK(cudaEventRecord(ctx->ev_staged[slot], st));
      CK(cudaStreamWaitEvent(ctx->offload_stream, ctx->ev_staged[slot], 0));
      for (int h = 0; h < H; ++h) {
        const std::vector<int32_t> &hpv = set_of(ctx, req, layer, h).host_pages;
        for (int i = 0; i < m;) {
          const int32_t hp0 = hpv[(size_t)(p0 + i)];
          if (hp0 < 0) { ++i; continue; }                                               // this head has fewer pages
          int len = 1;
          while (i + len < m && hpv[(size_t)(p0 + i + len)] == hp0 + len) ++len;
          CK(cudaMemcpyAsync(ctx->h_pages + (size_t)hp0 * kPageBytes, stage + ((size_t)h * m + i) * kPageBytes,
                             (size_t)len * kPageBytes, cudaMemcpyDeviceToHost, ctx->offload_stream));
          i += len;
        }
      }
      CK(cudaEventRecord(ctx->ev_done[slot], ctx->offload_stream));
      ctx->slot_used[slot] = true;
      ctx->offload_last = slot;
      ++ctx->offload_gen;
    }
    CK(cudaStreamSynchronize(st));          // the host-side sources of this call's copies end here; the drain goes on
  } else {
  // rows -> host pages, in chunks through the staging buffers
  const int64_t chunk = g.stage_tokens;
  for (int64_t t0 = 0; t0 < n; t0 += chunk) {
    const int64_t m = std::min(chunk, n - t0);
    const size_t rows = (size_t)m * H;
    const __nv_bfloat16 *kk = reinterpret_cast<const __nv_bfloat16 *>(k) + (size_t)t0 * H * kHeadDim;
    const __nv_bfloat16 *vv = reinterpret_cast<const __nv_bfloat16 *>(v) + (size_t)t0 * H * kHeadDim;
    if (!dev_kv) {
      CK(cudaMemcpyAsync(ctx->stage_k, kk, rows * kRowBytes, cudaMemcpyHostToDevice, st));
      CK(cudaMemcpyAsync(ctx->stage_v, vv, rows * kRowBytes, cudaMemcpyHostToDevice, st));
      kk = ctx->stage_k;
      vv = ctx->stage_v;
    }
    CK(cudaMemcpyAsync(ctx->stage_dest, dest.data() + (size_t)t0 * H, rows * 8, cudaMemcpyHostToDevice, st));
    ctx->launches += launch_cluster_scatter(d, req, layer, kk, vv, ctx->stage_dest, (int)m, st);
    CK(cudaStreamSynchronize(st));
  }
  }
  if (cen_tmp) CK(cudaFree(cen_tmp));
  CK(cudaGetLastError());
  L.n_tokens = n;
  L.n_partitions = C;
  L.n_host_pages = total_pages_max;
  L.tail_first = total_pages_max;
  L.tail_pages = 0;
  L.tail_len = 0;
  L.clustered = true;
  return SPIN_OK;
}

}  // namespace

namespace spin {
void Prof::mark(cudaStream_t st, int kernel) {
  if (!ev) {
    ev = new cudaEvent_t[kMaxMarks];
    id = new int[kMaxMarks];
    for (size_t i = 0; i < kMaxMarks; ++i) cudaEventCreate(&ev[i]);
  }
  if (used >= kMaxMarks) return;
  cudaEventRecord(ev[used], st);
  id[used++] = kernel;
}
}  // namespace spin

// ---------------------------------------------------------------------------------------
extern "C" {

int spin_profile(spin_ctx *ctx, int32_t enable) {
  if (!ctx) return SPIN_ERR_INVALID;
  CK(cudaDeviceSynchronize());
  ctx->prof.on = enable != 0;
  ctx->prof.used = 0;
  return SPIN_OK;
}

int spin_profile_read(spin_ctx *ctx, spin_profile_t *out) {
  if (!ctx || !out) return SPIN_ERR_INVALID;
  if (out->struct_size != sizeof(spin_profile_t)) return fail(ctx, SPIN_ERR_INVALID, "spin_profile_t.struct_size mismatch");
  CK(cudaDeviceSynchronize());
  out->n_kernels = kProfKernels;
  for (int i = 0; i < 8; ++i) { out->launches[i] = 0; out->ms[i] = 0.0; }
  const Prof &p = ctx->prof;
  for (size_t i = 1; i < p.used; ++i) {
    if (p.id[i] < 0) continue;
    float ms = 0.f;
    CK(cudaEventElapsedTime(&ms, p.ev[i - 1], p.ev[i]));
    out->launches[p.id[i]] += 1;
    out->ms[p.id[i]] += ms;
  }
  return SPIN_OK;
}


const char *spin_version(void) { return "spin-b200 0.1"; }

const char *spin_last_error(spin_ctx *ctx) { return ctx ? ctx->err.c_str() : "null context"; }

int spin_required_bytes(const spin_config *cfg, size_t *device_bytes, size_t *host_bytes) {
  if (!cfg) return SPIN_ERR_INVALID;
  Geometry g{};
  std::string err;
  int rc = compute_geometry(*cfg, g, err);
  if (rc) return rc;
  Arena a;
  DevCtx d{};
  carve(a, *cfg, g, d, nullptr);
  if (device_bytes) *device_bytes = align_up(a.off, 256);
  if (host_bytes) *host_bytes = host_bytes_needed(g, *cfg);
  return SPIN_OK;
}

int spin_create(const spin_config *cfg, spin_ctx **out) {
  if (!out) return SPIN_ERR_INVALID;
  *out = nullptr;
  if (!cfg) return SPIN_ERR_INVALID;
  spin_ctx *ctx = new spin_ctx();
  ctx->cfg = *cfg;
  int rc = compute_geometry(*cfg, ctx->g, ctx->err);
  if (rc) { fprintf(stderr, "spin_create: %s\n", ctx->err.c_str()); delete ctx; return rc; }
  const Geometry &g = ctx->g;
  auto cuda_fail = [&](const char *what, cudaError_t e) {
    fprintf(stderr, "spin_create: %s: %s\n", what, cudaGetErrorString(e));
    if (ctx->host_base) cudaFreeHost(ctx->host_base);
    delete ctx;
    return (int)SPIN_ERR_CUDA;
  };
  cudaError_t e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess && sms > 0) ctx->sm_count = sms;
  if (!cfg->hbm_pool || ((uintptr_t)cfg->hbm_pool & 255)) { delete ctx; return SPIN_ERR_INVALID; }
  Arena a;
  a.base = reinterpret_cast<uint8_t *>(cfg->hbm_pool);
  DevCtx &d = ctx->d;
  carve(a, *cfg, g, d, ctx);
  if (a.off > cfg->hbm_pool_bytes) {
    fprintf(stderr, "spin_create: hbm_pool too small (%zu < %zu)\n", cfg->hbm_pool_bytes, a.off);
    delete ctx;
    return SPIN_ERR_OOM_DEVICE;
  }
  ctx->host_bytes = host_bytes_needed(g, *cfg);
  e = cudaHostAlloc(reinterpret_cast<void **>(&ctx->host_base), ctx->host_bytes, cudaHostAllocMapped | cudaHostAllocPortable);
  if (e != cudaSuccess) { cudaGetLastError(); fprintf(stderr, "spin_create: pinned allocation of %zu bytes failed\n", ctx->host_bytes); delete ctx; return SPIN_ERR_OOM_HOST; }
  uint8_t *dev_view = nullptr;
  e = cudaHostGetDevicePointer(reinterpret_cast<void **>(&dev_view), ctx->host_base, 0);
  if (e != cudaSuccess) return cuda_fail("cudaHostGetDevicePointer", e);
  size_t o = 0;
  ctx->h_pages = ctx->host_base;
  d.host_pages = dev_view;
  o += align_up((size_t)cfg->host_pages * kPageBytes, 4096);
  ctx->h_off_pool = reinterpret_cast<int32_t *>(ctx->host_base + o);
  d.off_pool = reinterpret_cast<int32_t *>(dev_view + o);
  o += align_up((size_t)g.n_off_segs * g.seg * 4, 4096);
  ctx->h_cpt_pool = reinterpret_cast<int32_t *>(ctx->host_base + o);
  d.cpt_pool = reinterpret_cast<int32_t *>(dev_view + o);

  d.num_layers = cfg->num_layers; d.Hq = cfg->num_q_heads; d.Hkv = cfg->num_kv_heads;
  d.G = cfg->num_q_heads / cfg->num_kv_heads; d.kind = cfg->partition_kind; d.topk = cfg->topk;
  d.n_buckets = cfg->lru_buckets; d.trace = cfg->trace ? 1 : 0;
  d.seg_shift = g.seg_shift; d.sum_shift = g.sum_shift; d.sum_entry_bytes = g.sum_entry_bytes;
  d.dir_part = g.dir_part; d.dir_slot = g.dir_slot; d.dir_page = g.dir_page; d.dir_sum = g.dir_sum;
  d.max_sel = g.max_sel; d.max_parts = g.max_parts; d.max_pages = g.max_pages; d.tail_cap = g.tail_cap;
  d.max_cand = (int32_t)g.max_cand; d.max_slots = (int32_t)g.max_slots; d.max_chunks = g.max_chunks;
  d.fetch_cap = (int32_t)g.fetch_cap;
  d.n_gpu_pages = (int32_t)g.n_gpu_pages_total;
  d.n_host_pages = (int32_t)cfg->host_pages;
  d.fetch_mode = cfg->fetch_mode ? 1 : 0;
  d.evict_exact = cfg->evict_exact ? 1 : 0;
  d.resident_scoring = cfg->resident_scoring == 2 ? 2 : cfg->resident_scoring > 0 ? 1 : cfg->resident_scoring < 0 ? -1 : 0;
  d.sm_scale = cfg->sm_scale != 0.f ? cfg->sm_scale : 1.0f / sqrtf((float)kHeadDim);

  // directories start unmapped (-1); states, counters and the miss queue start at zero
  auto fill = [&](void *p, int v, size_t bytes) { return cudaMemset(p, v, bytes); };
  if ((e = fill(d.dir_meta, 0xff, (size_t)g.n_sets * g.dir_part * 4)) != cudaSuccess) return cuda_fail("cudaMemset", e);
  fill(d.dir_off, 0xff, (size_t)g.n_sets * g.dir_part * 4);
  fill(d.dir_gpt, 0xff, (size_t)g.n_sets * g.dir_slot * 4);
  fill(d.dir_cpt, 0xff, (size_t)g.n_sets * g.dir_page * 4);
  fill(d.dir_sumseg, 0xff, (size_t)g.n_sets * g.dir_sum * 4);
  // every byte a kernel may read as K/V is finite from the start (rows past a page's valid
  // tokens are masked out of the softmax but still enter the P*V tiles with weight 0)
  fill(d.gpu_pages, 0, (size_t)g.n_gpu_pages_total * kPageBytes);
  memset(ctx->host_base, 0, ctx->host_bytes);
  fill(d.score_xfer, 0xff, (size_t)g.max_batch_sets * g.max_cand * 4);       // every word "not written"
  fill(d.att_count, 0, (size_t)g.max_batch_sets * 4);
  fill(d.sel_count, 0, (size_t)g.max_batch_sets * 4);
  fill(d.score_queue, 0, 4);
  fill(d.score_done, 0, 4);
  fill(d.scored, 0, (size_t)g.max_batch_sets * 4);
  fill(d.ready, 0, (size_t)g.max_batch_sets * 4);
  fill(d.tail_ready, 0, (size_t)g.max_batch_sets * 4);
  fill(d.ready1, 0, (size_t)g.max_batch_sets * 4);
  fill(d.n_miss, 0, (size_t)g.max_batch_sets * 4);
  fill(d.state, 0, (size_t)g.n_sets * sizeof(SetState));
  fill(d.counters, 0, sizeof(Counters));
  fill(d.fetch_count, 0, 4);
  fill(d.n_pages, 0, (size_t)g.max_batch_sets * 4);
  fill(d.n_parts, 0, (size_t)g.max_batch_sets * 4);
  fill(d.n_sel, 0, (size_t)g.max_batch_sets * 4);
  if (d.evict_trace) fill(d.evict_trace, 0xff, (size_t)g.n_sets * g.max_slots * 8);
  if ((e = cudaDeviceSynchronize()) != cudaSuccess) return cuda_fail("cudaDeviceSynchronize", e);
  if (ctx->offload_slot_units > 0) {
    if ((e = cudaStreamCreateWithFlags(&ctx->offload_stream, cudaStreamNonBlocking)) != cudaSuccess) return cuda_fail("cudaStreamCreateWithFlags", e);
    for (int i = 0; i < spin_ctx::kOffloadSlots; ++i) {
      if ((e = cudaEventCreateWithFlags(&ctx->ev_staged[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail("cudaEventCreateWithFlags", e);
      if ((e = cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming)) != cudaSuccess) return cuda_fail("cudaEventCreateWithFlags", e);
    }
  }

  ctx->gpu_page_pool.init(cfg->gpu_cache_pages);
  ctx->host_page_pool.init(cfg->host_pages);
  ctx->gpt_segs.init(g.n_gpt_segs);
  ctx->meta_segs.init(g.n_meta_segs);
  ctx->off_segs.init(g.n_off_segs);
  ctx->cpt_segs.init(g.n_cpt_segs);
  ctx->sum_segs.init(g.n_sum_segs);
  ctx->reqs.resize((size_t)cfg->max_requests);
  ctx->sets.resize((size_t)g.n_sets);
  *out = ctx;
  return SPIN_OK;
}

int spin_destroy(spin_ctx *ctx) {
  if (!ctx) return SPIN_ERR_INVALID;
  cudaDeviceSynchronize();
  if (ctx->prof.ev) {
    for (size_t i = 0; i < Prof::kMaxMarks; ++i) cudaEventDestroy(ctx->prof.ev[i]);
    delete[] ctx->prof.ev;
    delete[] ctx->prof.id;
  }
  if (ctx->offload_stream) {
    for (int i = 0; i < spin_ctx::kOffloadSlots; ++i) { cudaEventDestroy(ctx->ev_staged[i]); cudaEventDestroy(ctx->ev_done[i]); }
    cudaStreamDestroy(ctx->offload_stream);
  }
  if (ctx->host_base) cudaFreeHost(ctx->host_base);
  delete ctx;
  return SPIN_OK;
}

int spin_request_open(spin_ctx *ctx, int64_t slots, int32_t *out_req) {
  if (!ctx || !out_req) return SPIN_ERR_INVALID;
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  if (slots < 0 || slots > g.max_slots) return fail(ctx, SPIN_ERR_INVALID, "budget %lld outside 0..%lld", (long long)slots, (long long)g.max_slots);
  int req = -1;
  for (int r = 0; r < ctx->cfg.max_requests; ++r) if (!ctx->reqs[(size_t)r].open) { req = r; break; }
  if (req < 0) return fail(ctx, SPIN_ERR_STATE, "all %d request slots are open", ctx->cfg.max_requests);
  const int64_t sets_per_req = (int64_t)ctx->cfg.num_layers * ctx->cfg.num_kv_heads;
  const int64_t segs_per_set = (slots + g.seg - 1) / g.seg;
  if (ctx->gpu_page_pool.available() < slots * sets_per_req)
    return fail(ctx, SPIN_ERR_BUDGET, "budget needs %lld GPU pages, %lld free", (long long)(slots * sets_per_req), (long long)ctx->gpu_page_pool.available());
  if (ctx->gpt_segs.available() < segs_per_set * sets_per_req)
    return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of GPU page table segments");
  std::vector<GptEntry> ent((size_t)g.seg);
  for (int l = 0; l < ctx->cfg.num_layers; ++l)
    for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
      const int set = set_index(d, req, l, h);
      SetHost &S = ctx->sets[(size_t)set];
      S = SetHost();
      S.dir_meta.assign((size_t)g.dir_part, -1);
      S.dir_off.assign((size_t)g.dir_part, -1);
      S.dir_gpt.assign((size_t)g.dir_slot, -1);
      S.dir_cpt.assign((size_t)g.dir_page, -1);
      S.dir_sum.assign((size_t)g.dir_sum, -1);
      for (int64_t s0 = 0; s0 < slots; s0 += g.seg) {
        const int64_t seg = ctx->gpt_segs.alloc();
        S.dir_gpt[(size_t)(s0 >> g.seg_shift)] = (int32_t)seg;
        ctx->dir_bytes_in_use += 4;
        const int cnt = (int)std::min<int64_t>(g.seg, slots - s0);
        for (int i = 0; i < g.seg; ++i) {
          int32_t phys = -1;
          if (i < cnt) { phys = (int32_t)ctx->gpu_page_pool.alloc(); S.gpu_pages.push_back(phys); }
          ent[(size_t)i] = GptEntry{-1, phys, 0, -1};
        }
        CK(cudaMemcpy(d.gpt_pool + ((size_t)seg << g.seg_shift), ent.data(), (size_t)g.seg * sizeof(GptEntry), cudaMemcpyHostToDevice));
      }
      CK(cudaMemcpy(d.dir_gpt + (size_t)set * g.dir_slot, S.dir_gpt.data(), (size_t)g.dir_slot * 4, cudaMemcpyHostToDevice));
      CK(cudaMemcpy(d.dir_meta + (size_t)set * g.dir_part, S.dir_meta.data(), (size_t)g.dir_part * 4, cudaMemcpyHostToDevice));
      CK(cudaMemcpy(d.dir_off + (size_t)set * g.dir_part, S.dir_off.data(), (size_t)g.dir_part * 4, cudaMemcpyHostToDevice));
      CK(cudaMemcpy(d.dir_cpt + (size_t)set * g.dir_page, S.dir_cpt.data(), (size_t)g.dir_page * 4, cudaMemcpyHostToDevice));
      CK(cudaMemcpy(d.dir_sumseg + (size_t)set * g.dir_sum, S.dir_sum.data(), (size_t)g.dir_sum * 4, cudaMemcpyHostToDevice));
      std::vector<int32_t> tails((size_t)g.tail_cap);
      for (int j = 0; j < g.tail_cap; ++j) tails[(size_t)j] = (int32_t)(ctx->cfg.gpu_cache_pages + (int64_t)set * g.tail_cap + j);
      CK(cudaMemcpy(d.tail_phys + (size_t)set * g.tail_cap, tails.data(), (size_t)g.tail_cap * 4, cudaMemcpyHostToDevice));
      SetState s{};
      s.slots = (int32_t)slots;
      CK(cudaMemcpy(d.state + set, &s, sizeof s, cudaMemcpyHostToDevice));
    }
  RequestHost &R = ctx->reqs[(size_t)req];
  R.open = true;
  R.slots = slots;
  R.layers.assign((size_t)ctx->cfg.num_layers, LayerHost());
  *out_req = req;
  return SPIN_OK;
}

int spin_reindex(spin_ctx *ctx, int32_t req, int32_t layer, void *cuda_stream) {
  int rc = validate_req_layer(ctx, req, layer);
  if (rc) return rc;
  if (ctx->cfg.partition_kind != SPIN_PART_CLUSTER_CENTROID)
    return fail(ctx, SPIN_ERR_INVALID, "spin_reindex applies to cluster granularity only");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  if (!L.clustered) return fail(ctx, SPIN_ERR_STATE, "request %d has no cluster prefill yet", req);
  if (int rc2 = wait_for_offload(ctx, st)) return rc2;     // prefill pages still on their way must not land on the moved rows
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  const int H = ctx->cfg.num_kv_heads, C = ctx->cfg.num_clusters;
  // full tail pages, as many as the staging buffers take in one go
  int n_full = L.tail_pages - (L.tail_pages > 0 && L.tail_len == kPageTokens ? 0 : 1);
  n_full = std::min<int>(n_full, (int)(g.stage_tokens / kPageTokens));
  if (n_full <= 0) return SPIN_OK;
  const int n_tok = n_full * kPageTokens;

  // 1. the best cluster of every token (device), brought to the host; everything enqueued on
  //    the stream before this call has finished once the copy is here
  int32_t *d_assign = reinterpret_cast<int32_t *>(ctx->stage_k);
  ctx->launches += launch_assign(d, req, layer, C, n_tok, d_assign, st);
  std::vector<int32_t> assign((size_t)n_tok * H);
  CK(cudaMemcpyAsync(assign.data(), d_assign, assign.size() * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));

  // 2. new page lists and layout, head by head.  First pass: how many host pages it takes.
  int64_t need = 0;
  for (int h = 0; h < H; ++h) {
    std::vector<int32_t> cnt = set_of(ctx, req, layer, h).cl_tokens;
    for (int t = 0; t < n_tok; ++t) {
      const int32_t c = assign[(size_t)t * H + h];
      if (c < 0 || c >= C) return fail(ctx, SPIN_ERR_CUDA, "cluster assignment out of range");
      if (cnt[(size_t)c]++ % kPageTokens == 0) ++need;
    }
  }
  if (ctx->host_page_pool.available() < need) return fail(ctx, SPIN_ERR_OOM_HOST, "out of host pages");
  std::vector<int64_t> dest((size_t)n_tok * H);
  std::vector<int32_t> new_tokens((size_t)H * C);
  const int words = (C + 31) / 32;
  std::vector<uint32_t> touched((size_t)H * words, 0u);
  std::vector<std::vector<int32_t>> old_tail((size_t)H);
  std::vector<std::vector<std::vector<int32_t>>> lists((size_t)H);
  int32_t total_max = 0;
  for (int h = 0; h < H; ++h) {
    SetHost &S = set_of(ctx, req, layer, h);
    for (int i = 0; i < L.tail_pages; ++i) old_tail[(size_t)h].push_back(S.host_pages[(size_t)(L.tail_first + i)]);
    auto &ls = lists[(size_t)h];
    ls.resize((size_t)C);
    for (int c = 0; c < C; ++c) {
      const int32_t seg = S.dir_off[(size_t)(c >> g.seg_shift)];
      const int32_t off = ctx->h_off_pool[((size_t)seg << g.seg_shift) + (c & (g.seg - 1))];
      const int npg = (S.cl_tokens[(size_t)c] + kPageTokens - 1) / kPageTokens;
      ls[(size_t)c].assign(S.host_pages.begin() + off, S.host_pages.begin() + off + npg);
    }
    for (int t = 0; t < n_tok; ++t) {
      const int32_t c = assign[(size_t)t * H + h];
      const int32_t m = S.cl_tokens[(size_t)c];
      if (m % kPageTokens == 0) ls[(size_t)c].push_back((int32_t)ctx->host_page_pool.alloc());
      dest[(size_t)t * H + h] = (int64_t)ls[(size_t)c][(size_t)(m / kPageTokens)] * kPageTokens + m % kPageTokens;
      S.cl_tokens[(size_t)c] = m + 1;
      touched[(size_t)h * words + (c >> 5)] |= 1u << (c & 31);
    }
    int32_t total = 0;
    for (int c = 0; c < C; ++c) total += (int32_t)ls[(size_t)c].size();
    total_max = std::max(total_max, total);
    std::copy(S.cl_tokens.begin(), S.cl_tokens.end(), new_tokens.begin() + (size_t)h * C);
  }

  // 3. the sets' Partition Offset and CPU page tables laid out afresh (clusters in order, each
  //    one's pages together), what is left of the tail behind the longest head's clusters
  const int n_rem = L.tail_pages - n_full;
  if ((int64_t)total_max + g.tail_cap > (int64_t)g.dir_page * g.seg)
    return fail(ctx, SPIN_ERR_INVALID, "request %d outgrew its CPU page table", req);
  for (int h = 0; h < H; ++h) {
    const int set = set_index(d, req, layer, h);
    SetHost &S = ctx->sets[(size_t)set];
    S.host_pages.assign((size_t)(total_max + n_rem), -1);
    auto put = [&](int64_t j, int32_t hp) -> bool {
      const int cs = ensure_seg(ctx, ctx->cpt_segs, S.dir_cpt, d.dir_cpt + (size_t)set * g.dir_page, j, g.seg_shift, st);
      if (cs < 0) return false;
      ctx->h_cpt_pool[((size_t)cs << g.seg_shift) + (j & (g.seg - 1))] = hp;
      S.host_pages[(size_t)j] = hp;
      return true;
    };
    int32_t off = 0;
    for (int c = 0; c < C; ++c) {
      const int32_t seg = S.dir_off[(size_t)(c >> g.seg_shift)];
      ctx->h_off_pool[((size_t)seg << g.seg_shift) + (c & (g.seg - 1))] = off;
      for (int32_t hp : lists[(size_t)h][(size_t)c])
        if (!put(off++, hp)) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
    }
    for (int i = 0; i < n_rem; ++i)
      if (!put((int64_t)total_max + i, old_tail[(size_t)h][(size_t)(n_full + i)])) return fail(ctx, SPIN_ERR_OOM_HOST, "out of CPU page table segments");
    for (int i = 0; i < n_full; ++i) ctx->host_page_pool.release(old_tail[(size_t)h][(size_t)i]);   // their rows live in the clusters now
  }

  // 4. device side: rows to their places; counts, residency and tail; the tables' HBM copies
  int32_t *d_new_tokens = reinterpret_cast<int32_t *>(ctx->stage_v);
  uint32_t *d_touched = reinterpret_cast<uint32_t *>(d_new_tokens + new_tokens.size());
  const size_t stage_bytes = (size_t)std::max<int64_t>(g.stage_tokens, ctx->cfg.max_requests) * H * kRowBytes;
  if ((new_tokens.size() + touched.size()) * 4 > stage_bytes) return fail(ctx, SPIN_ERR_INVALID, "too many clusters for the staging buffer");
  CK(cudaMemcpyAsync(ctx->stage_dest, dest.data(), dest.size() * 8, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(d_new_tokens, new_tokens.data(), new_tokens.size() * 4, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(d_touched, touched.data(), touched.size() * 4, cudaMemcpyHostToDevice, st));
  ctx->launches += launch_move_rows(d, req, layer, ctx->stage_dest, n_tok, st);
  ctx->launches += launch_reindex_apply(d, req, layer, C, n_full, total_max, n_rem, n_rem ? L.tail_len : 0,
                                        total_max + n_rem, d_new_tokens, d_touched, st);
  if (d.off_mirror) {
    for (int h = 0; h < H; ++h) {
      const SetHost &S = set_of(ctx, req, layer, h);
      for (int32_t seg : S.dir_off)
        if (seg >= 0) CK(cudaMemcpyAsync(d.off_mirror + ((size_t)seg << g.seg_shift), ctx->h_off_pool + ((size_t)seg << g.seg_shift), (size_t)g.seg * 4, cudaMemcpyHostToDevice, st));
      for (int32_t seg : S.dir_cpt)
        if (seg >= 0) CK(cudaMemcpyAsync(d.cpt_mirror + ((size_t)seg << g.seg_shift), ctx->h_cpt_pool + ((size_t)seg << g.seg_shift), (size_t)g.seg * 4, cudaMemcpyHostToDevice, st));
    }
  }
  L.tail_first = total_max;
  L.tail_pages = n_rem;
  if (n_rem == 0) L.tail_len = 0;
  L.n_host_pages = total_max + n_rem;
  CK(cudaStreamSynchronize(st));          // the host-side sources of the copies above end here
  CK(cudaGetLastError());
  return SPIN_OK;
}
int spin_request_close(spin_ctx *ctx, int32_t req) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (req < 0 || req >= ctx->cfg.max_requests) return fail(ctx, SPIN_ERR_INVALID, "request id %d out of range", req);
  RequestHost &R = ctx->reqs[(size_t)req];
  if (!R.open) return fail(ctx, SPIN_ERR_STATE, "request %d is not open", req);
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  if (ctx->offload_stream) CK(cudaStreamSynchronize(ctx->offload_stream));   // its pages may still be on their way
  for (int l = 0; l < ctx->cfg.num_layers; ++l)
    for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
      const int set = set_index(d, req, l, h);
      SetHost &S = ctx->sets[(size_t)set];
      for (int32_t p : S.gpu_pages) ctx->gpu_page_pool.release(p);
      for (int32_t p : S.host_pages) ctx->host_page_pool.release(p);
      auto drop = [&](BitmapPool &pool, std::vector<int32_t> &dir) {
        for (int32_t s : dir) if (s >= 0) { pool.release(s); ctx->dir_bytes_in_use -= 4; }
      };
      drop(ctx->gpt_segs, S.dir_gpt);
      drop(ctx->meta_segs, S.dir_meta);
      drop(ctx->off_segs, S.dir_off);
      drop(ctx->cpt_segs, S.dir_cpt);
      drop(ctx->sum_segs, S.dir_sum);
      CK(cudaMemset(d.dir_gpt + (size_t)set * g.dir_slot, 0xff, (size_t)g.dir_slot * 4));
      CK(cudaMemset(d.dir_meta + (size_t)set * g.dir_part, 0xff, (size_t)g.dir_part * 4));
      CK(cudaMemset(d.dir_off + (size_t)set * g.dir_part, 0xff, (size_t)g.dir_part * 4));
      CK(cudaMemset(d.dir_cpt + (size_t)set * g.dir_page, 0xff, (size_t)g.dir_page * 4));
      CK(cudaMemset(d.dir_sumseg + (size_t)set * g.dir_sum, 0xff, (size_t)g.dir_sum * 4));
      CK(cudaMemset(d.state + set, 0, sizeof(SetState)));
      S = SetHost();
    }
  R = RequestHost();
  return SPIN_OK;
}

int spin_set_budget(spin_ctx *ctx, int32_t req, int64_t slots) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (req < 0 || req >= ctx->cfg.max_requests) return fail(ctx, SPIN_ERR_INVALID, "request id %d out of range", req);
  RequestHost &R = ctx->reqs[(size_t)req];
  if (!R.open) return fail(ctx, SPIN_ERR_STATE, "request %d is not open", req);
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  if (slots < 0 || slots > g.max_slots) return fail(ctx, SPIN_ERR_INVALID, "budget %lld outside 0..%lld", (long long)slots, (long long)g.max_slots);
  const int64_t old = R.slots;
  if (slots == old) return SPIN_OK;
  const int64_t sets_per_req = (int64_t)ctx->cfg.num_layers * ctx->cfg.num_kv_heads;
  CK(cudaDeviceSynchronize());
  if (slots < old) {
    // reclaim the tail of every set's GPU page table on the device, then give the pages and
    // the segments that lie wholly beyond the cut back to their pools
    ctx->launches += launch_shrink(d, req, (int)old, (int)slots, nullptr);
    CK(cudaDeviceSynchronize());
    const int64_t keep_segs = (slots + g.seg - 1) / g.seg;
    for (int l = 0; l < ctx->cfg.num_layers; ++l)
      for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
        const int set = set_index(d, req, l, h);
        SetHost &S = ctx->sets[(size_t)set];
        for (int64_t s = slots; s < old; ++s) ctx->gpu_page_pool.release(S.gpu_pages[(size_t)s]);
        S.gpu_pages.resize((size_t)slots);
        for (int64_t di = keep_segs; di < (int64_t)S.dir_gpt.size(); ++di)
          if (S.dir_gpt[(size_t)di] >= 0) {
            ctx->gpt_segs.release(S.dir_gpt[(size_t)di]);
            ctx->dir_bytes_in_use -= 4;
            S.dir_gpt[(size_t)di] = -1;
          }
        CK(cudaMemcpy(d.dir_gpt + (size_t)set * g.dir_slot, S.dir_gpt.data(), (size_t)g.dir_slot * 4, cudaMemcpyHostToDevice));
      }
  } else {
    const int64_t add = slots - old;
    const int64_t new_segs = (slots + g.seg - 1) / g.seg - (old + g.seg - 1) / g.seg;
    if (ctx->gpu_page_pool.available() < add * sets_per_req)
      return fail(ctx, SPIN_ERR_BUDGET, "growing needs %lld GPU pages, %lld free", (long long)(add * sets_per_req), (long long)ctx->gpu_page_pool.available());
    if (ctx->gpt_segs.available() < new_segs * sets_per_req) return fail(ctx, SPIN_ERR_OOM_DEVICE, "out of GPU page table segments");
    for (int l = 0; l < ctx->cfg.num_layers; ++l)
      for (int h = 0; h < ctx->cfg.num_kv_heads; ++h) {
        const int set = set_index(d, req, l, h);
        SetHost &S = ctx->sets[(size_t)set];
        for (int64_t s = old; s < slots; ++s) {
          const size_t di = (size_t)(s >> g.seg_shift);
          if (S.dir_gpt[di] < 0) {
            S.dir_gpt[di] = (int32_t)ctx->gpt_segs.alloc();
            ctx->dir_bytes_in_use += 4;
          }
          const int32_t phys = (int32_t)ctx->gpu_page_pool.alloc();
          S.gpu_pages.push_back(phys);
          const GptEntry e{-1, phys, 0, -1};
          CK(cudaMemcpy(d.gpt_pool + ((size_t)S.dir_gpt[di] << g.seg_shift) + (s & (g.seg - 1)), &e, sizeof e, cudaMemcpyHostToDevice));
        }
        CK(cudaMemcpy(d.dir_gpt + (size_t)set * g.dir_slot, S.dir_gpt.data(), (size_t)g.dir_slot * 4, cudaMemcpyHostToDevice));
        const int32_t ns = (int32_t)slots;
        CK(cudaMemcpy(&d.state[set].slots, &ns, 4, cudaMemcpyHostToDevice));
      }
  }
  R.slots = slots;
  return SPIN_OK;
}

int spin_append_kv(spin_ctx *ctx, int32_t req, int32_t layer, const void *k, const void *v,
                   int64_t n_tokens, const int32_t *token_partition, const void *centroids,
                   void *cuda_stream) {
  int rc = validate_req_layer(ctx, req, layer);
  if (rc) return rc;
  if (!k || !v || n_tokens < 0) return fail(ctx, SPIN_ERR_INVALID, "null k/v or negative n_tokens");
  if (n_tokens == 0) return SPIN_OK;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  const bool cluster = ctx->cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID;
  if (cluster && !L.clustered) {
    if (!token_partition || !centroids) return fail(ctx, SPIN_ERR_INVALID, "cluster prefill needs token_partition and centroids");
    return prefill_clustered(ctx, req, layer, k, v, n_tokens, token_partition, centroids, st);
  }
  if (token_partition || centroids) return fail(ctx, SPIN_ERR_INVALID, "token_partition/centroids only belong to the cluster prefill");
  const bool dev = is_device_ptr(k);
  if (dev != is_device_ptr(v)) return fail(ctx, SPIN_ERR_INVALID, "k and v must both be device or both be host pointers");
  const int H = ctx->cfg.num_kv_heads;
  const int64_t chunk = dev && !cluster ? n_tokens : (cluster ? 1 : ctx->g.stage_tokens);
  for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
    const int64_t m = std::min(chunk, n_tokens - t0);
    const __nv_bfloat16 *kk = reinterpret_cast<const __nv_bfloat16 *>(k) + (size_t)t0 * H * kHeadDim;
    const __nv_bfloat16 *vv = reinterpret_cast<const __nv_bfloat16 *>(v) + (size_t)t0 * H * kHeadDim;
    if (!dev) {
      CK(cudaMemcpyAsync(ctx->stage_k, kk, (size_t)m * H * kRowBytes, cudaMemcpyHostToDevice, st));
      CK(cudaMemcpyAsync(ctx->stage_v, vv, (size_t)m * H * kRowBytes, cudaMemcpyHostToDevice, st));
      kk = ctx->stage_k;
      vv = ctx->stage_v;
    }
    if (cluster) {
      rc = grow_cluster_tail(ctx, req, layer, m, st);
      if (rc) return rc;
      AppendEdgeArgs a{};
      a.n_req = 1; a.layer = layer; a.req[0] = req;
      a.n_tokens[0] = (int32_t)(L.n_tokens - m);
      ctx->launches += launch_append_edge(ctx->d, a, kk, vv, (int)m, st, &ctx->prof);
    } else {
      rc = append_paged_device(ctx, req, layer, kk, vv, m, st);
      if (rc) return rc;
    }
    if (!dev) CK(cudaStreamSynchronize(st));      // the staging buffers are reused
  }
  CK(cudaGetLastError());
  return SPIN_OK;
}

int spin_append_kv_batch(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req,
                         const void *k, const void *v, void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (!req_ids || !k || !v || n_req < 1 || n_req > ctx->cfg.max_requests) return fail(ctx, SPIN_ERR_INVALID, "bad batch arguments");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  AppendEdgeArgs a{};
  a.n_req = n_req;
  a.layer = layer;
  for (int i = 0; i < n_req; ++i) {
    int rc = validate_req_layer(ctx, req_ids[i], layer);
    if (rc) return rc;
    for (int j = 0; j < i; ++j) if (req_ids[j] == req_ids[i]) return fail(ctx, SPIN_ERR_INVALID, "request %d listed twice", req_ids[i]);
    a.req[i] = req_ids[i];
  }
  const bool cluster = ctx->cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID;
  const bool k_dev = is_device_ptr(k);
  if (k_dev != is_device_ptr(v)) return fail(ctx, SPIN_ERR_INVALID, "k and v must both be device or both be host pointers");
  if (int rc = precheck_append_one(ctx, layer, req_ids, n_req)) return rc;
  // all checks passed: from here on the call changes state
  for (int i = 0; i < n_req; ++i) {
    LayerHost &L = ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer];
    int rc = cluster ? grow_cluster_tail(ctx, req_ids[i], layer, 1, st) : grow_paged(ctx, req_ids[i], layer, L.n_tokens + 1, st);
    if (rc) return rc;
    a.n_tokens[i] = (int32_t)(L.n_tokens - 1);
  }
  const __nv_bfloat16 *kk = reinterpret_cast<const __nv_bfloat16 *>(k), *vv = reinterpret_cast<const __nv_bfloat16 *>(v);
  if (!k_dev) {
    const size_t bytes = (size_t)n_req * ctx->cfg.num_kv_heads * kRowBytes;
    CK(cudaMemcpyAsync(ctx->stage_k, k, bytes, cudaMemcpyHostToDevice, st));
    CK(cudaMemcpyAsync(ctx->stage_v, v, bytes, cudaMemcpyHostToDevice, st));
    kk = ctx->stage_k;
    vv = ctx->stage_v;
  }
  prof_mark(&ctx->prof, st, -1);
  ctx->launches += launch_append_edge(ctx->d, a, kk, vv, 1, st, &ctx->prof);
  CK(cudaGetLastError());
  return SPIN_OK;
}

// One decode step, optionally preceded by the append of one token per request.
static int step_impl(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req, const void *k,
                     const void *v, const void *q, void *out, cudaStream_t st) {
  if (!req_ids || !q || !out || n_req < 1 || n_req > ctx->cfg.max_requests) return fail(ctx, SPIN_ERR_INVALID, "bad batch arguments");
  const bool with_append = k != nullptr;
  if (with_append && !v) return fail(ctx, SPIN_ERR_INVALID, "k without v");
  const bool cluster = ctx->cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID;
  Batch b{};
  b.n_req = n_req;
  b.layer = layer;
  bool completes_page = false;
  for (int i = 0; i < n_req; ++i) {
    int rc = validate_req_layer(ctx, req_ids[i], layer);
    if (rc) return rc;
    for (int j = 0; j < i; ++j) if (req_ids[j] == req_ids[i]) return fail(ctx, SPIN_ERR_INVALID, "request %d listed twice", req_ids[i]);
    b.req[i] = req_ids[i];
    const LayerHost &L = ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer];
    if (with_append && cluster && !L.clustered) return fail(ctx, SPIN_ERR_STATE, "request %d has no cluster prefill yet", req_ids[i]);
    if (with_append && L.n_tokens % kPageTokens == 0) completes_page = true;     // a new page starts
  }
  const __nv_bfloat16 *kk = nullptr, *vv = nullptr;
  const void *k_alias = nullptr, *v_alias = nullptr, *q_alias = nullptr, *out_alias = nullptr;
  const size_t kv_bytes = (size_t)n_req * ctx->cfg.num_kv_heads * kRowBytes;
  const size_t qbytes = (size_t)n_req * ctx->cfg.num_q_heads * kRowBytes;
  bool in_grid = false, kv_pinned = false;
  // q and new k/v in pinned host memory: one zero-copy staging kernel brings them in
  const int qc = classify_ptr(q, &q_alias), oc = classify_ptr(out, &out_alias);
  int kc = 0;
  if (with_append) {
    // every check comes before the first change of state: a refused call leaves the context as it was
    kc = classify_ptr(k, &k_alias);
    if (kc != classify_ptr(v, &v_alias)) return fail(ctx, SPIN_ERR_INVALID, "k_new and v_new must live in the same kind of memory");
    if (int rc = precheck_append_one(ctx, layer, req_ids, n_req)) return rc;
  }
  if (int rc = wait_for_offload(ctx, st)) return rc;       // missed pages are fetched from the host tier
  if (with_append) {
    for (int i = 0; i < n_req; ++i) {
      LayerHost &L = ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer];
      int rc = cluster ? grow_cluster_tail(ctx, req_ids[i], layer, 1, st) : grow_paged(ctx, req_ids[i], layer, L.n_tokens + 1, st);
      if (rc) return rc;
    }
    kk = reinterpret_cast<const __nv_bfloat16 *>(k);
    vv = reinterpret_cast<const __nv_bfloat16 *>(v);
    if (kc == 2) {
      CK(cudaMemcpyAsync(ctx->stage_k, k, kv_bytes, cudaMemcpyHostToDevice, st));
      CK(cudaMemcpyAsync(ctx->stage_v, v, kv_bytes, cudaMemcpyHostToDevice, st));
    }
    if (kc != 0) { kk = ctx->stage_k; vv = ctx->stage_v; }
    kv_pinned = kc == 1;
    // An append that completes no page cannot change what Select sees: it then runs inside
    // the scoring kernel (one extra CTA per set).  Otherwise it runs first, on its own.
    in_grid = !completes_page;
    if (kv_pinned || qc == 1)
      ctx->launches += launch_stage_in(ctx->stage_q, qc == 1 ? q_alias : nullptr, qc == 1 ? qbytes : 0, ctx->stage_k,
                                       k_alias, ctx->stage_v, v_alias, kv_pinned ? kv_bytes : 0, st);
    if (!in_grid) {
      AppendEdgeArgs a{};
      a.n_req = n_req;
      a.layer = layer;
      for (int i = 0; i < n_req; ++i) {
        a.req[i] = req_ids[i];
        a.n_tokens[i] = (int32_t)(ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer].n_tokens - 1);
      }
      prof_mark(&ctx->prof, st, -1);
      ctx->launches += launch_append_edge(ctx->d, a, kk, vv, 1, st, &ctx->prof);
    }
  }
  int64_t max_cand = 0, max_pages = 0;
  bool may_be_empty = false;
  for (int i = 0; i < n_req; ++i) {
    LayerHost &L = ctx->reqs[(size_t)req_ids[i]].layers[(size_t)layer];
    const int64_t cand = ctx->cfg.partition_kind == SPIN_PART_TOKEN_DOT ? (int64_t)L.n_partitions * kPageTokens : L.n_partitions;
    max_cand = std::max(max_cand, cand);
    int64_t pages = cluster ? ctx->g.max_pages : std::min<int64_t>(ctx->cfg.topk, L.n_partitions);
    max_pages = std::max(max_pages, pages + L.tail_pages);
    may_be_empty = may_be_empty || L.n_tokens == 0;
    L.last_batch_pos = i;
    b.tail_pages[i] = (int16_t)L.tail_pages;
    b.tail_len[i] = (int16_t)L.tail_len;
    b.slots[i] = (int32_t)ctx->reqs[(size_t)req_ids[i]].slots;
    b.step[i] = L.steps++;
    b.n_partitions[i] = L.n_partitions;
    b.n_tokens[i] = (int32_t)(L.n_tokens - (with_append ? 1 : 0));
  }
  const __nv_bfloat16 *qd = reinterpret_cast<const __nv_bfloat16 *>(q);
  __nv_bfloat16 *od = reinterpret_cast<__nv_bfloat16 *>(out);
  if (qc == 2) CK(cudaMemcpyAsync(ctx->stage_q, q, qbytes, cudaMemcpyHostToDevice, st));
  if (qc == 1 && !with_append)
    ctx->launches += launch_stage_in(ctx->stage_q, q_alias, qbytes, nullptr, nullptr, nullptr, nullptr, 0, st);
  if (qc != 0) qd = ctx->stage_q;
  // pinned host output: the attention kernel writes it directly (visible once the stream is synchronised)
  if (oc == 1) od = reinterpret_cast<__nv_bfloat16 *>(const_cast<void *>(out_alias));
  else if (oc == 2) od = ctx->stage_out;
  prof_mark(&ctx->prof, st, -1);
  b.epoch = ++ctx->epoch;
  b.append_in_grid = in_grid ? 1 : 0;
  ctx->launches += launch_select(ctx->d, b, qd, kk, vv, (int)max_cand, st, &ctx->prof);
  ctx->launches += launch_fetch(ctx->d, st, ctx->sm_count, &ctx->prof);
  ctx->launches += launch_attention(ctx->d, b, qd, od, (int)max_pages, may_be_empty, st, &ctx->prof);
  if (oc == 2) CK(cudaMemcpyAsync(out, ctx->stage_out, qbytes, cudaMemcpyDeviceToHost, st));
  CK(cudaGetLastError());
  return SPIN_OK;
}

int spin_decode_step(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req,
                     const void *q, void *out, void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  return step_impl(ctx, layer, req_ids, n_req, nullptr, nullptr, q, out, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int spin_decode_step_append(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req,
                            const void *k_new, const void *v_new, const void *q, void *out,
                            void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (!k_new || !v_new) return fail(ctx, SPIN_ERR_INVALID, "null k_new / v_new");
  return step_impl(ctx, layer, req_ids, n_req, k_new, v_new, q, out, reinterpret_cast<cudaStream_t>(cuda_stream));
}

int spin_stats(spin_ctx *ctx, spin_stats_t *out) {
  if (!ctx || !out) return SPIN_ERR_INVALID;
  if (out->struct_size != sizeof(spin_stats_t)) return fail(ctx, SPIN_ERR_INVALID, "spin_stats_t.struct_size mismatch");
  CK(cudaDeviceSynchronize());
  Counters c{};
  CK(cudaMemcpy(&c, ctx->d.counters, sizeof c, cudaMemcpyDeviceToHost));
  const Geometry &g = ctx->g;
  out->error_bits = c.error_bits;
  out->first_error_site = c.first_site;
  for (int i = 0; i < 4; ++i) out->debug_words[i] = c.dbg[i];
  out->set_steps = c.set_steps;
  out->selected_partitions = c.selected_partitions;
  out->selected_pages = c.selected_pages;
  out->tail_pages = c.tail_pages;
  out->hit_pages = c.hit_pages;
  out->miss_pages = c.miss_pages;
  out->evicted_pages = c.evicted_pages;
  out->bypass_pages = c.bypass_pages;
  out->candidates_scored = c.candidates_scored;
  out->pcie_bytes = c.miss_pages * (uint64_t)kPageBytes;
  out->hbm_bytes = c.candidates_scored * (uint64_t)g.sum_entry_bytes +
                   (c.selected_pages + c.tail_pages) * (uint64_t)kPageBytes +
                   (c.miss_pages - c.bypass_pages) * (uint64_t)kPageBytes;
  out->kernel_launches = ctx->launches;
  out->gpu_meta_bytes = (uint64_t)ctx->gpt_segs.in_use * g.seg * sizeof(GptEntry) +
                        (uint64_t)ctx->meta_segs.in_use * g.seg * sizeof(MetaEntry) + ctx->dir_bytes_in_use +
                        (ctx->d.off_mirror ? (uint64_t)(ctx->off_segs.in_use + ctx->cpt_segs.in_use) * g.seg * 4 : 0);
  out->host_meta_bytes = (uint64_t)(ctx->off_segs.in_use + ctx->cpt_segs.in_use) * g.seg * 4;
  out->summary_bytes = (uint64_t)ctx->sum_segs.in_use * g.sum_entries * g.sum_entry_bytes;
  out->gpu_pages_in_use = (uint64_t)ctx->gpu_page_pool.in_use;
  out->host_pages_in_use = (uint64_t)ctx->host_page_pool.in_use;
  if (c.error_bits & kErrTimeout)
    return fail(ctx, SPIN_ERR_TIMEOUT, "a bounded device-side wait ran out (first check that tripped: %u)", c.first_site);
  return SPIN_OK;
}

int spin_debug_link_probe(spin_ctx *ctx, int64_t n_pages, void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (n_pages < 1 || n_pages > (1ll << 22)) return fail(ctx, SPIN_ERR_INVALID, "n_pages must be 1..4194304");
  ctx->launches += launch_link_probe(ctx->d, (int)n_pages, reinterpret_cast<cudaStream_t>(cuda_stream), ctx->sm_count);
  CK(cudaGetLastError());
  return SPIN_OK;
}

int spin_debug_launch_floor(spin_ctx *ctx, void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  ctx->launches += launch_floor(ctx->d, -(int)(++ctx->floor_calls & 0xffffff) - 1, reinterpret_cast<cudaStream_t>(cuda_stream));
  CK(cudaGetLastError());
  return SPIN_OK;
}

int spin_debug_wait_probe(spin_ctx *ctx, int32_t max_polls, void *cuda_stream) {
  if (!ctx) return SPIN_ERR_INVALID;
  if (max_polls < 1 || max_polls > 4096) return fail(ctx, SPIN_ERR_INVALID, "max_polls must be 1..4096");
  ctx->launches += launch_wait_probe(ctx->d, max_polls, reinterpret_cast<cudaStream_t>(cuda_stream));
  CK(cudaGetLastError());
  return SPIN_OK;
}

int spin_debug_dump(spin_ctx *ctx, int32_t req, int32_t layer, int32_t kv_head, spin_dump_t *o) {
  int rc = validate_req_layer(ctx, req, layer);
  if (rc) return rc;
  if (!o || o->struct_size != sizeof(spin_dump_t)) return fail(ctx, SPIN_ERR_INVALID, "bad spin_dump_t");
  if (kv_head < 0 || kv_head >= ctx->cfg.num_kv_heads) return fail(ctx, SPIN_ERR_INVALID, "kv_head out of range");
  CK(cudaDeviceSynchronize());
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  const int set = set_index(d, req, layer, kv_head);
  const SetHost &S = ctx->sets[(size_t)set];
  const LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  SetState s{};
  CK(cudaMemcpy(&s, d.state + set, sizeof s, cudaMemcpyDeviceToHost));
  o->n_tokens = s.n_tokens;
  o->step = s.step;
  o->tail_pages = s.tail_pages;
  o->tail_len = s.tail_len;
  o->n_slots = s.slots;
  o->n_partitions = s.n_partitions;
  o->n_selected = o->n_parts = o->n_pages = o->n_scores = 0;
  auto pull = [&](void *dst, const void *src, size_t bytes) { return cudaMemcpy(dst, src, bytes, cudaMemcpyDeviceToHost); };
  if (L.last_batch_pos >= 0 && s.step > 0) {
    const size_t b = (size_t)L.last_batch_pos * ctx->cfg.num_kv_heads + kv_head;
    int32_t n_sel = 0, n_parts = 0, n_pages = 0;
    CK(pull(&n_sel, d.n_sel + b, 4));
    CK(pull(&n_parts, d.n_parts + b, 4));
    CK(pull(&n_pages, d.n_pages + b, 4));
    o->n_selected = n_sel; o->n_parts = n_parts; o->n_pages = n_pages;
    if ((o->selected && n_sel > o->cap_selected) || ((o->parts || o->part_state) && n_parts > o->cap_parts) ||
        ((o->page_partition || o->page_idx || o->page_mask || o->page_slot) && n_pages > o->cap_pages))
      return fail(ctx, SPIN_ERR_INVALID, "dump capacity too small (selected %d, parts %d, pages %d)", n_sel, n_parts, n_pages);
    if (o->selected) CK(pull(o->selected, d.sel_ids + b * g.max_sel, (size_t)n_sel * 4));
    if (o->parts) CK(pull(o->parts, d.parts + b * g.max_parts, (size_t)n_parts * 4));
    if (o->part_state) CK(pull(o->part_state, d.part_state + b * g.max_parts, (size_t)n_parts * 4));
    const size_t pl = b * (size_t)(g.max_pages + g.tail_cap);
    if (o->page_partition) CK(pull(o->page_partition, d.page_part + pl, (size_t)n_pages * 4));
    if (o->page_idx) CK(pull(o->page_idx, d.page_pidx + pl, (size_t)n_pages * 4));
    if (o->page_mask) CK(pull(o->page_mask, d.page_mask + pl, (size_t)n_pages * 4));
    if (o->page_slot) CK(pull(o->page_slot, d.page_slot + pl, (size_t)n_pages * 4));
    if (o->scores) {
      // candidates of the last step: the partitions indexed before it
      const int64_t parts_then = ctx->cfg.partition_kind == SPIN_PART_CLUSTER_CENTROID ? s.n_partitions : s.n_partitions;
      const int64_t n_sc = ctx->cfg.partition_kind == SPIN_PART_TOKEN_DOT ? parts_then * kPageTokens : parts_then;
      if (n_sc > o->cap_scores) return fail(ctx, SPIN_ERR_INVALID, "dump capacity too small (scores %lld)", (long long)n_sc);
      o->n_scores = (int32_t)n_sc;
      CK(pull(o->scores, d.scores + b * (size_t)g.max_cand, (size_t)n_sc * 4));
    }
  }
  if (o->slot_partition || o->slot_page_idx || o->slot_ts || o->slot_evicted_partition || o->slot_evicted_page_idx) {
    if (s.slots > o->cap_slots) return fail(ctx, SPIN_ERR_INVALID, "dump capacity too small (slots %d)", s.slots);
    std::vector<GptEntry> ent((size_t)g.seg);
    for (int s0 = 0; s0 < s.slots; s0 += g.seg) {
      const int cnt = std::min(g.seg, s.slots - s0);
      CK(pull(ent.data(), d.gpt_pool + ((size_t)S.dir_gpt[(size_t)(s0 >> g.seg_shift)] << g.seg_shift), (size_t)cnt * sizeof(GptEntry)));
      for (int i = 0; i < cnt; ++i) {
        if (o->slot_partition) o->slot_partition[s0 + i] = ent[(size_t)i].partition;
        if (o->slot_page_idx) o->slot_page_idx[s0 + i] = ent[(size_t)i].page_idx;
        if (o->slot_ts) o->slot_ts[s0 + i] = ent[(size_t)i].ts;
      }
    }
    if (o->slot_evicted_partition || o->slot_evicted_page_idx) {
      if (!d.evict_trace) return fail(ctx, SPIN_ERR_STATE, "eviction trace needs spin_config.trace");
      std::vector<int32_t> tr((size_t)s.slots * 2);
      if (s.slots) CK(pull(tr.data(), d.evict_trace + (size_t)set * g.max_slots * 2, tr.size() * 4));
      for (int i = 0; i < s.slots; ++i) {
        if (o->slot_evicted_partition) o->slot_evicted_partition[i] = tr[(size_t)i * 2];
        if (o->slot_evicted_page_idx) o->slot_evicted_page_idx[i] = tr[(size_t)i * 2 + 1];
      }
    }
  }
  if (o->part_tokens || o->part_resident) {
    if (s.n_partitions > o->cap_partitions) return fail(ctx, SPIN_ERR_INVALID, "dump capacity too small (partitions %d)", s.n_partitions);
    std::vector<MetaEntry> ent((size_t)g.seg);
    for (int p0 = 0; p0 < s.n_partitions; p0 += g.seg) {
      const int cnt = std::min(g.seg, s.n_partitions - p0);
      CK(pull(ent.data(), d.meta_pool + ((size_t)S.dir_meta[(size_t)(p0 >> g.seg_shift)] << g.seg_shift), (size_t)cnt * sizeof(MetaEntry)));
      for (int i = 0; i < cnt; ++i) {
        if (o->part_tokens) o->part_tokens[p0 + i] = ent[(size_t)i].tokens;
        if (o->part_resident) o->part_resident[p0 + i] = ent[(size_t)i].resident;
      }
    }
  }
  return SPIN_OK;
}

int spin_debug_read_page(spin_ctx *ctx, int32_t req, int32_t layer, int32_t kv_head,
                         int32_t slot, int32_t partition, int32_t page_idx, void *out) {
  int rc = validate_req_layer(ctx, req, layer);
  if (rc) return rc;
  if (!out || kv_head < 0 || kv_head >= ctx->cfg.num_kv_heads) return fail(ctx, SPIN_ERR_INVALID, "bad arguments");
  CK(cudaDeviceSynchronize());
  const Geometry &g = ctx->g;
  const DevCtx &d = ctx->d;
  const int set = set_index(d, req, layer, kv_head);
  const SetHost &S = ctx->sets[(size_t)set];
  const LayerHost &L = ctx->reqs[(size_t)req].layers[(size_t)layer];
  if (slot >= 0) {
    if (slot >= (int32_t)S.gpu_pages.size()) return fail(ctx, SPIN_ERR_INVALID, "slot out of range");
    CK(cudaMemcpy(out, d.gpu_pages + (size_t)S.gpu_pages[(size_t)slot] * kPageBytes, kPageBytes, cudaMemcpyDeviceToHost));
    return SPIN_OK;
  }
  int64_t logical;
  if (partition < 0) {
    if (page_idx < 0 || page_idx >= L.tail_pages) return fail(ctx, SPIN_ERR_INVALID, "tail page out of range");
    logical = (int64_t)L.tail_first + page_idx;
  } else {
    if (partition >= L.n_partitions) return fail(ctx, SPIN_ERR_INVALID, "partition out of range");
    const int32_t seg = S.dir_off[(size_t)(partition >> g.seg_shift)];
    logical = (int64_t)ctx->h_off_pool[((size_t)seg << g.seg_shift) + (partition & (g.seg - 1))] + page_idx;
  }
  if (logical < 0 || logical >= (int64_t)S.host_pages.size() || S.host_pages[(size_t)logical] < 0)
    return fail(ctx, SPIN_ERR_INVALID, "page out of range");
  memcpy(out, ctx->h_pages + (size_t)S.host_pages[(size_t)logical] * kPageBytes, kPageBytes);
  return SPIN_OK;
}

}  // extern "C"
