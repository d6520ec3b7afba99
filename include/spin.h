/*
 * spin.h -- C ABI of the sparse decode step over a hierarchical (HBM + pinned host DRAM)
 * paged KV cache, after "Spin" (arXiv 2604.26837).
 *
 * One decode step of one layer runs, entirely on the GPU and on the caller's stream,
 *   Select   : score every candidate partition against the query, keep the top-k
 *              (Table 1, Select column; Section 4.1 "Select")
 *   Retrieve : residency check, bucketed-LRU replacement, CPU page lookup, page fetch
 *              from pinned host memory (Section 5.2, steps 1-4; Section 5.3, steps 1-4)
 *   Attention: softmax attention over the tokens of the selected pages plus the local tail
 *              (Section 4.1 "Attention")
 * over per-(request, layer, kv-head) "sets", each with its own partitions, summaries, four
 * two-level mapping tables (Section 5.2 "Tier-Split Mapping Table", Section 5.4) and GPU page
 * slots.  The paper defines no C interface (its interface is a Python plug-in class, Section
 * 4.2); the names below follow its five-operation pipeline (Section 4.1).
 *
 * Conventions
 *  - every call returns a spin_status; nothing throws or aborts.  Argument and state errors
 *    are found synchronously and leave the context unchanged.  Conditions met on the device
 *    (a bounds check that tripped, a page list that overflowed its scratch) set bits in a
 *    device status word that spin_stats() reports.
 *  - "device pointer" = CUDA device memory of the context's device; "host pointer" = ordinary
 *    or pinned host memory.  Where a call accepts either, it says so and finds out itself.
 *  - the caller owns every buffer it passes in (q, out, k, v, hbm_pool); the library owns the
 *    pinned host memory it allocates and frees it in spin_destroy().
 *  - one host thread per context.  Calls that take a stream only enqueue work on it.
 *  - element type of q, k, v, out, summaries: bfloat16.  head_dim must be 128, page_tokens 16.
 */
#ifndef SPIN_H
#define SPIN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SPIN_API __attribute__((visibility("default")))
#else
#define SPIN_API
#endif

typedef struct spin_ctx spin_ctx;

typedef enum spin_status {
  SPIN_OK = 0,
  SPIN_ERR_INVALID = 1,     /* bad argument */
  SPIN_ERR_STATE = 2,       /* call not allowed in this state (closed request, ...) */
  SPIN_ERR_OOM_DEVICE = 3,  /* hbm_pool too small, or a device pool ran out */
  SPIN_ERR_OOM_HOST = 4,    /* pinned allocation failed, or host pages ran out */
  SPIN_ERR_BUDGET = 5,      /* not enough free GPU pages for the requested budget */
  SPIN_ERR_CUDA = 6,        /* a CUDA runtime call failed; see spin_last_error() */
  SPIN_ERR_TIMEOUT = 7      /* a bounded device-side wait ran out */
} spin_status;

/* Partition granularity and scoring rule (Section 5.2 "Partition Abstraction"; the three
 * rules are those of the benchmark configurations). */
typedef enum spin_partition_kind {
  SPIN_PART_PAGE_MINMAX = 0,      /* partition = one page; summary = per-channel min and max
                                     of its keys; score = sum_c max(q_c*min_c, q_c*max_c) */
  SPIN_PART_TOKEN_DOT = 1,        /* partition = one token scored by q.k; the selected tokens
                                     are cached and fetched as their containing pages and
                                     attended through a per-page token mask */
  SPIN_PART_CLUSTER_CENTROID = 2, /* partition = caller-given cluster of tokens packed into
                                     1..n pages; summary = centroid; score = q.centroid */
  SPIN_PART_PAGE_MEAN = 3         /* partition = one page; summary = mean of its keys (Table 1,
                                     ShadowKV's Index: landmarks), keys added in token order in
                                     fp32, x 1/16, rounded to bf16; score = q.mean */
} spin_partition_kind;

/* Bits of spin_stats_t.error_bits (set on the device, sticky). */
#define SPIN_DEV_ERR_BOUNDS 1u      /* an index left its table; the access was skipped */
#define SPIN_DEV_ERR_PAGE_LIST 2u   /* a set selected more pages than max_selected_pages */
#define SPIN_DEV_ERR_TIMEOUT 4u     /* a bounded wait ran out */
#define SPIN_DEV_ERR_STATE 8u       /* a per-set state word disagreed with the host's count (the host's
                                       count was used and the word rewritten) */

typedef struct spin_config {
  uint32_t struct_size;         /* sizeof(spin_config), for versioning */
  int32_t device;               /* CUDA device ordinal */
  int32_t num_layers;
  int32_t num_q_heads;          /* multiple of num_kv_heads; group size 1, 2, 4 or 8 */
  int32_t num_kv_heads;
  int32_t head_dim;             /* 128 */
  int32_t page_tokens;          /* 16 */
  int32_t max_requests;         /* open requests at any time (<= 256) */
  int64_t max_context_tokens;   /* per request, prefill + decode */
  int32_t partition_kind;       /* spin_partition_kind */
  int32_t topk;                 /* partitions kept per set and step (tokens for TOKEN_DOT) */
  int32_t num_clusters;         /* CLUSTER_CENTROID: clusters per set; else 0 */
  int32_t max_selected_pages;   /* CLUSTER_CENTROID: bound on the pages of topk clusters;
                                   0 = derive (topk for the page-sized kinds) */
  int32_t max_tail_tokens;      /* CLUSTER_CENTROID: bound on decode tokens per request
                                   (they extend the always-attended tail); else ignored */
  int32_t lru_buckets;          /* n: number of timestamp values, 1..64 (Section 5.3) */
  int32_t segment_entries;      /* entries per second-level segment, power of two; 0 = 256 */
  float sm_scale;               /* softmax scale; 0 = 1/sqrt(head_dim) */
  int32_t trace;                /* != 0: record per-step eviction traces for spin_debug_dump */
  int32_t fetch_mode;           /* 0: missed pages are fetched inside the attention kernel (they
                                   cross the host link while the hits are attended from HBM);
                                   1: by a separate persistent warp-per-page copy kernel */
  int32_t host_tables_only;     /* 0: the decode kernels read the Partition Offset and CPU page
                                   tables through an HBM mirror (4 B per entry) that the append
                                   kernels keep up to date; 1: they read the pinned host tables
                                   over the host link, as in Section 5.2 (saves the mirror's HBM,
                                   but those small reads queue behind the page traffic) */
  int32_t evict_exact;          /* 0: the paper's eviction (every page up to the threshold
                                   timestamp goes, Section 5.3); 1: a variant for measuring
                                   what that over-eviction costs: of the threshold bucket only
                                   as many pages as the misses still need are taken, lowest
                                   slots first (a partition that loses a page goes whole) */
  int32_t resident_scoring;     /* how the scoring kernel is laid out when the selection continues
                                   in it: 0 = automatic (one CTA per work item; a grid that is
                                   resident all at once and draws items from a queue when a step
                                   has more than 12 items per SM, so that attention can start
                                   fetching from the first sets), 1 = always the resident
                                   form, -1 = never, 2 = the streaming form: one scoring CTA per
                                   SM fed by a ring of TMA stages, sets scored in order, one
                                   selection CTA per set behind it (query groups of up to 4) */
  int32_t reserved0;
  int64_t offload_stage_bytes;  /* 0: appended pages are written through to pinned host memory on
                                   the caller's stream (Offload, Section 4.1).  > 0: asynchronous
                                   offload: the complete pages of an append from device memory are
                                   indexed and copied into a staging ring of this many bytes of
                                   the HBM pool on the caller's stream (HBM speed), and move to
                                   host memory on a stream of the library's own; the caller's
                                   stream goes on at once (it waits only when the ring is full),
                                   and a later decode step waits for the pages it may fetch.
                                   Cluster granularity: the prefill's rows are packed into their
                                   clusters' pages in the ring, range by range of the sets'
                                   pages, and drain the same way.  At least 4 pages of every kv
                                   head must fit (4 x 8 KiB x num_kv_heads x 4 bytes) */
  int64_t gpu_cache_pages;      /* HBM pages (8 KiB each) shared by all sets' cache slots */
  int64_t host_pages;           /* pinned host pages (8 KiB each) for the complete KV */
  void *hbm_pool;               /* device pointer, 256-byte aligned, caller-owned */
  size_t hbm_pool_bytes;        /* >= spin_required_bytes() */
} spin_config;

/* Counters since spin_create(); spin_stats() synchronises the device to read them. */
typedef struct spin_stats_t {
  uint32_t struct_size;
  uint32_t error_bits;            /* SPIN_DEV_ERR_* */
  uint64_t set_steps;             /* decode steps x sets */
  uint64_t selected_partitions;   /* partitions handed to the cache manager */
  uint64_t selected_pages;        /* their pages (tail pages not counted) */
  uint64_t tail_pages;            /* always-attended local pages read */
  uint64_t hit_pages;
  uint64_t miss_pages;            /* fetched or bypassed: every one crosses the host link */
  uint64_t evicted_pages;
  uint64_t bypass_pages;          /* missed pages attended straight from host memory */
  uint64_t candidates_scored;     /* summaries read by Select */
  uint64_t pcie_bytes;            /* miss_pages x page bytes (Eq. 3, rho x KV_topk) */
  uint64_t hbm_bytes;             /* modelled: summaries + selected KV + miss writes (Eq. 1-2) */
  uint64_t kernel_launches;       /* kernels this library launched */
  uint64_t gpu_meta_bytes;        /* second-level segments + directories in HBM, in use */
  uint64_t host_meta_bytes;       /* second-level segments in pinned host memory, in use */
  uint64_t summary_bytes;         /* summary segments in HBM, in use */
  uint64_t gpu_pages_in_use;
  uint64_t host_pages_in_use;
  uint64_t first_error_site;      /* where the first device-side check tripped: source file id x
                                     100000 + line (1 append, 2 select, 3 cache, 4 attention); 0 = none */
  uint32_t debug_words[4];        /* first SPIN_DEV_ERR_STATE: set index + 1, the device's token count,
                                     the host's, the decode call's number (-1: stand-alone append) */
} spin_stats_t;

/* Logical view of one set after its last decode step (what the parity tests compare).
 * The caller allocates every array and states its capacity; the call fills the n_* counts
 * and fails with SPIN_ERR_INVALID if a capacity is too small.  Any array pointer may be
 * NULL to skip it. */
typedef struct spin_dump_t {
  uint32_t struct_size;
  int32_t cap_selected, cap_parts, cap_pages, cap_slots, cap_partitions, cap_scores;
  int32_t n_selected;   int32_t *selected;         /* chosen candidate ids, ascending */
  int32_t n_parts;      int32_t *parts;            /* partitions given to the cache manager */
                        int32_t *part_state;       /* 0 hit, 1 miss admitted, 2 miss bypassed */
  int32_t n_pages;      int32_t *page_partition;   /* attention order; -1 for a tail page */
                        int32_t *page_idx;
                        uint32_t *page_mask;       /* bit r set = token r of the page attended */
                        int32_t *page_slot;        /* set-local slot, -1 bypassed, -2 tail */
  int32_t n_slots;      int32_t *slot_partition;   /* -1 = empty */
                        int32_t *slot_page_idx;
                        int32_t *slot_ts;          /* -1 = empty */
                        int32_t *slot_evicted_partition; /* evicted from this slot in the last
                                                      step, else -1 (needs config.trace) */
                        int32_t *slot_evicted_page_idx;
  int32_t n_partitions; int32_t *part_tokens;      /* Meta-partition table: token count */
                        int32_t *part_resident;    /* Meta-partition table: residency 0/1 */
  int32_t n_scores;     float *scores;             /* last step's candidate scores */
  int64_t n_tokens;                                /* tokens appended so far */
  int32_t step;                                    /* decode steps done (t of the next one) */
  int32_t tail_pages, tail_len;
} spin_dump_t;

/* Device and pinned-host bytes a context with this configuration needs (hbm_pool and
 * hbm_pool_bytes are ignored).  Host call, no CUDA work. */
SPIN_API int spin_required_bytes(const spin_config *cfg, size_t *device_bytes, size_t *host_bytes);

/* Build a context on cfg->device inside cfg->hbm_pool; allocates the pinned host tier.
 * Synchronous.  *out is NULL on failure. */
SPIN_API int spin_create(const spin_config *cfg, spin_ctx **out);
SPIN_API int spin_destroy(spin_ctx *ctx);

/* Open a request whose every (layer, kv-head) set gets `hbm_budget_pages_per_set` GPU page
 * slots (Section 5.3: per-request GPU buffer, per-head replacement), all empty (cold cache).
 * Synchronous. */
SPIN_API int spin_request_open(spin_ctx *ctx, int64_t hbm_budget_pages_per_set, int32_t *out_req);
/* Buffer elasticity (Section 5.3 "Buffer Elasticity"): change the GPU page slots of every set
 * of an open request between decode steps.  Shrinking reclaims the tail of each set's GPU page
 * table; a partition with a page in the reclaimed tail becomes non-resident as a whole (the
 * paper does not say what happens to a straddling partition); its pages and the reclaimed
 * slots' physical pages go back to the pool.  Growing appends empty slots (SPIN_ERR_BUDGET if
 * the pool cannot cover them).  Timestamps of surviving pages are untouched.  Synchronous: it
 * waits for the device before and after.  The policy -- when to resize whom -- is the caller's
 * (the paper's scheduler); this is the mechanism. */
SPIN_API int spin_set_budget(spin_ctx *ctx, int32_t req, int64_t hbm_budget_pages_per_set);
/* Index during decode, cluster granularity (Section 4.1 "Index": it also runs from time to time
 * during decode so that new tokens are taken in; the rule is left to the algorithm).  Folds the FULL
 * pages of the local tail of every kv head's set of (request, layer) into the clusters: each
 * token, in arrival order, joins the cluster whose centroid scores highest against its key
 * (the fp32 summation order of Select, ties to the lower cluster id) and goes to the end of
 * that cluster (a new host page when its last one is full); centroids stay as they are.  A
 * cluster that takes a token loses its GPU residency (the cached copy is stale): flag and
 * slots cleared.  The partly filled newest page stays the tail.  The set's CPU page table and
 * Partition Offset table are laid out afresh.  Host-driven and synchronous: the call waits for
 * the stream twice (it needs the assignment on the host) and returns when the fold is done.
 * At most 2048 tail tokens per call.  SPIN_ERR_INVALID for the other granularities,
 * SPIN_ERR_STATE before the cluster prefill, SPIN_ERR_OOM_HOST if host pages run out (nothing
 * has been changed then). */
SPIN_API int spin_reindex(spin_ctx *ctx, int32_t req, int32_t layer, void *cuda_stream);

/* Give back the request's pages and segments.  No work of this request may be in flight. */
SPIN_API int spin_request_close(spin_ctx *ctx, int32_t req);

/* Index + Offload (Section 4.1): append n_tokens tokens to every kv-head set of
 * (req, layer).  k, v: bf16 [n_tokens][num_kv_heads][head_dim], device or host pointer.
 * The complete KV goes to the pinned host tier (written through by the GPU), summaries stay
 * in HBM.  Page-sized kinds: a page becomes a candidate when the first token of the next
 * page arrives; the newest page is the local tail.  CLUSTER_CENTROID: the first call of a
 * (req, layer) is the prefill and must pass token_partition int32 [n_tokens][num_kv_heads]
 * (cluster of each token, 0..num_clusters-1; device or host pointer) and centroids bf16
 * [num_clusters][num_kv_heads][head_dim]; later calls pass NULL for both and extend the
 * tail.  The prefill form synchronises; single-token appends only enqueue on `cuda_stream`
 * (a cudaStream_t, NULL = default stream). */
SPIN_API int spin_append_kv(spin_ctx *ctx, int32_t req, int32_t layer, const void *k, const void *v,
                   int64_t n_tokens, const int32_t *token_partition, const void *centroids,
                   void *cuda_stream);

/* Decode-time form: one new token for each of n_req requests of one layer.
 * k, v: bf16 [n_req][num_kv_heads][head_dim], device or host pointer.  Asynchronous. */
SPIN_API int spin_append_kv_batch(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req,
                         const void *k, const void *v, void *cuda_stream);

/* One decode step of one layer for a batch of requests: Select -> Retrieve -> Attention.
 * req_ids: host array of n_req distinct open requests.  q, out: bf16
 * [n_req][num_q_heads][head_dim], device or host pointer (host buffers are copied on the
 * stream; read `out` after synchronising it).  Asynchronous on cuda_stream; no host
 * synchronisation inside.  Advances each set's step counter. */
SPIN_API int spin_decode_step(spin_ctx *ctx, int32_t layer, const int32_t *req_ids, int32_t n_req,
                     const void *q, void *out, void *cuda_stream);

/* The decode loop's usual pair in one call: spin_append_kv_batch(k_new, v_new) followed by
 * spin_decode_step(q, out), same arguments and results.  When the appended tokens complete no
 * page (15 steps out of 16), the append runs inside the scoring kernel (one extra CTA per set)
 * instead of in a launch of its own.  Asynchronous on cuda_stream. */
SPIN_API int spin_decode_step_append(spin_ctx *ctx, int32_t layer, const int32_t *req_ids,
                                     int32_t n_req, const void *k_new, const void *v_new,
                                     const void *q, void *out, void *cuda_stream);

/* Counters and sticky device error bits.  Synchronises the device.  `out` is always filled; the
 * status is SPIN_ERR_TIMEOUT (instead of SPIN_OK) when SPIN_DEV_ERR_TIMEOUT is among the bits:
 * a kernel gave up a bounded wait, so results since then are void (the other bits report
 * accesses that were skipped and leave the status at SPIN_OK). */
SPIN_API int spin_stats(spin_ctx *ctx, spin_stats_t *out);

/* Measures what the host link gives a kernel (Section 5.5 aims to saturate it; Eq. 3's BW_PCIe):
 * reads `n_pages` pages of 8 KiB of the context's pinned host tier (wrapping around it) with a
 * grid that fills the GPU, a warp per page as the page fetch does, and discards them.  The
 * caller times it with events on cuda_stream: n_pages x 8192 bytes over the elapsed time is the
 * rate of SM-issued reads over the link.  Asynchronous; no state is changed. */
SPIN_API int spin_debug_link_probe(spin_ctx *ctx, int64_t n_pages, void *cuda_stream);

/* The latency floor of a decode step in this design (Section 5.3 keeps control on the GPU: a step
 * is two kernels chained by programmatic dependent launch that hand work over through flags):
 * enqueues two one-warp kernels launched the same way, the second of which waits for a flag the
 * first raises, and nothing else.  Timed by the caller with events on cuda_stream, it is what a
 * step costs before it has touched a byte of KV; a single-set step is a small multiple of it.
 * Asynchronous. */
SPIN_API int spin_debug_launch_floor(spin_ctx *ctx, void *cuda_stream);

/* Exercises the bounded-wait path (Section 5.3 keeps all control on the GPU, so kernels of a
 * step wait on one another's flags; every such wait has a poll limit): one warp polls, at most
 * `max_polls` times (1..4096, well under a millisecond), a flag word for a value that is never
 * published, gives up, sets SPIN_DEV_ERR_TIMEOUT and returns.  Nothing else is touched; the
 * context stays usable, the bit is sticky.  Asynchronous on cuda_stream. */
SPIN_API int spin_debug_wait_probe(spin_ctx *ctx, int32_t max_polls, void *cuda_stream);

/* Per-kernel timing (tracing aid, off by default).  spin_profile(ctx, 1) synchronises, clears
 * the record and makes every later append / decode call record a CUDA event after each kernel
 * it launches on the caller's stream (up to 32768 marks, then recording stops);
 * spin_profile_read() synchronises and returns, per kernel, its launches and the summed
 * event-to-event time.  Kernel order: 0 append, 1 score, 2 top-k, 3 cache manager (LRU +
 * translation), 4 page fetch, 5 attention splits, 6 attention merge. */
typedef struct spin_profile_t {
  uint32_t struct_size;
  uint32_t n_kernels;
  uint64_t launches[8];
  double ms[8];
} spin_profile_t;
SPIN_API int spin_profile(spin_ctx *ctx, int32_t enable);
SPIN_API int spin_profile_read(spin_ctx *ctx, spin_profile_t *out);

/* Logical state of one set (see spin_dump_t).  Synchronises the device. */
SPIN_API int spin_debug_dump(spin_ctx *ctx, int32_t req, int32_t layer, int32_t kv_head, spin_dump_t *d);

/* Copy one 8 KiB page (K rows then V rows) to `out` (host pointer): the GPU slot `slot` of
 * the set, or with slot < 0 the host-tier page `page_idx` of `partition` (partition -1 =
 * tail page number page_idx).  Synchronises the device. */
SPIN_API int spin_debug_read_page(spin_ctx *ctx, int32_t req, int32_t layer, int32_t kv_head,
                         int32_t slot, int32_t partition, int32_t page_idx, void *out);

/* Paged attention that allocates nothing (the paper has no counterpart: it is an addition for
 * callers that cannot allocate GPU memory -- code that runs inside another component's fixed
 * memory budget, or on a path where touching an allocator is forbidden -- and therefore
 * cannot create a context, whose scratch comes out of a caller-allocated pool).
 * It runs the same split-K attention + log-sum-exp merge as spin_decode_step's last stage over
 * page lists the caller supplies; the split-K partials and counters use an 8 MiB array built into the
 * library image (every GPU that loads the library holds it until the process exits).
 *   q, out      bf16 [n_sets][group][128], device pointers (out is written)
 *   page_pool   device pointer to 8 KiB pages: 16 K rows then 16 V rows of 128 bf16
 *   page_ids    int32 [n_sets][list_stride], device: pages of each set.  The call does not know
 *               the pool's size: an id is only checked for being non-negative (a negative id is
 *               skipped, its page contributes nothing); that ids lie inside the pool is the
 *               caller's responsibility
 *   page_masks  uint32 [n_sets][list_stride], device: bit r set = token r of that page attended
 *   n_pages     int32 [n_sets], device: entries used per set; values outside 0..list_stride are
 *               clamped into that range.  A set without pages gets a zero output
 *   group       query heads per set: 1, 2, 4 or 8;  sm_scale 0 = 1/sqrt(128)
 * Limit: n_sets x ceil(list_stride/8) x group x 130 + n_sets (rounded up to 64) <= 2097152
 * four-byte words; a larger request is refused with SPIN_ERR_INVALID and a message on stderr,
 * nothing is launched.
 * The first call on each device looks up the built-in array's device address (no allocation);
 * make that first call outside any stream capture.  Asynchronous on cuda_stream.  All calls
 * share the one array and it keeps the previous call's contents; the call clears the per-set
 * arrival counters at its start (the only part that must begin at zero) and overwrites what
 * else it later reads, but two calls whose kernels can overlap on the GPU (different streams,
 * no ordering) would race on it. */
SPIN_API int spin_paged_attention_static(const void *q, const void *page_pool,
                                         const int32_t *page_ids, const uint32_t *page_masks,
                                         const int32_t *n_pages, int32_t n_sets,
                                         int32_t list_stride, int32_t group, float sm_scale,
                                         void *out, void *cuda_stream);

/* Text of the last error on this context (never NULL; valid until the next call). */
SPIN_API const char *spin_last_error(spin_ctx *ctx);

/* Library version string. */
SPIN_API const char *spin_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPIN_H */
