/*
 * hisparse.h — C-ABI of the B200-native HiSparse selection-resolution library.
 *
 * The library implements one thing: the per-layer selection-resolution hot path of HiSparse, a
 * hierarchical KV cache for top-k sparse-attention decoding.  For every decode step and layer a
 * batch of selected logical KV positions per request is resolved against a small fixed-size
 * per-(request, layer) GPU cache: hits are found, misses evict LRU victims, the missing records
 * are pulled from pinned host KV history over the host link by the GPU's own threads, and the
 * table of device slots that a sparse-attention kernel reads is emitted (paper Sec. 3.2-3.5).
 *
 * Conventions
 *   - Every function returns HISPARSE_OK (0) or a negative HISPARSE_E* code; nothing throws.
 *   - "dev" pointers are device pointers, "host" pointers are host pointers.  `stream` arguments
 *     are `cudaStream_t` values passed as `void *` (NULL = the legacy default stream).
 *   - append / resolve / prefetch / gather* only enqueue work; they never synchronise the host
 *     with the device and keep all step-dependent state (lengths, step counters, miss counts,
 *     miss plans) in device memory, so a sequence of them can be captured in a CUDA graph and
 *     replayed.  Create, destroy, status, dump and the probes synchronise.
 *   - The caller owns the host histories (which must stay pinned, mapped and alive until
 *     destroy), the selection / slot-table / counter buffers and the streams.  The library owns
 *     the cache pools and all metadata.
 *   - One handle is bound to one device and is not thread-safe; use one handle per GPU.
 */
#ifndef HISPARSE_H_
#define HISPARSE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hisparse hisparse_t; /* opaque, library-owned */

/* error codes */
#define HISPARSE_OK 0
#define HISPARSE_EINVAL (-1)      /* bad argument or geometry (k > B, E % 16, layer out of range ...) */
#define HISPARSE_ENOTPINNED (-2)  /* a host history is not pinned + device-mapped host memory        */
#define HISPARSE_ENOMEM (-3)      /* device or host allocation failed                                */
#define HISPARSE_ECUDA (-4)       /* a CUDA call failed; hisparse_last_cuda_error() has the code      */
#define HISPARSE_ESTATE (-5)      /* call not valid now (e.g. prefetch of a layer whose anchor has not run) */
#define HISPARSE_ETOOBIG (-6)     /* geometry exceeds the fixed scratch of hisparse_resolve_noalloc          */

/* create flags */
#define HISPARSE_FLAG_SKIP_IO 1u          /* timing mode of Sec. 4.6's "no-IO oracle": misses are resolved
                                             in metadata but no record is fetched (cache bytes go stale)   */
#define HISPARSE_FLAG_DEBUG_VALIDATE 2u   /* after every anchor resolve a checking kernel verifies that the
                                             page table and the slot array are mutual inverses and that the
                                             recency order is a permutation; failures set a status bit      */
#define HISPARSE_FLAG_INLINE_WRITE_THROUGH 4u /* append writes through on the caller's stream instead of
                                             the library's backup stream                                   */

#define HISPARSE_FLAG_PHASE_TIMERS 8u      /* the resolve kernel records %globaltimer at its phase boundaries
                                             (hisparse_phase_times); for the phase breakdown of Fig. 7        */

#define HISPARSE_FLAG_NO_PDL 16u           /* launch Resolve without programmatic dependent launch.  By default the
                                             kernel waits for its predecessor in the stream with
                                             griddepcontrol.wait and lets its own successor be scheduled early; a
                                             successor that the caller launches with programmatic stream
                                             serialization must itself wait for the grid dependency before it reads
                                             what Resolve wrote (kernels launched the ordinary way are unaffected)  */

#define HISPARSE_FLAG_EAGER_ORDER 32u      /* bring the recency list up to date in every Resolve.  By default a
                                             Resolve in which nothing missed only stamps its hits (the stamps of
                                             Sec. 3.2 are the policy's state) and leaves the list behind; the next
                                             Resolve that needs victims first re-sorts the slots stamped since
                                             (hisparse_order_lag).  Results are the same either way            */

#define HISPARSE_FLAG_WIDE_BLOCKS 64u       /* always one 1024-thread block per SM.  By default a handle whose grid
                                             would take several waves (more blocks than SMs) runs ONE resident wave
                                             of 512-thread blocks, three or two per SM, that loop over the requests,
                                             when B <= 8192 and k <= 2048 (hisparse_launch_geometry)              */

#define HISPARSE_FLAG_NARROW_BLOCKS 128u    /* always 512-thread blocks; EINVAL when the shape does not allow them
                                             (or together with WIDE_BLOCKS).  Results do not depend on the block size */

/* sticky device status bits (hisparse_status) */
#define HISPARSE_STATUS_OUT_OF_RANGE 1u   /* a selected position was outside [0, len) (and not -1)       */
#define HISPARSE_STATUS_DUPLICATE 2u      /* a position occurred twice in one row                        */
#define HISPARSE_STATUS_CAPACITY 4u       /* an append found a request's history full; it was dropped    */
#define HISPARSE_STATUS_INCONSISTENT 8u   /* DEBUG_VALIDATE found broken metadata                        */
#define HISPARSE_STATUS_TIMEOUT 16u       /* a bounded device-side wait expired                          */

/* replacement policies (hisparse_config_t.policy).  LRU with hits ranked above the step's fetched records is the
 * paper's policy (Sec. 3.2); FIFO and RANDOM are the alternatives its cache study replays (Sec. 4.3, Fig. 6):
 * FIFO - a hit does not refresh its slot (stamps record fetches only); victims are still the non-hit slots in
 * ascending (stamp, slot) order.  RANDOM - recency is kept as for LRU but victims are the m non-hit slots with the
 * smallest (key, slot), key = low 32 bits of mix64(mix64(seed ^ (r << 32 | group)) + (t << 32 | slot)), and the
 * i-th miss takes the i-th victim in ascending slot order. */
#define HISPARSE_POLICY_LRU 0
#define HISPARSE_POLICY_FIFO 1
#define HISPARSE_POLICY_RANDOM 2

/* limits */
#define HISPARSE_MAX_CACHE_SLOTS 16384
#define HISPARSE_MAX_TOP_K 4096

/*
 * Geometry of one handle (notation of the paper's Table 2: N_batch, N_l, B, k, W_KV * s).
 * A "record" is the unit the selector picks: a token's KV (DSA), a block (NSA) or a page (Quest).
 */
typedef struct {
  int32_t num_requests;      /* N: concurrent decode requests, fixed for the handle's life            */
  int32_t num_layers;        /* L: sparse-attention layers                                            */
  int32_t layers_per_group;  /* 1: every layer selects for itself.  g > 1: layers [a, a+g) share the
                                selection of their anchor layer a = multiple of g (Sec. 3.5); L % g == 0 */
  int32_t cache_slots;       /* B: LRU-managed slots per (request, layer); one more slot per (request,
                                layer) is reserved for the newest record (Sec. 3.3 step 4)              */
  int32_t top_k;             /* k: row length of sel / slot_table; 1 <= k <= B                          */
  int64_t entry_bytes;       /* E: bytes per record, a positive multiple of 16                         */
  const int64_t *capacity;   /* host [N]: maximum number of records of each request's history          */
  const int64_t *init_len;   /* host [N]: records already present in the history, <= capacity          */
  void *const *host_history; /* host [N]: base of each request's history, pinned and device-mapped host
                                memory (cudaHostAlloc / cudaHostRegister with the Mapped flag), 16-byte
                                aligned, laid out [L][capacity[r]][E]                                   */
  int32_t device;            /* CUDA device ordinal                                                    */
  uint32_t flags;            /* HISPARSE_FLAG_*                                                         */
  int32_t ctas_per_request;  /* thread blocks (one cluster) that share one request's fetch work;
                                0 = choose from N (about 32 blocks in all); otherwise 1, 2, 4 or 8             */
  int32_t policy;            /* HISPARSE_POLICY_*; 0 = the paper's LRU                                  */
  uint64_t policy_seed;      /* RANDOM policy only                                                     */
} hisparse_config_t;

/* Sec. 3.3 step (2) "Admission": reserve the per-layer caches and metadata of N requests.  All
 * caches start cold.  Validates the geometry (EINVAL) and that every history is pinned and mapped
 * (ENOTPINNED).  Synchronises. */
int hisparse_create(const hisparse_config_t *cfg, hisparse_t **out);

/* Releases everything the library owns after waiting for its outstanding work.  Synchronises. */
int hisparse_destroy(hisparse_t *h);

/* Sec. 3.3 step (4) "Write-through of generated KV": every request appends one record per layer.
 * new_kv_dev is device memory [N][L][E], 16-byte aligned (EINVAL otherwise); request r's records land at position len[r], which then
 * grows by one.  The records are placed in the reserved slot of each (request, layer) cache, so
 * the newest position is always resident, and written through to the host history on the
 * library's backup stream (on `stream` itself with INLINE_WRITE_THROUGH), ordered by events so
 * that the host copy is complete before any later fetch can reference it.  new_kv_dev may be
 * reused as soon as work enqueued on `stream` after this call runs.  A request whose history is
 * full sets STATUS_CAPACITY and keeps its length. */
int hisparse_append(hisparse_t *h, const void *new_kv_dev, void *stream);

/* Sec. 3.3 step (3) / Sec. 3.4 (the fused Resolve kernel): resolve `layer` for all N requests in
 * ONE kernel launch, one thread-block cluster per request.
 *   sel_dev        int32 [N][k]  selected positions of each request, any order; -1 = padding
 *   slot_table_dev int32 [N][k]  out: for each selection the index of its record in
 *                                hisparse_layer_pool(layer), i.e. r*(B+1) + slot with slot in [0, B]
 *                                (slot B = the reserved newest-record slot); -1 for padding and for
 *                                out-of-range positions
 *   hits_dev, misses_dev int32 [N]  out: selections found resident / fetched; hits + misses = number
 *                                of distinct valid selections of the row
 * Semantics (deterministic): selections already resident are hits, keep their slot and are stamped
 * first (recency stamp 2t+1, t = number of resolves of this (request, group) so far); the misses
 * then take the slots that were not hit, in ascending (stamp, slot) order, the i-th miss of the row
 * taking the i-th such slot, and are stamped 2t; their records are copied from the host history
 * into those slots before the kernel ends.  The anchor layer also records its miss plan.
 * For a shared layer (layer % layers_per_group != 0) sel_dev is ignored: the call waits for that
 * layer's prefetch (or, if hisparse_prefetch was not called for it since the anchor's resolve,
 * replays the anchor's plan on `stream`), then emits the anchor's table and counts (Sec. 3.5).
 * Every layer of a group must be resolved once per step, anchor first.
 * A position outside [0, len) sets STATUS_OUT_OF_RANGE and yields -1; a position repeated in a row
 * sets STATUS_DUPLICATE, takes the slot of its first occurrence and is counted once. */
int hisparse_resolve(hisparse_t *h, int layer, const int32_t *sel_dev, int32_t *slot_table_dev,
                     int32_t *hits_dev, int32_t *misses_dev, void *stream);

/* Sec. 3.5 "Exact prefetch with shared selections": replay the miss plan recorded by `layer`'s
 * anchor into `layer`'s cache with a copy-only kernel on side_stream (no probing, no LRU update),
 * ordered after the anchor's resolve by an event.  `layer` must be a shared layer whose anchor has
 * been resolved in this step (ESTATE otherwise).  The later hisparse_resolve(layer) waits for it. */
int hisparse_prefetch(hisparse_t *h, int layer, void *side_stream);

/* Sec. 3.5 "A speculative alternative": for models WITHOUT shared selections, use some other selection (the
 * paper: the previous layer's) as a hint for `layer` and bring the hinted records in ahead of the layer's own
 * resolve.  Defined here as exactly a resolve of `layer` with hint_sel_dev [N][k] as its selection, run on
 * side_stream after the work already enqueued on `stream`, with its slot table and counts discarded: hinted
 * records that were host-only are fetched (evicting LRU victims) and the hinted positions are stamped.  A wrong
 * hint costs transfers and cache space, never correctness: the layer's own hisparse_resolve, which waits for the
 * hint, still finds or fetches every selected record.  Only with layers_per_group == 1 (EINVAL otherwise). */
int hisparse_prefetch_hint(hisparse_t *h, int layer, const int32_t *hint_sel_dev, void *stream, void *side_stream);

/* Makes `stream` wait for everything the library has in flight on its own backup stream and on
 * side streams given to hisparse_prefetch.  Needed before ending a stream capture that contains an
 * append, and before the host reads the histories.  The resolve of the last layer joins the
 * write-through by itself. */
int hisparse_join(hisparse_t *h, void *stream);

/* Device base of one layer's cache pool: N*(B+1) records of E bytes (what the attention kernel
 * gathers from with the slot table).  Valid until destroy. */
const void *hisparse_layer_pool(const hisparse_t *h, int layer);

/* The sparse-attention consumer of the slot table (Sec. 2.1: attention is exact over the selected set; Sec. 3.4
 * Phase 5: the attention kernel takes the selected records out of the GPU cache through the emitted slots), for
 * records laid out as the DSA configurations have them: E = 2 D bytes = D bf16 numbers, the key of a record being all
 * D of them and its value the first value_dims (the absorbed form of multi-head latent attention; D = 576,
 * value_dims = 512 for a 512-number latent followed by a 64-number rotary key).  For every request n and head h
 *     out[n][h][:] = sum_j softmax_j(scale * q[n][h][:] . rec[n][j]) * rec[n][j][:value_dims],
 *     lse[n][h]    = log sum_j exp(scale * q[n][h][:] . rec[n][j])
 * over the entries j of slot_table_dev [N][k] (as hisparse_resolve emits it for `layer`) that are >= 0; a row with no
 * valid entry gives out = 0, lse = -inf.
 *   q_dev      bf16  [N][num_heads][D], 16-byte aligned; num_heads a multiple of 16
 *   out_dev    float [N][num_heads][value_dims]; lse_dev float [N][num_heads]
 *   value_dims 128, 256 or 512, at most D; E a multiple of 32, at most 1152 (records of up to 576 numbers)
 *   workspace_dev  device scratch of at least hisparse_attention_workspace_bytes bytes (the partial results of the
 *                  blocks that share one row), caller-owned so that the call allocates nothing; 16-byte aligned
 * Arithmetic: bf16 products accumulated in fp32 on the tensor cores, softmax weights rounded to bf16 before they
 * multiply the values: out is within 1e-2 * max |value| of the exact result (tests/test_gpu_attention.py).
 * Enqueues two kernels on `stream` after joining the library's side streams; capturable.  EINVAL for shapes the kernel
 * does not take. */
int hisparse_attention_workspace_bytes(const hisparse_t *h, int num_heads, int value_dims, size_t *bytes);
int hisparse_sparse_attention(hisparse_t *h, int layer, const void *q_dev, int num_heads, int value_dims,
                              const int32_t *slot_table_dev, float scale, float *out_dev, float *lse_dev,
                              void *workspace_dev, size_t workspace_bytes, void *stream);

/* Stand-in for the sparse-attention consumer, which takes the selected records out of the GPU cache through
 * the slot table (Sec. 3.4 Phase 5): copies the record of every table entry into
 * out_dev, uint8 [N][k][E], 16-byte aligned (EINVAL otherwise); entries with table value -1 are zero-filled. */
int hisparse_gather(hisparse_t *h, int layer, const int32_t *slot_table_dev, void *out_dev, void *stream);

/* Exactness check of Sec. 3.1 (the hierarchy moves records between tiers but never changes which positions are
 * selected or what the attention computes from them): for every valid selection compares the E bytes its table entry
 * addresses with the host history's record at that position and adds the number of differing
 * selections to *mismatches_dev (int32, not cleared).  Joins the write-through first. */
int hisparse_gather_check(hisparse_t *h, int layer, const int32_t *sel_dev, const int32_t *slot_table_dev,
                          int32_t *mismatches_dev, void *stream);

/* Sticky status bits accumulated by the device code (HISPARSE_STATUS_*).  Synchronises the device. */
int hisparse_status(hisparse_t *h, uint32_t *bits);
int hisparse_clear_status(hisparse_t *h);

/* Copies one (request, layer)'s metadata to host buffers; any pointer may be NULL.  slot_pos [B]
 * (position held by each slot, -1 = empty), last_use [B] (recency stamps), lru_order [B] (slots from
 * least to most recent as the device holds them: equal to the slots sorted by (last_use, slot) whenever
 * hisparse_order_lag reports 0), pos2slot [capacity[req]] (page table, -1 = host-only).  Synchronises. */
int hisparse_dump_state(hisparse_t *h, int req, int layer, int32_t *slot_pos, uint32_t *last_use,
                        int32_t *lru_order, int32_t *pos2slot, int64_t *len, int64_t *newest,
                        uint32_t *resolves);

/* Number of Resolves of (req, layer's group) that the recency list has not absorbed yet: Resolves in which
 * nothing missed stamp their hits and leave the list alone; the next Resolve with a miss catches up before it
 * picks victims, after which the lag is 0 again.  Always 0 with HISPARSE_FLAG_EAGER_ORDER.  The paper keeps
 * stamps only (Sec. 3.2); the list is this library's own structure.  Synchronises. */
int hisparse_order_lag(hisparse_t *h, int req, int layer, uint32_t *lag);

/* Checkpoint / resume, the counterparts of hisparse_dump_state (the paper has no such step; its scheduler only
 * releases state).  hisparse_load_appends sets how many records every request has appended so far (lengths =
 * init_len + appends; the histories must already hold those records).  hisparse_load_state then installs
 * slot_pos [B] and last_use [B] (host arrays as dumped) as the metadata of (req, layer's group): it rebuilds the page
 * table and the recency order from them, sets the resolve counter, and refills the cache of every layer of the
 * group from the host history, which is authoritative (resident records and the newest record's reserved slot).
 * EINVAL if a position is out of range or held by two slots.  Call between steps; synchronises. */
int hisparse_load_appends(hisparse_t *h, int32_t appends);
int hisparse_load_state(hisparse_t *h, int req, int layer, const int32_t *slot_pos, const uint32_t *last_use,
                        uint32_t resolves);

/* Miss plan recorded by the last resolve of `layer`'s anchor for request req: plan_pos / plan_slot
 * are host int32 [k]; *n receives the number of entries.  Synchronises. */
int hisparse_dump_plan(hisparse_t *h, int req, int layer, int32_t *plan_pos, int32_t *plan_slot, int32_t *n);

/* Device bytes a handle of this geometry allocates: the KV term N*L*(B+1)*E (Sec. 3.1 "Bounded
 * device footprint", plus the reserved slot) in *kv_bytes and the metadata in *meta_bytes. */
int hisparse_device_bytes(const hisparse_config_t *cfg, size_t *kv_bytes, size_t *meta_bytes);

/* With PHASE_TIMERS: stamps of the last anchor resolve, host uint64 [N][16], per request.
 * %globaltimer nanoseconds: [0] kernel start, [3] plan ready = fetch begins (end of Phases 1-3), [4] slot table
 * and recency order published (Phase 5), [5] this request's first block done fetching, [6] its last block done
 * fetching (Phase 4), [7] = [3]; [1], [2] unused.  SM cycle-counter readings of the first block, for splits
 * inside Phases 1-3: [15] kernel start, [8] loads issued, [9] loads landed, [10] selections looked up and
 * classified, [11] / [12] counted, before / after the barrier, [13] scanned, [14] plan ready.  Synchronises. */
int hisparse_phase_times(hisparse_t *h, uint64_t *out);

/* With PHASE_TIMERS: for every layer, when its last resolve kernel started its first request and finished its last
 * one (%globaltimer nanoseconds; host uint64 [2][L]: the L starts, then the L ends; a layer that was not resolved
 * since the last call reads start = UINT64_MAX, end = 0).  Inside a CUDA-graph replay of a whole step this gives the
 * duration of each launch and the gaps between launches without a profiler.  Synchronises, then clears the stamps. */
int hisparse_layer_times(hisparse_t *h, uint64_t *out);

/* Failure-detection self-test.  Every device-side wait of the library (on the mbarriers of its bulk copies) is
 * bounded: after 2 s it gives up, sets STATUS_TIMEOUT and the kernel returns, so a lost completion can never hang
 * the GPU.  This call runs that very wait on a barrier that nothing completes, with a limit of limit_ns
 * (<= 1 s): it must return after about that long with STATUS_TIMEOUT set (clear it with hisparse_clear_status)
 * and the handle still usable.  *waited_ns receives the time the kernel spent waiting.  Synchronises. */
int hisparse_selftest_wait_timeout(hisparse_t *h, uint64_t limit_ns, uint64_t *waited_ns);

/* Launch geometry chosen at create: thread blocks per request and threads per block. */
int hisparse_launch_geometry(const hisparse_t *h, int32_t *ctas_per_request, int32_t *threads, int32_t *smem_bytes);

/* Pinned + device-mapped host memory for histories (cudaHostAlloc, portable | mapped). */
int hisparse_host_alloc(size_t bytes, void **out);
int hisparse_host_free(void *p);

/* Host-link peak: best-of-`reps` bulk cudaMemcpyAsync of `bytes` from pinned host memory to the
 * device, timed with CUDA events; *gb_per_s = bytes / best time.  Allocates and frees its own
 * buffers.  Synchronises. */
int hisparse_host_link_probe(int device, size_t bytes, int reps, double *gb_per_s);

/* Ceiling for thread-issued scattered reads over the host link: a copy-only kernel (no metadata)
 * fetches `num_records` records of entry_bytes each from pseudo-random record slots of the pinned
 * buffer host_buf (host_bytes long) into device memory; best-of-`reps` CUDA-event time is returned
 * as *gb_per_s.  Allocates and frees its own device buffers.  Synchronises. */
int hisparse_scatter_read_probe(int device, const void *host_buf, size_t host_bytes, int64_t entry_bytes,
                                int32_t num_records, int32_t num_ctas, int reps, double *gb_per_s);

/*
 * hisparse_resolve_noalloc — Resolve for callers that must not allocate device memory.  (The paper has no
 * counterpart of this entry point; it exists for integration.)
 *
 * Who needs it: code that runs where cudaMalloc / cudaFree are off limits — an engine that has handed all of
 * HBM to its own pool allocator at start-up and forbids later driver allocations, a plugin called while the
 * host application is capturing a stream (allocation calls are illegal during capture), or a latency-critical
 * path that may not take the driver's allocation lock.  hisparse_create allocates its caches and metadata with
 * cudaMalloc, so such callers cannot use a handle.  Here the caller owns ALL persistent state of one layer's
 * caches and passes it in; the only memory the kernel needs beyond those inputs and outputs — its scratch: the
 * miss plan that the blocks of a cluster hand to one another, and a few counters — lives in a fixed array that
 * is part of the library image (about 0.5 MB of device memory on every GPU that loads the library, held until
 * the process exits).  The call allocates nothing and frees nothing, neither directly nor through a library.
 *
 * Limits (HISPARSE_ETOOBIG beyond them): num_requests <= HISPARSE_NOALLOC_MAX_REQUESTS and
 * num_requests * top_k <= HISPARSE_NOALLOC_MAX_SELECTIONS; otherwise the limits of hisparse_create apply
 * (HISPARSE_EINVAL).  One layer per state struct, no shared-selection groups, no prefetch.
 *
 * The first call on a device looks up the device address of the scratch array and raises the kernel's
 * shared-memory limit; make that first call before any stream capture begins.
 * Later calls only enqueue a memset of the scratch counters and the kernel on `stream`.
 * Every call makes state->device the current device for its own duration and restores the caller's current
 * device before it returns, so it may be called from a thread whose current device is another GPU.
 * pool_dev and every address in host_layer_dev must be 16-byte aligned (the records travel as bulk copies);
 * a misaligned pool_dev is refused with HISPARSE_EINVAL, the addresses in device memory cannot be checked.
 * Every call on a device shares the one scratch array, which keeps the previous call's contents: the call
 * clears what has to start from zero itself, and two calls whose kernels overlap on the GPU (different streams)
 * race on it — serialise them.
 *
 * Semantics are exactly those of hisparse_resolve on an anchor layer; the state arrays use the layouts listed
 * below and must start as: slot_pos = -1, last_use = 0, lru_order[r][i] = i, pos2slot = -1, resolves = 0, pool
 * arbitrary.  *status_dev (may be NULL) receives HISPARSE_STATUS_* bits by atomic OR; the caller clears it.
 */
#define HISPARSE_NOALLOC_MAX_REQUESTS 1024
#define HISPARSE_NOALLOC_MAX_SELECTIONS 65536

typedef struct {
  int32_t num_requests;          /* N                                                                     */
  int32_t cache_slots;           /* B                                                                     */
  int32_t top_k;                 /* k                                                                     */
  int64_t entry_bytes;           /* E, multiple of 16                                                     */
  int32_t device;                /* CUDA device ordinal the pointers below belong to                      */
  void *pool_dev;                /* uint8 [N][B+1][E]: this layer's cache pool (slot B = newest record)   */
  int32_t *slot_pos_dev;         /* int32 [N][B]                                                          */
  uint32_t *last_use_dev;        /* uint32 [N][B]                                                         */
  uint16_t *lru_order_dev;       /* uint16 [N][B]                                                         */
  int16_t *pos2slot_dev;         /* int16, request r's page table at [p2s_offset[r], p2s_offset[r] + capacity[r]) */
  const int64_t *capacity_dev;   /* int64 [N]                                                             */
  const int64_t *init_len_dev;   /* int64 [N]: history length before any append                           */
  const int64_t *p2s_offset_dev; /* int64 [N]                                                             */
  void *const *host_layer_dev;   /* [N] device-visible addresses of this layer's pinned host history,
                                    each laid out [capacity[r]][E]                                        */
  uint32_t *resolves_dev;        /* uint32 [N]: resolves done so far per request                          */
  const int32_t *num_appends_dev;/* int32 scalar: records appended so far (length = init_len + appends)   */
} hisparse_external_state_t;

int hisparse_resolve_noalloc(const hisparse_external_state_t *state, const int32_t *sel_dev,
                             int32_t *slot_table_dev, int32_t *hits_dev, int32_t *misses_dev,
                             uint32_t *status_dev, void *stream);

const char *hisparse_strerror(int code);
int hisparse_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* HISPARSE_H_ */
