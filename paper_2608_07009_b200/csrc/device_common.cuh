// Included by hisparse.cu (one translation unit): the state every kernel receives by value, constants, device
// helpers (bounded mbarrier wait, block scan, staging) and the bulk-copy fetch pipeline shared by the Resolve and
// replay kernels.

namespace {

thread_local int g_last_cuda_error = 0;

#define HS_CUDA(call)                                   \
  do {                                                  \
    cudaError_t e_ = (call);                            \
    if (e_ != cudaSuccess) {                            \
      g_last_cuda_error = (int)e_;                      \
      return e_ == cudaErrorMemoryAllocation ? HISPARSE_ENOMEM : HISPARSE_ECUDA; \
    }                                                   \
  } while (0)

constexpr int kThreads = 1024;       // most threads per block of the resolve / replay kernels (one block per SM)
constexpr int kThreadsSmall = 512;   // block size when the grid takes several waves: two blocks share an SM
constexpr int kFetchUnroll = 4;      // 16-byte host loads in flight per thread (probe kernel)
constexpr int32_t kMiss = -2;        // classification of a row entry: valid selection, not found resident
constexpr int32_t kDupBase = -3;     // slot-table marker (kernel-internal): repeats the missing position of row entry -(v + 3)

// Everything a kernel needs, passed by value.
struct DevState {
  int N, L, lpg, G, B, k, H, W, hshift;
  int64_t E;
  int64_t layer_pool_bytes;
  uint32_t upe;  // 16-byte units per record
  uint32_t flags;
  uint8_t *pool;
  int32_t *slot_pos;
  uint32_t *last_use;
  uint16_t *order;
  int16_t *pos2slot;               // page table entries are slots (< 16384) or -1; request r's G slices start at
                                   // p2s_off[r], p2s_stride(cap[r]) entries apart
  const int64_t *cap, *init_len, *p2s_off;
  int64_t uni_cap, uni_init_len;   // capacity / initial length when every request has the same (else -1): the kernels
                                   // then need no load for them and for p2s_off = r * G * capacity
  uint8_t *const *host;
  uint32_t *t;
  uint32_t *order_t;               // [N][G] resolve count up to which `order` is current; null = the list is never left stale
  int32_t *plan_pos, *plan_slot, *plan_n;
  int32_t *anchor_out, *anchor_hits, *anchor_misses;
  int32_t *n_appends;
  uint32_t *ticket;
  uint32_t *status;
  // Dynamic shared memory of the resolve / replay kernels (byte offsets, fixed at create): the selected row at 0
  // (its space is reused for the recency list once the row has been consumed), then the arrays below, the
  // mbarriers at meta_smem and the staging ring of the fetch pipeline behind them.
  int sm_plan_pos, sm_plan_slot;   // int32 [k] each: positions / victim slots of the misses, in selection order
  int sm_missj;                    // uint16 [k]: row index of each miss
  int sm_marks;                    // uint8: per-slot hit marks (a tag per request), zero-padded to a multiple of 2048
  int marks_spare;                 // offset (from sm_marks) of a spare byte behind the padding
  int sm_bits;                     // uint32 [4][W]: hit marks as a bitset, victim marks and their word-level prefix counts
  int sm_hist;                     // int32 [260]: histogram of the RANDOM policy's radix select
  int sm_got;                      // int16 [k]: page-table answers from the whole cluster (0 = not allocated)
  int sm_misc;                     // int32 [64]: scratch of the block scans, per-request flags
  int sm_tab;                      // uint64 [H]: table of the missing positions; -1 = it lives at the start of the ring
                                   // and is cleared only once a miss has been seen
  int meta_smem;                   // bytes of shared memory the arrays above take
  int bar_bytes;                   // (threads + 2) mbarriers: one per thread for the fetch ring, two for staging
  int io_threads, io_depth, io_chunk;  // fetch pipeline: issuing threads, ring slots per thread, bytes per piece
  int ring_bytes;                  // io_threads * io_depth * io_chunk
  int io_ppr;                      // pieces per record = ceil(E / io_chunk)
  int policy;                      // HISPARSE_POLICY_*
  unsigned long long policy_seed;  // RANDOM policy
  unsigned long long *phase_ns;    // [N][16]: 8 globaltimer stamps, then 8 SM cycle-counter stamps (PHASE_TIMERS)
  unsigned long long *layer_ns;    // [2][L]: earliest request start / latest request end of each layer's last resolve (PHASE_TIMERS)
};

// ------------------------------------------------------------------------------------------ device helpers

__device__ __forceinline__ uint4 ld_host16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Entries between the page-table slices of consecutive groups of one request: the capacity rounded up to whole
// 16-byte units, so that every slice of a library-owned table starts on a 16-byte boundary and can travel to shared
// memory as one bulk copy (the padding entries stay -1).
__host__ __device__ __forceinline__ int64_t p2s_stride(int64_t cap) { return (cap + 7) & ~(int64_t)7; }

// Multiplicative hash of a position into a table of H = 2^(32 - shift) entries.
__device__ __forceinline__ uint32_t hash_pos(int32_t p, int shift) {
  return ((uint32_t)p * 0x9E3779B1u) >> shift;
}

__device__ __forceinline__ void history_state(const DevState &d, int r, int64_t &len, int64_t &newest) {
  const int64_t na = *(volatile int32_t *)d.n_appends;
  const int64_t il = d.init_len[r], cap = d.cap[r];
  len = il + na < cap ? il + na : cap;
  newest = (na > 0 && il + na <= cap) ? il + na - 1 : -1;
}

// ---- Phase 4 (Sec. 3.4): fetch of the missing records as a bulk-async-copy (TMA) pipeline ----
//
// Records travel host -> shared memory -> cache slot with cp.async.bulk in both directions, so no thread holds
// data in registers and a block keeps its whole staging ring (up to ~150 KB) in flight over the host link.
// A record is cut into pieces of d.io_chunk bytes.  Each of the first d.io_threads threads of a block owns
// d.io_depth ring slots and one mbarrier: it issues a batch of loads (one expect_tx for the batch), goes on with
// other work, later waits for the batch, issues the stores to the cache slots and reuses its ring slots.  Threads
// never wait for one another.  Every wait is bounded (2 s of %globaltimer); on expiry STATUS_TIMEOUT is set and
// the thread stops fetching.

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  unsigned long long limit_ns = 2000000000ull) {
  uint32_t done = 0;
  uint64_t t0 = 0;
  for (uint32_t spin = 0;; ++spin) {
    // (no suspend-time hint: with a hint of 1 us a waiting warp was measured to sleep on, long after the phase had
    // completed, which made the wait for 24 KB of staged inputs take 5 us)
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if ((spin & 63u) == 63u) {
      const uint64_t now = global_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) return false;
    }
  }
}

struct TmaFetch {
  const uint8_t *hbase;
  uint8_t *pbase;
  const int32_t *s_pos, *s_slot;
  uint32_t ring, bar;      // shared-memory addresses of this thread's ring slots and mbarrier
  int64_t total;           // number of pieces to move in this request
  int part, nparts;
  int batch;
  uint32_t parity;
  bool active;
  // The pipeline's geometry (record bytes, piece size, pieces per record, ring slots per thread, issuing threads) is
  // read from the kernel's DevState argument where it is used: constant-bank reads instead of live registers.

  __device__ __forceinline__ void init(const DevState &d, int r, int layer, int m, const int32_t *pos,
                                       const int32_t *slot, unsigned char *ring_base, unsigned long long *bars,
                                       int part_, int nparts_, uint32_t parity_ = 0) {
    const int tid = threadIdx.x;
    total = (int64_t)m * d.io_ppr;
    part = part_; nparts = nparts_;
    s_pos = pos; s_slot = slot;
    hbase = d.host[r] + (int64_t)layer * d.cap[r] * d.E;
    pbase = d.pool + (int64_t)layer * d.layer_pool_bytes + (int64_t)r * (d.B + 1) * d.E;
    ring = smem_u32(ring_base) + (uint32_t)tid * (uint32_t)(d.io_depth * d.io_chunk);
    bar = smem_u32(bars + tid);
    batch = 0; parity = parity_;  // the phase this thread's barrier is in (a block that loops over requests carries it along)
    active = tid < d.io_threads && m > 0 && !(d.flags & HISPARSE_FLAG_SKIP_IO);
  }

  // piece number of this thread's q-th transfer
  __device__ __forceinline__ int64_t piece_of(const DevState &d, int q) const {
    return ((int64_t)q * d.io_threads + threadIdx.x) * nparts + part;
  }

  // Issues the loads of the next batch; false when this thread has nothing left.
  __device__ __forceinline__ bool issue(const DevState &d) {
    if (!active) return false;
    const int depth = d.io_depth, chunk = d.io_chunk, ppr = d.io_ppr;
    const int64_t E = d.E;
    uint32_t bytes_total = 0;
    for (int s = 0; s < depth; ++s) {
      const int64_t c = piece_of(d, batch * depth + s);
      if (c >= total) break;
      const int piece = ppr == 1 ? 0 : (int)(c % ppr);
      const int64_t rest = E - (int64_t)piece * chunk;
      bytes_total += (uint32_t)(rest < chunk ? rest : chunk);
    }
    if (bytes_total == 0) { active = false; return false; }
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes_total) : "memory");
    for (int s = 0; s < depth; ++s) {
      const int64_t c = piece_of(d, batch * depth + s);
      if (c >= total) break;
      const int64_t rec = ppr == 1 ? c : c / ppr;
      const int piece = (int)(c - rec * ppr);
      const int64_t rest = E - (int64_t)piece * chunk;
      const uint32_t bytes = (uint32_t)(rest < chunk ? rest : chunk);
      const uint8_t *src = hbase + (int64_t)s_pos[rec] * E + (int64_t)piece * chunk;
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(ring + (uint32_t)(s * chunk)), "l"(src), "r"(bytes), "r"(bar) : "memory");
    }
    return true;
  }

  // Waits for the batch issued last, stores it to the cache slots and frees the ring slots.  False = the bounded
  // wait expired.
  __device__ __forceinline__ bool complete(const DevState &d, uint32_t *status) {
    if (!mbar_wait_bounded(bar, parity)) {
      // Give the loads in flight one more bounded chance to land before this thread stops using its ring slots: the
      // block must not hand its shared memory to the next block while bulk copies are still writing into it.
      atomicOr(status, HISPARSE_STATUS_TIMEOUT);
      mbar_wait_bounded(bar, parity);
      active = false;
      return false;
    }
    parity ^= 1u;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const int depth = d.io_depth, chunk = d.io_chunk, ppr = d.io_ppr;
    const int64_t E = d.E;
    for (int s = 0; s < depth; ++s) {
      const int64_t c = piece_of(d, batch * depth + s);
      if (c >= total) break;
      const int64_t rec = ppr == 1 ? c : c / ppr;
      const int piece = (int)(c - rec * ppr);
      const int64_t rest = E - (int64_t)piece * chunk;
      const uint32_t bytes = (uint32_t)(rest < chunk ? rest : chunk);
      uint8_t *dst = pbase + (int64_t)s_slot[rec] * E + (int64_t)piece * chunk;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                   ::"l"(dst), "r"(ring + (uint32_t)(s * chunk)), "r"(bytes) : "memory");
    }
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // ring slots reusable
    ++batch;
    return true;
  }

  // Returns false when a bounded wait expired (the barrier's phase is then unknown).
  __device__ __forceinline__ bool drain(const DevState &d, uint32_t *status) {
    bool pending = active;  // a batch is in flight whenever the thread is still active here
    bool ok = true;
    while (pending) {
      ok = complete(d, status) && ok;
      pending = issue(d);
    }
    // complete() already waited until every store of this thread had read its ring slot (wait_group.read), which
    // is what shared memory needs before the block exits; the writes themselves are complete at grid end.
    return ok;
  }
};

// Barriers [0, blockDim.x): one per thread of the fetch pipeline; the two behind them complete the staging of the
// selected row + page-table slice and of the recency list.  Every thread of the block must pass a block barrier
// after this call before any of the barriers is used.
__device__ __forceinline__ void fetch_barriers_init(unsigned long long *bars, int io_threads) {
  if ((int)threadIdx.x < io_threads)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + threadIdx.x)) : "memory");
  if (threadIdx.x < 2)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + blockDim.x + threadIdx.x)) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

}  // namespace
