// HiSparse selection resolution for B200 (sm_100a): kernels and the C-ABI declared in hisparse.h.
//
// Data layout in HBM (N requests, L layers in G = L / layers_per_group groups, B slots, k selections,
// E bytes per record):
//   pool      uint8  [L][N][B+1][E]   cache pools; slot B of each (r, l) is the reserved newest-record slot
//   slot_pos  int32  [N][G][B]        position held by each slot, -1 = empty
//   last_use  uint32 [N][G][B]        recency stamps: 2t+1 hit at resolve t, 2t fetched at resolve t, 0 unused
//   order     uint16 [N][G][B]        slots from least to most recent: equal to sorting the slots by (last_use,
//                                     slot) whenever order_t == t.  Kept so that victim choice is a prefix scan,
//                                     not a sort; resolves without misses leave it behind (rebuild_order)
//   order_t   uint32 [N][G]           resolve count the list is current for
//   pos2slot  int16  ragged [N][G][capacity[r]]  the page table (Sec. 3.2), -1 = host-only
//   plan_*    int32  [N][G][k]        miss plan of the last anchor resolve (Sec. 3.5)
// All step-dependent scalars (resolve counters, number of appends, plan sizes) live in device memory so
// that every launch is replayable from a CUDA graph.
//
// The Resolve kernel (Sec. 3.4, Phases 1-5) runs one thread-block cluster per request.  The cluster's first
// block does the metadata: it stages the selected row, the recency order and (when it fits) the request's slice of
// the page table in shared memory with bulk copies, looks every selection up in the page table, marks hit slots in
// a bitset and compacts the misses in selection order (one block scan).  As soon as the missing positions exist the
// records start travelling host -> shared memory -> cache slot with cp.async.bulk in both directions (Phase 4);
// while the first loads fly the block walks the recency order once (a second scan) to split the non-hit slots
// into the first m (victims, needed only when a record is stored) and the rest, and rewrites the order as
// (untouched ++ victims by slot ++ hits by slot); the plan is published to the other blocks of the
// cluster, which take their share of the records, so the fetch parallelism does not depend on the number of
// requests.  A resolve in which nothing missed stops after the lookups: slot table, hit stamps, counters.
// The launch carries the programmatic-dependent-launch attribute: everything before
// griddepcontrol.wait depends on nothing an earlier kernel wrote.  Blocks have 1024 threads and an SM each;
// grids of more blocks than SMs run the 512-thread instantiation, two blocks per SM.
#include "hisparse.h"

#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

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
constexpr int kBarBytes = (kThreads + 2) * 8;  // one mbarrier per thread for the fetch ring + one for staging
constexpr int32_t kMiss = -2;        // s_out marker: valid selection, not (yet) found resident
constexpr int32_t kDupBase = -3;     // s_out marker: duplicate of row entry -(v + 3)
constexpr int32_t kRankBase = -(1 << 20);  // s_out marker: the (kRankBase - v)-th miss of the row (slot = plan_slot of it)

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
  int16_t *pos2slot;               // page table entries are slots (< 16384) or -1
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
  int meta_smem;                   // bytes of shared memory the metadata arrays take (ring follows)
  int io_threads, io_depth, io_chunk;  // fetch pipeline: issuing threads, ring slots per thread, bytes per piece
  int ring_bytes;                  // io_threads * io_depth * io_chunk
  int io_ppr;                      // pieces per record = ceil(E / io_chunk)
  int policy;                      // HISPARSE_POLICY_*
  unsigned long long policy_seed;  // RANDOM policy
  unsigned long long *phase_ns;    // [N][16]: 8 globaltimer stamps, then 8 SM cycle-counter stamps (PHASE_TIMERS)
};

// ------------------------------------------------------------------------------------------ device helpers

__device__ __forceinline__ uint4 ld_host16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

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
                                       int part_, int nparts_) {
    const int tid = threadIdx.x;
    total = (int64_t)m * d.io_ppr;
    part = part_; nparts = nparts_;
    s_pos = pos; s_slot = slot;
    hbase = d.host[r] + (int64_t)layer * d.cap[r] * d.E;
    pbase = d.pool + (int64_t)layer * d.layer_pool_bytes + (int64_t)r * (d.B + 1) * d.E;
    ring = smem_u32(ring_base) + (uint32_t)tid * (uint32_t)(d.io_depth * d.io_chunk);
    bar = smem_u32(bars + tid);
    batch = 0; parity = 0;
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

  // Waits for the batch issued last, stores it to the cache slots and frees the ring slots.
  __device__ __forceinline__ void complete(const DevState &d, uint32_t *status) {
    if (!mbar_wait_bounded(bar, parity)) {
      atomicOr(status, HISPARSE_STATUS_TIMEOUT);
      active = false;
      return;
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
  }

  __device__ __forceinline__ void drain(const DevState &d, uint32_t *status) {
    bool pending = active;  // a batch is in flight whenever the thread is still active here
    while (pending) {
      complete(d, status);
      pending = issue(d);
    }
    // complete() already waited until every store of this thread had read its ring slot (wait_group.read), which
    // is what shared memory needs before the block exits; the writes themselves are complete at grid end.
  }
};

__device__ __forceinline__ void fetch_barriers_init(unsigned long long *bars, int io_threads) {
  if ((int)threadIdx.x < io_threads)
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + threadIdx.x)) : "memory");
  if (threadIdx.x == 0)  // the staging barrier of the page-table slice
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + kThreads)) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// ------------------------------------------------------------------------------------------ Resolve (Sec. 3.4)

// Block-wide exclusive prefix sum of one int per thread (one barrier).  s_warp: 32 ints of scratch, which the
// caller must not reuse (another scan included) before the block has passed a barrier of its own.
__device__ __forceinline__ int block_scan_excl(int v, int *s_warp, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  const int w = lane < nw ? s_warp[lane] : 0;
  int wincl = w;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, wincl, o);
    if (lane >= o) wincl += n;
  }
  const int warp_excl = __shfl_sync(0xffffffffu, wincl - w, warp);
  total = __shfl_sync(0xffffffffu, wincl, 31);
  return warp_excl + incl - v;
}

// Asynchronous global -> shared staging (cp.async, 16 bytes per thread and step); falls back to plain 4- or
// 2-byte copies when the size or an address is not a multiple of 16.  Complete after cp.async.wait_all + barrier.
__device__ __forceinline__ void stage_async(void *smem_dst, const void *gmem_src, int bytes) {
  const uint32_t sdst = (uint32_t)__cvta_generic_to_shared(smem_dst);
  if (((bytes | (int)sdst | (int)(uintptr_t)gmem_src) & 15) == 0) {
    for (int o = threadIdx.x * 16; o < bytes; o += blockDim.x * 16)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sdst + o), "l"((const char *)gmem_src + o) : "memory");
  } else if (((bytes | (int)sdst | (int)(uintptr_t)gmem_src) & 3) == 0) {
    for (int o = threadIdx.x * 4; o < bytes; o += blockDim.x * 4)
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sdst + o), "l"((const char *)gmem_src + o) : "memory");
  } else {
    for (int o = threadIdx.x * 2; o < bytes; o += blockDim.x * 2)
      *reinterpret_cast<uint16_t *>((char *)smem_dst + o) = *reinterpret_cast<const uint16_t *>((const char *)gmem_src + o);
  }
}

// The selected set as an open-addressing hash table in shared memory (Phase 1): one 8-byte entry per bucket,
// (position << 32) | row index, all ones = empty.  Key and value travel in one load, and several independent
// probe sequences per thread are advanced together so that their shared-memory latencies overlap.
constexpr unsigned long long kEmptyEntry = ~0ull;
constexpr int kSelPerThread = HISPARSE_MAX_TOP_K / kThreads;  // row entries per thread

template <int N>
__device__ __forceinline__ void table_lookup(const unsigned long long *tab, const uint32_t mask, const int shift,
                                             const int32_t (&key)[N], int32_t (&found)[N]) {
  uint32_t h[N];
  uint32_t open = 0;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    found[i] = -1;
    h[i] = hash_pos(key[i], shift);
    if (key[i] >= 0) open |= 1u << i;
  }
  for (uint32_t round = 0; open && round <= mask; ++round) {
    unsigned long long e[N];
#pragma unroll
    for (int i = 0; i < N; ++i)
      if ((open >> i) & 1u) e[i] = tab[h[i]];
#pragma unroll
    for (int i = 0; i < N; ++i)
      if ((open >> i) & 1u) {
        if ((int32_t)(e[i] >> 32) == key[i]) {
          found[i] = (int32_t)(uint32_t)e[i];
          open &= ~(1u << i);
        } else if (e[i] == kEmptyEntry) {
          open &= ~(1u << i);
        } else {
          h[i] = (h[i] + 1u) & mask;
        }
      }
  }
}


// Key of the RANDOM replacement policy for one slot at resolve t of (request r, group g): the low 32 bits of
// mix64(mix64(seed ^ (r << 32 | g)) + (t << 32 | slot)), mix64 being the splitmix64 finaliser after adding its
// golden-ratio increment.  Victims are the m candidate slots with the smallest (key, slot).
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__device__ __forceinline__ uint32_t random_key(unsigned long long base, uint32_t t, int slot) {
  return (uint32_t)mix64(base + (((unsigned long long)t << 32) | (uint32_t)slot));
}

// RANDOM policy: marks in s_vicbits the m slots without a hit bit that have the smallest (key, slot).
// Radix select, most significant byte first, with a 256-bin histogram in shared memory (s_hist: 257 ints).
template <int IPT>
__device__ __forceinline__ void select_random_victims(const int B, const int m, const unsigned long long base,
                                                      const uint32_t t, const uint32_t *s_hitbits, uint32_t *s_vicbits,
                                                      int *s_hist, int *s_warp) {
  const int tid = threadIdx.x;
  if (m == 0) return;
  uint32_t key[IPT];
  uint32_t cand = 0;  // this thread owns slots tid*IPT .. tid*IPT+IPT-1 (consecutive: ties are broken by slot)
#pragma unroll
  for (int i = 0; i < IPT; ++i) {
    const int s = tid * IPT + i;
    key[i] = 0;
    if (s < B && !((s_hitbits[s >> 5] >> (s & 31)) & 1u)) {
      cand |= 1u << i;
      key[i] = random_key(base, t, s);
    }
  }
  uint32_t prefix = 0;
  int remaining = m;
#pragma unroll 1
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 257; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
#pragma unroll
    for (int i = 0; i < IPT; ++i)
      if (((cand >> i) & 1u) && (shift == 24 || (key[i] >> (shift + 8)) == prefix))
        atomicAdd(&s_hist[(key[i] >> shift) & 255u], 1);
    __syncthreads();
    if (tid == 0) {  // the byte at which the running count reaches `remaining`
      int acc = 0, b = 0;
      for (; b < 255; ++b) {
        if (acc + s_hist[b] >= remaining) break;
        acc += s_hist[b];
      }
      s_hist[256] = (b << 16) | acc;  // acc < 2^15 (at most B candidates)
    }
    __syncthreads();
    const int packed = s_hist[256];
    prefix = (prefix << 8) | (uint32_t)(packed >> 16);
    remaining -= packed & 0xffff;
    __syncthreads();
  }
  // keys below the threshold are victims; of the keys equal to it, the first `remaining` in slot order
  uint32_t eq = 0;
#pragma unroll
  for (int i = 0; i < IPT; ++i)
    if ((cand >> i) & 1u) {
      const int s = tid * IPT + i;
      if (key[i] < prefix) atomicOr(&s_vicbits[s >> 5], 1u << (s & 31));
      else if (key[i] == prefix) eq |= 1u << i;
    }
  int total;
  int rank = block_scan_excl(__popc(eq), s_warp, total);
#pragma unroll
  for (int i = 0; i < IPT; ++i)
    if ((eq >> i) & 1u) {
      const int s = tid * IPT + i;
      if (rank < remaining) atomicOr(&s_vicbits[s >> 5], 1u << (s & 31));
      ++rank;
    }
  __syncthreads();
}


// Page-table lookups shared by the blocks of a cluster (used when a request's slice of the table is too large to
// stage in shared memory: k uncoalesced reads are bound by one SM's load path, so each block of the cluster does
// k/S of them).  Block `part` answers row entries [part*chunk, (part+1)*chunk) and stores the answers (slot, or -1
// for padding / out of range / host-only) into the FIRST block's s_got through distributed shared memory.
// Cluster barrier phases: every block arrives on phase A when it starts; a block stores into the first block's
// memory only after waiting for phase A (all blocks are running by then); phase B = all answers are in.
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// phase A only says "this block is running": no memory needs to be ordered by it
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait_relaxed() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }

template <int T>
__device__ __forceinline__ void cluster_lookups(const int32_t *__restrict__ row, const int16_t *__restrict__ p2s,
                                                const int k, const int64_t len, const int part, const int S,
                                                int16_t *s_got) {
  constexpr int kMaxPer = (HISPARSE_MAX_TOP_K / 2 + T - 1) / T;  // S >= 2, so a block's share <= k/2
  const int chunk = (k + S - 1) / S;
  const int lo = part * chunk, hi = lo + chunk < k ? lo + chunk : k;
  int16_t v[kMaxPer];
#pragma unroll
  for (int i = 0; i < kMaxPer; ++i) {
    const int j = lo + (int)threadIdx.x + i * T;
    v[i] = -1;
    if (j < hi) {
      const int32_t p = __ldg(row + j);
      if (p >= 0 && (int64_t)p < len) v[i] = __ldg(p2s + p);
    }
  }
  cluster_wait_relaxed();  // phase A: the first block is running, its shared memory may be written
  uint32_t remote_base;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote_base) : "r"(smem_u32(s_got)), "r"(0));
#pragma unroll
  for (int i = 0; i < kMaxPer; ++i) {
    const int j = lo + (int)threadIdx.x + i * T;
    if (j < hi) asm volatile("st.shared::cluster.u16 [%0], %1;" ::"r"(remote_base + 2u * (uint32_t)j), "h"(v[i]) : "memory");
  }
  cluster_arrive();  // phase B
  cluster_wait();
}

// Brings a stale recency list up to date.  A resolve without misses leaves the list alone and only stamps its
// hits, so the list may lag `nsteps` resolves behind the stamps; every slot stamped since (last_use >= thr, all of
// them hit stamps thr+1, thr+3, ..) belongs behind the untouched slots, ordered by (stamp, slot).  The untouched
// slots keep their old relative order (one scan, compacted in place); the touched ones are laid out by slot behind
// them and then sorted by the step that stamped them with one stable in-place split per bit of the step index
// (no pass at all when a single resolve is outstanding).  s_bits / s_pre: W words each, s_bits is zero on return.
template <int T, int IPT>
__device__ __forceinline__ void rebuild_order(const int B, const int W, const uint32_t *__restrict__ last_use,
                                              const uint32_t thr, const uint32_t nsteps, uint16_t *s_order,
                                              uint32_t *s_bits, int32_t *s_pre, int *s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int sb = 0; sb < B; sb += T) {  // the loop bound is uniform, so every lane takes part in the ballot
    const int s = sb + tid;
    const uint32_t word = __ballot_sync(0xffffffffu, s < B && last_use[s] >= thr);
    if (lane == 0 && (s >> 5) < W) s_bits[s >> 5] = word;
  }
  __syncthreads();
  if (warp == 0) {
    int run = 0;
    for (int wb = 0; wb < W; wb += 32) {
      const int w = wb + lane;
      const int c = w < W ? __popc(s_bits[w]) : 0;
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      if (w < W) s_pre[w] = run + inc - c;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
  }
  int n_un;
  {
    int slot[IPT];
    uint32_t un_mask = 0;
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int q = tid * IPT + i;
      slot[i] = 0;
      if (q < B) {
        slot[i] = s_order[q];
        if (!((s_bits[slot[i] >> 5] >> (slot[i] & 31)) & 1u)) un_mask |= 1u << i;
      }
    }
    int rank = block_scan_excl(__popc(un_mask), s_warp, n_un);  // its barrier also publishes s_pre
#pragma unroll
    for (int i = 0; i < IPT; ++i)
      if ((un_mask >> i) & 1u) s_order[rank++] = (uint16_t)slot[i];  // in place: everything was read before the barrier
  }
  for (int s = tid; s < B; s += T) {
    const int w = s >> 5;
    const uint32_t bit = 1u << (s & 31), tw = s_bits[w];
    if (tw & bit) s_order[n_un + s_pre[w] + __popc(tw & (bit - 1u))] = (uint16_t)s;
  }
  __syncthreads();
  for (int i = tid; i < W; i += T) s_bits[i] = 0u;
  for (uint32_t b = 0; b < 32u && ((nsteps - 1u) >> b) != 0u; ++b) {
    int slot[IPT];
    uint32_t valid = 0, one = 0;
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int q = tid * IPT + i;
      slot[i] = 0;
      if (q >= n_un && q < B) {
        slot[i] = s_order[q];
        valid |= 1u << i;
        if ((((last_use[slot[i]] - thr) >> 1) >> b) & 1u) one |= 1u << i;
      }
    }
    int n_zero;
    int z = block_scan_excl(__popc(valid & ~one), s_warp, n_zero);  // zeros before this thread's entries
#pragma unroll
    for (int i = 0; i < IPT; ++i)
      if ((valid >> i) & 1u) {
        const int idx = tid * IPT + i - n_un;  // place in the touched segment = zeros + ones before it
        if ((one >> i) & 1u) {
          s_order[n_un + n_zero + (idx - z)] = (uint16_t)slot[i];
        } else {
          s_order[n_un + z] = (uint16_t)slot[i];
          ++z;
        }
      }
    __syncthreads();
  }
  __syncthreads();
}

// Everything the first block of a cluster does before the fetch can start: Phases 1-2 of Sec. 3.4 and the list of
// misses.  KPT = row entries per thread (k <= KPT * T).  On return s_plan_pos[i] holds the position of the i-th miss,
// s_out[j] the slot of every row entry that hit (or -1, a duplicate marker, or the rank of its miss), s_hitbits the
// hit marks and s_order the staged recency list; `fast` = nothing missed (and the list may be left behind).
template <int T, int IPT, int KPT>
__device__ __forceinline__ void resolve_metadata(const DevState &d, const int r, const int64_t rg, const int32_t *row,
                                                 int32_t *s_sel, int32_t *s_out, int32_t *s_plan_pos,
                                                 int32_t *s_plan_slot, unsigned long long *s_tab, uint32_t *s_hitbits,
                                                 uint32_t *s_vicbits, uint16_t *s_order, int *s_warp, int *s_misc,
                                                 const int64_t cap_r, const int64_t init_len_r,
                                                 const int64_t p2s_off_r, unsigned long long *stamps,
                                                 unsigned char *s_ring, unsigned long long *s_bars,
                                                 const uint32_t t_now, int *s_warp_pre, int16_t *s_got, const int S,
                                                 int &m, uint32_t &my_status, bool &fast) {
  const int tid = threadIdx.x;
  const int k = d.k, B = d.B, H = d.H;
  const uint32_t mask = (uint32_t)(H - 1);
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  bool timed_out = false;

  // Phase 1: stage the row and the recency order (one round trip to HBM).  The request's slice of the page
  // table is streamed into the (still idle) fetch ring with bulk copies when it fits, so that Phase 2's k random
  // lookups hit shared memory instead of queueing as 32-byte sector reads on one SM.
  const int16_t *p2s = d.pos2slot + p2s_off_r + (int64_t)(rg - (int64_t)r * d.G) * cap_r;
  const uintptr_t p2s_aligned = (uintptr_t)p2s & ~(uintptr_t)15;
  const int lead = (int)(((uintptr_t)p2s - p2s_aligned) >> 1);
  const int64_t stage_bytes = ((int64_t)lead * 2 + cap_r * 2) & ~(int64_t)15;  // whole 16-byte units only
  const bool staged = stage_bytes + 16 <= (int64_t)d.ring_bytes;
  const bool coop = !staged && S > 1;  // same decision in every block of the cluster (depends on the request only)
  if (coop) cluster_arrive_relaxed();  // phase A, see cluster_lookups
  const uint32_t stage_bar = smem_u32(s_bars + kThreads);
  const uint16_t *order_g = d.order + rg * B;
  // 16-byte aligned arrays are fetched by ONE thread with bulk copies (a handful of instructions for the whole
  // block); anything else falls back to per-thread cp.async
  const bool sel_bulk = (((uintptr_t)row | (uintptr_t)(k * 4)) & 15) == 0;
  const bool ord_bulk = (((uintptr_t)order_g | (uintptr_t)(B * 2)) & 15) == 0;
  // one expect_tx for everything; each copy is issued by the first lane of a different warp, so that the copies
  // enter the bulk-copy engine side by side (a copy that lands before the expect_tx only makes the count dip)
  if (tid == 0) {
    const uint32_t tx = (sel_bulk ? (uint32_t)k * 4u : 0u) + (ord_bulk ? (uint32_t)B * 2u : 0u) +
                        (staged ? (uint32_t)stage_bytes : 0u);
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(stage_bar), "r"(tx) : "memory");
    if (sel_bulk)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(s_sel)), "l"(row), "r"((uint32_t)k * 4u), "r"(stage_bar) : "memory");
  }
  if (tid == 32 && ord_bulk)
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(s_order)), "l"(order_g), "r"((uint32_t)B * 2u), "r"(stage_bar) : "memory");
  if (staged && tid >= 64 && (tid & 31) == 0) {
    constexpr int kPiece = 16384;
    for (int64_t o = (int64_t)((tid >> 5) - 2) * kPiece; o < stage_bytes; o += (int64_t)(T / 32 - 2) * kPiece) {
      const uint32_t n = (uint32_t)(stage_bytes - o < kPiece ? stage_bytes - o : kPiece);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(s_ring) + (uint32_t)o), "l"((const char *)p2s_aligned + o), "r"(n), "r"(stage_bar) : "memory");
    }
  }
  if (!sel_bulk) stage_async(s_sel, row, k * 4);
  if (!ord_bulk) stage_async(s_order, order_g, B * 2);
  if (staged && tid >= 32 && tid < 40) {  // the last, partial 16-byte unit of the slice: plain copies
    const int64_t e = stage_bytes / 2 + (tid - 32);
    if (e < lead + cap_r) reinterpret_cast<int16_t *>(s_ring)[e] = reinterpret_cast<const int16_t *>(p2s_aligned)[e];
  }
  const int64_t na = *(volatile int32_t *)d.n_appends;
  const int64_t len = init_len_r + na < cap_r ? init_len_r + na : cap_r;
  const int64_t newest = (na > 0 && init_len_r + na <= cap_r) ? init_len_r + na - 1 : -1;
  if (timers && tid == 0) stamps[8] = clock64();
  if (!sel_bulk || !ord_bulk) asm volatile("cp.async.wait_all;" ::: "memory");
  bool use_staged = staged;
  if (!mbar_wait_bounded(stage_bar, 0u)) {
    // bounded wait expired: the row cannot be trusted either, so this request resolves nothing in this launch
    use_staged = false;
    my_status |= HISPARSE_STATUS_TIMEOUT;
    timed_out = true;
  }
  __syncthreads();
  if (timers && tid == 0) stamps[9] = clock64();
  const int16_t *s_p2s = reinterpret_cast<const int16_t *>(s_ring) + lead;
  if (coop) cluster_lookups<T>(row, p2s, k, len, 0, S, s_got);

  // Phase 2: hit detection through the page table (position -> slot): all of a thread's lookups are issued
  // before the first is used.  Hits keep their slot and are stamped first; the selections that are not
  // resident go into the hash table (position -> row index), whose only job is to catch a position that is
  // selected twice, so that it claims one victim, not two.
  int32_t pos[KPT], got[KPT];
#pragma unroll
  for (int i = 0; i < KPT; ++i) {
    const int j = tid + i * T;
    pos[i] = (j < k && !timed_out) ? s_sel[j] : -1;
    const bool ok = pos[i] >= 0 && (int64_t)pos[i] < len;
    if (pos[i] != -1 && !ok) my_status |= HISPARSE_STATUS_OUT_OF_RANGE;
    if (!ok) pos[i] = -1;
    got[i] = !ok ? -1 : (int32_t)(use_staged ? s_p2s[pos[i]] : coop ? s_got[j] : __ldg(p2s + pos[i]));
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the ring goes back to the bulk-copy engine later
  int any_miss = 0;
#pragma unroll
  for (int i = 0; i < KPT; ++i) {
    const int j = tid + i * T;
    if (j >= k) break;
    const int32_t p = pos[i];
    int32_t o = -1;
    if (p >= 0) {
      if ((int64_t)p == newest) {  // reserved newest-record slot, outside the LRU set
        o = B;
        if (atomicExch(&s_misc[2], 1) != 0) my_status |= HISPARSE_STATUS_DUPLICATE;
      } else if (got[i] >= 0) {
        const int s = got[i];
        o = s;
        const uint32_t bit = 1u << (s & 31);
        // a bit that is already set = the same resident position selected again: same slot, counted once.
        // The hit's stamp is written later, in slot order (coalesced), from the hit bits.
        if (atomicOr(&s_hitbits[s >> 5], bit) & bit) my_status |= HISPARSE_STATUS_DUPLICATE;
      } else {
        o = kMiss;
        any_miss = 1;
        const unsigned long long entry = ((unsigned long long)(uint32_t)p << 32) | (uint32_t)j;
        uint32_t h = hash_pos(p, d.hshift);
        for (uint32_t it = 0; it <= mask; ++it) {
          const unsigned long long old = atomicCAS(&s_tab[h], kEmptyEntry, entry);
          if (old == kEmptyEntry) break;
          if ((int32_t)(old >> 32) == p) {  // selected twice: the lowest row index owns the entry
            atomicMin(&s_tab[h], entry);
            s_misc[0] = 1;
            break;
          }
          h = (h + 1u) & mask;
        }
      }
    }
    s_out[j] = o;
  }
  any_miss = __syncthreads_or(any_miss);
  if (!any_miss && d.order_t != nullptr) {
    // Nothing to fetch, no victim to choose: the caller writes the table and stamps the hits, and the recency list
    // is left as it is (rebuild_order brings it up to date in the next resolve that needs victims).
    fast = true;
    m = 0;
    return;
  }
  if (timers && tid == 0) stamps[10] = clock64();
  if (s_misc[0]) {  // rare: every later occurrence of a repeated missing position follows the first one
    for (int j = tid; j < k; j += T) {
      if (s_out[j] == kMiss) {
        const int32_t key[1] = {s_sel[j]};
        int32_t owner[1];
        table_lookup<1>(s_tab, mask, d.hshift, key, owner);
        if (owner[0] != j) {
          s_out[j] = kDupBase - owner[0];
          my_status |= HISPARSE_STATUS_DUPLICATE;
        }
      }
    }
    __syncthreads();
  }
  if (timers && tid == 0) stamps[11] = clock64();

  // Phase 3, first half: the misses in selection order (one block scan; thread t owns KPT consecutive row entries).
  // Their positions are all the fetch needs to start loading; the victims are only needed when a record is stored.
  {
    uint32_t miss_mask = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i) {
      const int j = tid * KPT + i;
      if (j < k && s_out[j] == kMiss) miss_mask |= 1u << i;
    }
    int mrank = block_scan_excl(__popc(miss_mask), s_warp, m);
#pragma unroll
    for (int i = 0; i < KPT; ++i)
      if ((miss_mask >> i) & 1u) {
        const int j = tid * KPT + i;
        s_plan_pos[mrank] = s_sel[j];      // position of the mrank-th miss
        s_out[j] = kRankBase - mrank;      // its slot is the mrank-th victim, looked up when the table is written
        ++mrank;
      }
  }
  if (timers && tid == 0) stamps[12] = clock64();
  __syncthreads();
}

// Phase 3, second half (runs while the first loads are in flight): brings the recency list up to date if it lags,
// then ONE block scan over the non-hit slots in recency order.  Thread t owns IPT consecutive entries of the list.
// On return s_plan_slot[i] holds the victim of the i-th miss, s_vicbits the victims' marks, s_order the untouched
// slots compacted at its front and n_nonhit the number of slots without a hit.
template <int T, int IPT>
__device__ __forceinline__ void choose_victims(const DevState &d, const int r, const int64_t rg, const int m,
                                               int32_t *s_plan_slot, unsigned long long *s_tab, const uint32_t *s_hitbits,
                                               uint32_t *s_vicbits, uint16_t *s_order, int *s_warp, int *s_warp_pre,
                                               unsigned long long *stamps, const uint32_t t_now, const uint32_t order_t,
                                               int &n_nonhit) {
  const int tid = threadIdx.x;
  const int B = d.B;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  if (order_t != t_now - 1u) {
    const uint32_t *last_use = d.last_use + rg * B;
    rebuild_order<T, IPT>(B, d.W, last_use, 2u * order_t + 2u, t_now - 1u - order_t, s_order, s_vicbits, s_warp_pre, s_warp);
  }
  {
    int slot[IPT];
    uint32_t nh_mask = 0;
#pragma unroll
    for (int i = 0; i < IPT; ++i) {
      const int q = tid * IPT + i;
      slot[i] = 0;
      if (q < B) {
        slot[i] = s_order[q];
        if (!((s_hitbits[slot[i] >> 5] >> (slot[i] & 31)) & 1u)) nh_mask |= 1u << i;
      }
    }
    int nrank = block_scan_excl(__popc(nh_mask), s_warp, n_nonhit);
    if (d.policy == HISPARSE_POLICY_LRU) {
      // the i-th miss (selection order) takes the i-th non-hit slot of the recency order
#pragma unroll
      for (int i = 0; i < IPT; ++i)
        if ((nh_mask >> i) & 1u) {
          const int s = slot[i];
          if (nrank < m) {
            s_plan_slot[nrank] = s;
            atomicOr(&s_vicbits[s >> 5], 1u << (s & 31));
          } else {
            s_order[nrank - m] = (uint16_t)s;  // in place: every thread read its entries before the scan's barriers
          }
          ++nrank;
        }
    } else if (d.policy == HISPARSE_POLICY_FIFO) {
      // same victims, but a hit does not move: everything that is not a victim keeps its place in the list
#pragma unroll
      for (int i = 0; i < IPT; ++i) {
        const int q = tid * IPT + i;
        if (q >= B) break;
        const int s = slot[i];
        const bool nonhit = (nh_mask >> i) & 1u;
        if (nonhit && nrank < m) {
          s_plan_slot[nrank] = s;
          atomicOr(&s_vicbits[s >> 5], 1u << (s & 31));
        } else {
          s_order[q - (nrank < m ? nrank : m)] = (uint16_t)s;
        }
        if (nonhit) ++nrank;
      }
    } else {
      // RANDOM: victims by hashed key, paired with the misses in ascending slot order; the list is kept as for LRU
      __syncthreads();
      const unsigned long long base = mix64(d.policy_seed ^ (((unsigned long long)(uint32_t)r << 32) | (uint32_t)(rg - (int64_t)r * d.G)));
      select_random_victims<IPT>(B, m, base, t_now, s_hitbits, s_vicbits, reinterpret_cast<int *>(s_tab), s_warp);
      uint32_t keep = 0;
#pragma unroll
      for (int i = 0; i < IPT; ++i)
        if (((nh_mask >> i) & 1u) && !((s_vicbits[slot[i] >> 5] >> (slot[i] & 31)) & 1u)) keep |= 1u << i;
      int tot2;
      int krank = block_scan_excl(__popc(keep), s_warp, tot2);
#pragma unroll
      for (int i = 0; i < IPT; ++i)
        if ((keep >> i) & 1u) s_order[krank++] = (uint16_t)slot[i];
      // i-th victim in slot order: running count of victim bits below each word, by warp 0
      if (tid < 32) {
        int run = 0;
        for (int wb = 0; wb < d.W; wb += 32) {
          const int w = wb + tid;
          const int c = w < d.W ? __popc(s_vicbits[w]) : 0;
          int inc = c;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, inc, o);
            if (tid >= o) inc += n;
          }
          if (w < d.W) s_warp_pre[w] = run + inc - c;
          run += __shfl_sync(0xffffffffu, inc, 31);
        }
      }
      __syncthreads();
      for (int s = tid; s < B; s += T) {
        const uint32_t vw = s_vicbits[s >> 5], bit = 1u << (s & 31);
        const int i = s_warp_pre[s >> 5] + __popc(vw & (bit - 1u));
        if ((vw & bit) && i < m) s_plan_slot[i] = s;
      }
    }
  }
  if (timers && tid == 0) stamps[13] = clock64();
  __syncthreads();
  if (timers && tid == 0) stamps[14] = clock64();
}

template <int T>
__global__ void __launch_bounds__(T, kThreads / T)
resolve_kernel(const DevState d, const int layer, const int32_t *__restrict__ sel, int32_t *__restrict__ table,
               int32_t *__restrict__ hits_out, int32_t *__restrict__ misses_out, const int S) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ int s_warp[32];
  __shared__ int s_misc[4];  // [0] a missing position was selected twice  [2] the newest position was selected
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x / S, part = blockIdx.x - r * S;
  const int g = layer / d.lpg;
  const int k = d.k, B = d.B, H = d.H, W = d.W;
  const int64_t rg = (int64_t)r * d.G + g;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  unsigned long long *stamps = d.phase_ns + (int64_t)r * 16;

  unsigned long long *s_tab = reinterpret_cast<unsigned long long *>(smem_raw);
  int32_t *s_sel = reinterpret_cast<int32_t *>(s_tab + H);
  int32_t *s_out = s_sel + k;
  int32_t *s_plan_pos = s_out + k;        // first the row indices of the misses, then their positions
  int32_t *s_plan_slot = s_plan_pos + k;  // victims, in order
  uint32_t *s_hitbits = reinterpret_cast<uint32_t *>(s_plan_slot + k);
  uint32_t *s_vicbits = s_hitbits + W;
  int32_t *s_hitpre = reinterpret_cast<int32_t *>(s_vicbits + W);
  int32_t *s_vicpre = s_hitpre + W;
  uint16_t *s_order = reinterpret_cast<uint16_t *>(s_vicpre + W);
  int16_t *s_got = reinterpret_cast<int16_t *>(s_order + ((B + 7) & ~7));  // page-table answers from the whole cluster
  unsigned long long *s_bars = reinterpret_cast<unsigned long long *>(smem_raw + d.meta_smem);
  unsigned char *s_ring = smem_raw + d.meta_smem + kBarBytes;

  // Prologue that depends on nothing an earlier kernel wrote: barriers, cleared marks and table.  With
  // programmatic dependent launch it overlaps the tail of whatever runs before this kernel in the stream.
  fetch_barriers_init(s_bars, d.io_threads);
  if (part == 0) {
    for (int i = tid; i < H; i += T) s_tab[i] = kEmptyEntry;
    for (int i = tid; i < W; i += T) { s_hitbits[i] = 0u; s_vicbits[i] = 0u; }
    if (tid < 4) s_misc[tid] = 0;
  }
  const bool uni = d.uni_cap >= 0;  // fixed at create
  const int64_t cap_r = uni ? d.uni_cap : d.cap[r], init_len_r = uni ? d.uni_init_len : d.init_len[r],
                p2s_off_r = uni ? (int64_t)r * d.G * d.uni_cap : d.p2s_off[r];
  if (part == 0 && tid < 3) {
    // Warm L2 with what Phase 1 will stage (row, recency order, page-table slice).  A prefetch consumes nothing, and
    // L2 is where earlier kernels' writes land, so this is safe before the dependency wait; when the previous kernel
    // lets its dependents start early, the staging after the wait then reads L2 instead of HBM.
    const char *p = tid == 0 ? reinterpret_cast<const char *>(sel + (int64_t)r * k)
                  : tid == 1 ? reinterpret_cast<const char *>(d.order + rg * B)
                             : reinterpret_cast<const char *>(d.pos2slot + p2s_off_r + (int64_t)g * cap_r);
    int64_t n = tid == 0 ? (int64_t)k * 4 : tid == 1 ? (int64_t)B * 2 : cap_r * 2;
    const uintptr_t a = ((uintptr_t)p + 15) & ~(uintptr_t)15;   // whole 16-byte units inside the array only
    n = (n - (int64_t)(a - (uintptr_t)p)) & ~(int64_t)15;
    if (n > (1 << 20)) n = 1 << 20;                             // no point warming more than the ring could stage
    if (n > 0)
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a), "r"((uint32_t)n) : "memory");
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (part != 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  TmaFetch fetch;
  fetch.active = false;
  int m = 0, n_nonhit = 0;
  uint32_t t = 0;
  bool fast = false;  // first block only: no selection missed, the short path below was taken
  if (part != 0) {
    // same test as in resolve_metadata: is this request's page-table slice too large to be staged?
    const int16_t *p2s = d.pos2slot + p2s_off_r + (int64_t)g * cap_r;
    const int lead = (int)((((uintptr_t)p2s) & 15) >> 1);
    const int64_t stage_bytes = ((int64_t)lead * 2 + cap_r * 2) & ~(int64_t)15;
    if (!(stage_bytes + 16 <= (int64_t)d.ring_bytes)) {
      const int64_t na = *(volatile int32_t *)d.n_appends;
      const int64_t len = init_len_r + na < cap_r ? init_len_r + na : cap_r;
      cluster_arrive_relaxed();  // phase A
      cluster_lookups<T>(sel + (int64_t)r * k, p2s, k, len, part, S, s_got);
    }
  }
  if (part == 0) {
    if (timers && tid == 0) { stamps[0] = global_ns(); stamps[6] = 0ull; stamps[15] = clock64(); }
    t = d.t[rg] + 1u;
    const uint32_t order_t = d.order_t ? d.order_t[rg] : t - 1u;  // resolve count the recency list is current for
    const uint32_t miss_stamp = 2u * t;
    uint32_t my_status = 0;
    const int32_t *row = sel + (int64_t)r * k;
#define HS_META(IPT, KPT)                                                                                         \
  resolve_metadata<T, IPT, KPT>(d, r, rg, row, s_sel, s_out, s_plan_pos, s_plan_slot, s_tab, s_hitbits, s_vicbits,     \
                             s_order, s_warp, s_misc, cap_r, init_len_r, p2s_off_r, stamps, s_ring, s_bars, t,      \
                             s_vicpre, s_got, S, m, my_status, fast)
    if constexpr (T == kThreads) {
      if (k <= 2 * T) {
        if (B <= 4 * T) HS_META(4, 2);
        else if (B <= 8 * T) HS_META(8, 2);
        else HS_META(16, 2);
      } else {
        if (B <= 4 * T) HS_META(4, kSelPerThread);
        else if (B <= 8 * T) HS_META(8, kSelPerThread);
        else HS_META(16, kSelPerThread);
      }
    } else {  // the small block is only chosen for B <= 16 T and k <= 4 T
      if (B <= 8 * T) HS_META(8, 4);
      else HS_META(16, 4);
    }
#undef HS_META
    if (timers && tid == 0) { stamps[3] = global_ns(); stamps[7] = stamps[3]; }
    if (fast) {
      // nothing to fetch: let whatever follows in the stream start its prologue now (measured: with a fetch ahead,
      // releasing the dependents before the first loads are issued costs the fetch about 2 us, so that path
      // releases them only once its metadata is written back)
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      // Every valid selection is resident (or the newest record): the slot table, the hit stamps in slot order
      // (coalesced) and the counters are all there is to write.  The recency list is not touched and
      // order_t stays behind; under FIFO a hit changes nothing, so the list stays current.
      int32_t *trow = table + (int64_t)r * k;
      int32_t *arow = d.anchor_out + rg * k;
      for (int j = tid; j < k; j += T) {
        const int32_t o = s_out[j];
        trow[j] = o < 0 ? -1 : r * (B + 1) + o;
        if (d.lpg > 1) arow[j] = o < 0 ? -1 : o;
      }
      int c = 0;
      for (int w = tid; w < W; w += T) c += __popc(s_hitbits[w]);
      if (warp * 32 < W) {
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0 && c) atomicAdd(&s_misc[3], c);
      }
      if (d.policy != HISPARSE_POLICY_FIFO) {
        uint32_t *last_use = d.last_use + rg * B;
        for (int s = tid; s < B; s += T)
          if ((s_hitbits[s >> 5] >> (s & 31)) & 1u) last_use[s] = 2u * t + 1u;
      }
      __syncthreads();
      if (tid == 0) {
        const int nhits = s_misc[3] + (s_misc[2] ? 1 : 0);
        hits_out[r] = nhits;
        misses_out[r] = 0;
        d.anchor_hits[rg] = nhits;
        d.anchor_misses[rg] = 0;
        d.plan_n[rg] = 0;
        d.t[rg] = t;
        if (d.policy == HISPARSE_POLICY_FIFO) d.order_t[rg] = t;
        if (timers) stamps[4] = global_ns();
      }
    } else {
      // Phase 4 starts here, with the positions of the misses: the first batch of host loads is in flight while the
      // victims are chosen (a record's slot is only needed when it is stored) and the metadata is written back
      fetch.init(d, r, layer, m, s_plan_pos, s_plan_slot, s_ring, s_bars, 0, S);
      fetch.issue(d);
#define HS_VICT(IPT)                                                                                              \
  choose_victims<T, IPT>(d, r, rg, m, s_plan_slot, s_tab, s_hitbits, s_vicbits, s_order, s_warp, s_vicpre, stamps, t, \
                         order_t, n_nonhit)
      if constexpr (T == kThreads) {
        if (B <= 4 * T) HS_VICT(4);
        else if (B <= 8 * T) HS_VICT(8);
        else HS_VICT(16);
      } else {
        if (B <= 8 * T) HS_VICT(8);
        else HS_VICT(16);
      }
#undef HS_VICT
      // same state as right after the first issue, recomputed instead of kept in registers across the victim choice
      fetch.init(d, r, layer, m, s_plan_pos, s_plan_slot, s_ring, s_bars, 0, S);
      fetch.active = fetch.active && fetch.piece_of(d, 0) < fetch.total;
      // Phase 5, metadata half: page table, slot array, stamps, plan
      int32_t *slot_pos = d.slot_pos + rg * B;
      uint32_t *last_use = d.last_use + rg * B;
      int16_t *p2s = d.pos2slot + p2s_off_r + (int64_t)g * cap_r;
      int32_t *plan_pos_g = d.plan_pos + rg * k, *plan_slot_g = d.plan_slot + rg * k;
      for (int i = tid; i < m; i += T) {
        const int v = s_plan_slot[i];
        const int32_t p = s_plan_pos[i];
        const int32_t old = slot_pos[v];
        if (old >= 0) p2s[old] = -1;
        slot_pos[v] = p;
        p2s[p] = (int16_t)v;
        last_use[v] = miss_stamp;
        plan_pos_g[i] = p;
        plan_slot_g[i] = v;
      }
      if (tid == 0) d.plan_n[rg] = m;
    }
    if (my_status) atomicOr(d.status, my_status);
  }
  // The plan is public: the other blocks of the cluster start fetching while this one publishes.  Every thread
  // arrives with release semantics after its own plan writes and every reader waits with acquire semantics, which
  // orders them at cluster scope: no separate fence.
  if (S > 1) asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");

  if (part == 0 && !fast) {
    uint16_t *order = d.order + rg * B;
    // new order = untouched ++ victims by slot ++ hits by slot: word-level prefix counts, then one pass.
    if (warp == 0) {
      int run_h = 0, run_v = 0;
      for (int wb = 0; wb < W; wb += 32) {
        const int w = wb + lane;
        const int ch = w < W ? __popc(s_hitbits[w]) : 0, cv = w < W ? __popc(s_vicbits[w]) : 0;
        int ih = ch, iv = cv;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int nh = __shfl_up_sync(0xffffffffu, ih, o), nv = __shfl_up_sync(0xffffffffu, iv, o);
          if (lane >= o) { ih += nh; iv += nv; }
        }
        if (w < W) { s_hitpre[w] = run_h + ih - ch; s_vicpre[w] = run_v + iv - cv; }
        run_h += __shfl_sync(0xffffffffu, ih, 31);
        run_v += __shfl_sync(0xffffffffu, iv, 31);
      }
    }
    // Phase 5: the slot table in selection order (does not depend on the order rewrite)
    int32_t *trow = table + (int64_t)r * k;
    int32_t *arow = d.anchor_out + rg * k;
    for (int j = tid; j < k; j += T) {
      int32_t o = s_out[j];
      if (o <= kDupBase && o > kRankBase) o = s_out[kDupBase - o];  // a repeated position follows its first occurrence
      if (o <= kRankBase) o = s_plan_slot[kRankBase - o];           // a miss takes its victim's slot
      trow[j] = o < 0 ? -1 : r * (B + 1) + o;
      if (d.lpg > 1) arow[j] = o < 0 ? -1 : o;
    }
    __syncthreads();
    uint32_t *last_use = d.last_use + rg * B;
    if (d.policy == HISPARSE_POLICY_FIFO) {
      // insertion order: the refilled slots go to the end, by slot; hits were left where they were, unstamped
      for (int s = tid; s < B; s += T) {
        const int w = s >> 5;
        const uint32_t bit = 1u << (s & 31), vw = s_vicbits[w];
        if (vw & bit) s_order[(B - m) + s_vicpre[w] + __popc(vw & (bit - 1u))] = (uint16_t)s;
      }
    } else {
      const int n_surv = n_nonhit - m;
      for (int s = tid; s < B; s += T) {
        const int w = s >> 5;
        const uint32_t bit = 1u << (s & 31), lt = bit - 1u;
        const uint32_t vw = s_vicbits[w], hw = s_hitbits[w];
        if (vw & bit) {
          s_order[n_surv + s_vicpre[w] + __popc(vw & lt)] = (uint16_t)s;
        } else if (hw & bit) {
          s_order[n_nonhit + s_hitpre[w] + __popc(hw & lt)] = (uint16_t)s;
          last_use[s] = 2u * t + 1u;  // hits are stamped above this step's fetched records
        }
      }
    }
    __syncthreads();
    for (int q = tid; q < B; q += T) order[q] = s_order[q];
    if (tid == 0) {
      // distinct hits = slots whose hit bit is set (+ the reserved slot if the newest position was selected)
      const int nhits = (B - n_nonhit) + (s_misc[2] ? 1 : 0);
      hits_out[r] = nhits;
      misses_out[r] = m;
      d.anchor_hits[rg] = nhits;
      d.anchor_misses[rg] = m;
      d.t[rg] = t;
      if (d.order_t) d.order_t[rg] = t;
    }
    if (timers && tid == 0) stamps[4] = global_ns();
  }

  if (S > 1) {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (part != 0) {
      m = __ldcg(d.plan_n + rg);
      const int32_t *pp = d.plan_pos + rg * k, *ps = d.plan_slot + rg * k;
      for (int i = tid; i < m; i += T) { s_plan_pos[i] = __ldcg(pp + i); s_plan_slot[i] = __ldcg(ps + i); }
      __syncthreads();
      fetch.init(d, r, layer, m, s_plan_pos, s_plan_slot, s_ring, s_bars, part, S);
      fetch.issue(d);
    }
  }
  // Phase 4, rest: wait for the batches, store them into the cache slots, issue what is left.  Whatever follows
  // in the stream may be scheduled from here on (it still waits for this grid to finish before it reads).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  fetch.drain(d, d.status);
  if (timers) {
    __syncthreads();
    if (tid == 0) {
      const unsigned long long now = global_ns();
      if (part == 0) stamps[5] = now;
      atomicMax(&stamps[6], now);
    }
  }
}

// ------------------------------------------------------------------------------------------ plan replay (Sec. 3.5)

// Copy-only kernel: replays the anchor's miss plan into a shared layer's cache.  grid = N * S blocks.
__global__ void __launch_bounds__(kThreads, 1) replay_kernel(const DevState d, const int layer, const int S) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int32_t *s_plan_pos = reinterpret_cast<int32_t *>(smem_raw);
  int32_t *s_plan_slot = s_plan_pos + d.k;
  unsigned long long *s_bars = reinterpret_cast<unsigned long long *>(smem_raw + d.meta_smem);
  unsigned char *s_ring = smem_raw + d.meta_smem + kBarBytes;
  const int r = blockIdx.x / S, part = blockIdx.x - r * S;
  const int64_t rg = (int64_t)r * d.G + layer / d.lpg;
  const int m = d.plan_n[rg];
  const int32_t *pp = d.plan_pos + rg * d.k, *ps = d.plan_slot + rg * d.k;
  fetch_barriers_init(s_bars, d.io_threads);
  for (int i = threadIdx.x; i < m; i += blockDim.x) { s_plan_pos[i] = pp[i]; s_plan_slot[i] = ps[i]; }
  __syncthreads();
  TmaFetch fetch;
  fetch.init(d, r, layer, m, s_plan_pos, s_plan_slot, s_ring, s_bars, part, S);
  fetch.issue(d);
  fetch.drain(d, d.status);
}

// A shared layer reuses its anchor's slot table (same local slots, same request offsets) and counts.
__global__ void shared_table_kernel(const DevState d, const int layer, int32_t *__restrict__ table,
                                    int32_t *__restrict__ hits_out, int32_t *__restrict__ misses_out) {
  const int r = blockIdx.x;
  const int64_t rg = (int64_t)r * d.G + layer / d.lpg;
  for (int j = threadIdx.x; j < d.k; j += blockDim.x) {
    const int32_t o = d.anchor_out[rg * d.k + j];
    table[(int64_t)r * d.k + j] = o < 0 ? -1 : r * (d.B + 1) + o;
  }
  if (threadIdx.x == 0) { hits_out[r] = d.anchor_hits[rg]; misses_out[r] = d.anchor_misses[rg]; }
}

// ------------------------------------------------------------------------------------------ append (Sec. 3.3 step 4)

__device__ __forceinline__ void copy16(uint8_t *dst, const uint8_t *src, uint32_t units) {
  for (uint32_t u = threadIdx.x; u < units; u += blockDim.x)
    reinterpret_cast<uint4 *>(dst)[u] = reinterpret_cast<const uint4 *>(src)[u];
}

// grid = N * L blocks.  Block (r, l) puts request r's new record of layer l into the reserved slot; with
// write_through != 0 it also stores it into the host history.  The last block to finish bumps the append count.
__global__ void append_kernel(const DevState d, const uint8_t *__restrict__ new_kv, const int write_through) {
  const int r = blockIdx.x / d.L, l = blockIdx.x - r * d.L;
  const int64_t na = *(volatile int32_t *)d.n_appends;
  const int64_t p = d.init_len[r] + na;
  if (p < d.cap[r]) {
    const uint8_t *src = new_kv + ((int64_t)r * d.L + l) * d.E;
    copy16(d.pool + (int64_t)l * d.layer_pool_bytes + ((int64_t)r * (d.B + 1) + d.B) * d.E, src, d.upe);
    if (write_through) {
      copy16(d.host[r] + ((int64_t)l * d.cap[r] + p) * d.E, src, d.upe);
      __threadfence_system();
    }
  } else if (threadIdx.x == 0 && l == 0) {
    atomicOr(d.status, HISPARSE_STATUS_CAPACITY);
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint32_t prev = atomicAdd(d.ticket, 1u);
    if (prev == gridDim.x - 1) {
      *(volatile int32_t *)d.n_appends = (int32_t)na + 1;
      *(volatile uint32_t *)d.ticket = 0u;
      __threadfence();
    }
  }
}

// Backup-stream half of the append: reserved slot -> host history at the position just appended.
__global__ void write_through_kernel(const DevState d) {
  const int r = blockIdx.x / d.L, l = blockIdx.x - r * d.L;
  const int64_t na = *(volatile int32_t *)d.n_appends;
  const int64_t p = d.init_len[r] + na - 1;
  if (na > 0 && p < d.cap[r]) {
    copy16(d.host[r] + ((int64_t)l * d.cap[r] + p) * d.E,
           d.pool + (int64_t)l * d.layer_pool_bytes + ((int64_t)r * (d.B + 1) + d.B) * d.E, d.upe);
    __threadfence_system();
  }
}

// ------------------------------------------------------------------------------------------ consumer stand-ins

// One warp per table entry: out[r][j] = pool[table[r][j]] (zeros for -1).
constexpr int kGatherThreads = 128;

// Stand-in for the consumer's gather (Sec. 3.4 Phase 5): out[e] = pool[table[e]].  Copy-only, so it is written like
// the fetch: every thread moves pieces of at most `chunk` bytes cache slot -> shared memory -> out with bulk copies
// (one ring slot and one mbarrier per thread; the first `active` threads of a block take part, so that two blocks
// fit an SM).  Entries with table value -1 are filled from a page of zeros.  Dynamic shared memory:
// [kGatherThreads mbarriers][chunk bytes of zeros][active * chunk bytes of ring].
__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(const DevState d, const int layer, const int32_t *__restrict__ table, uint8_t *__restrict__ out,
              const int chunk, const int active) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  unsigned long long *bars = reinterpret_cast<unsigned long long *>(smem_raw);
  unsigned char *zeros = smem_raw + kGatherThreads * 8;
  unsigned char *ring = zeros + chunk;
  const int tid = threadIdx.x;
  for (int o = tid * 16; o < chunk; o += kGatherThreads * 16) *reinterpret_cast<uint4 *>(zeros + o) = make_uint4(0, 0, 0, 0);
  if (tid < active) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + tid)) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the zeros are read by bulk stores
  __syncthreads();
  if (tid >= active) return;
  const uint8_t *pool = d.pool + (int64_t)layer * d.layer_pool_bytes;
  const int64_t E = d.E;
  const int ppr = (int)((E + chunk - 1) / chunk);
  const int64_t total = (int64_t)d.N * d.k * ppr, stride = (int64_t)gridDim.x * active;
  const uint32_t slot = smem_u32(ring) + (uint32_t)tid * (uint32_t)chunk, bar = smem_u32(bars + tid);
  uint32_t parity = 0;
  for (int64_t c = (int64_t)blockIdx.x * active + tid; c < total; c += stride) {
    const int64_t e = ppr == 1 ? c : c / ppr;
    const int piece = (int)(c - e * ppr);
    const int64_t rest = E - (int64_t)piece * chunk;
    const uint32_t bytes = (uint32_t)(rest < chunk ? rest : chunk);
    const int32_t s = table[e];
    uint8_t *dst = out + e * E + (int64_t)piece * chunk;
    uint32_t from = smem_u32(zeros);
    if (s >= 0) {
      const uint8_t *src = pool + (int64_t)s * E + (int64_t)piece * chunk;
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(slot), "l"(src), "r"(bytes), "r"(bar) : "memory");
      if (!mbar_wait_bounded(bar, parity)) {
        atomicOr(d.status, HISPARSE_STATUS_TIMEOUT);
        return;
      }
      parity ^= 1u;
      from = slot;
    }
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(from), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");  // the ring slot may be overwritten
  }
}

// One warp per selection: the bytes the table entry addresses must equal the host history's record.
__global__ void gather_check_kernel(const DevState d, const int layer, const int32_t *__restrict__ sel,
                                    const int32_t *__restrict__ table, int32_t *mismatches) {
  const int lane = threadIdx.x & 31;
  const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
  const uint8_t *pool = d.pool + (int64_t)layer * d.layer_pool_bytes;
  for (int64_t e = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); e < (int64_t)d.N * d.k; e += nwarps) {
    const int r = (int)(e / d.k);
    int64_t len, newest;
    history_state(d, r, len, newest);
    const int32_t p = sel[e];
    if (p < 0 || p >= len) continue;
    const int32_t s = table[e];
    bool bad = s < r * (d.B + 1) || s > r * (d.B + 1) + d.B;
    if (!bad) {
      const uint4 *a = reinterpret_cast<const uint4 *>(pool + (int64_t)s * d.E);
      const uint8_t *hb = d.host[r] + ((int64_t)layer * d.cap[r] + p) * d.E;
      for (uint32_t u = lane; u < d.upe; u += 32) {
        const uint4 x = a[u], y = ld_host16(hb + (int64_t)u * 16);
        bad |= x.x != y.x || x.y != y.y || x.z != y.z || x.w != y.w;
      }
    }
    bad = __any_sync(0xffffffffu, bad);
    if (bad && lane == 0) atomicAdd(mismatches, 1);
  }
}

// DEBUG_VALIDATE: one block per (request, group).
__global__ void validate_kernel(const DevState d, const int g) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t *seen = reinterpret_cast<uint32_t *>(smem_raw);
  const int r = blockIdx.x, B = d.B;
  const int64_t rg = (int64_t)r * d.G + g;
  const int32_t *slot_pos = d.slot_pos + rg * B;
  const uint32_t *last_use = d.last_use + rg * B;
  const uint16_t *order = d.order + rg * B;
  const int16_t *p2s = d.pos2slot + d.p2s_off[r] + (int64_t)g * d.cap[r];
  for (int i = threadIdx.x; i < d.W; i += blockDim.x) seen[i] = 0u;
  __syncthreads();
  // a list that lags behind the stamps (resolves without misses) is still a permutation, but not sorted by them
  const bool current = !d.order_t || d.order_t[rg] == d.t[rg];
  bool bad = false;
  for (int s = threadIdx.x; s < B; s += blockDim.x) {
    const int32_t p = slot_pos[s];
    if (p >= 0) bad |= p >= d.cap[r] || p2s[p] != s;
    else bad |= p != -1;
  }
  for (int64_t p = threadIdx.x; p < d.cap[r]; p += blockDim.x) {
    const int32_t s = p2s[p];
    if (s >= 0) bad |= s >= B || slot_pos[s] != (int32_t)p;
    else bad |= s != -1;
  }
  for (int q = threadIdx.x; q < B; q += blockDim.x) {
    const int s = order[q];
    if (s >= B) { bad = true; continue; }
    const uint32_t old = atomicOr(&seen[s >> 5], 1u << (s & 31));
    bad |= (old >> (s & 31)) & 1u;
    if (q + 1 < B && current) {
      const int s2 = order[q + 1];
      if (s2 < B) {
        const uint32_t a = last_use[s], b = last_use[s2];
        bad |= a > b || (a == b && s > s2);
      }
    }
  }
  if (bad) atomicOr(d.status, HISPARSE_STATUS_INCONSISTENT);
}

// Exercises the bounded wait on purpose: an mbarrier that nothing ever completes.  The wait gives up after
// limit_ns, sets STATUS_TIMEOUT and the kernel returns normally; *waited_ns receives how long it waited.
__global__ void wait_timeout_selftest_kernel(uint32_t *status, unsigned long long limit_ns,
                                             unsigned long long *waited_ns) {
  __shared__ __align__(8) unsigned long long bar;
  if (threadIdx.x == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = global_ns();
    if (!mbar_wait_bounded(smem_u32(&bar), 0u, limit_ns)) atomicOr(status, HISPARSE_STATUS_TIMEOUT);
    *waited_ns = global_ns() - t0;
  }
}

__global__ void init_order_kernel(uint16_t *order, int64_t n, int B) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    order[i] = (uint16_t)(i % B);
}

// Metadata-free scattered copy used by hisparse_scatter_read_probe.
__global__ void __launch_bounds__(kThreads, 1)
scatter_probe_kernel(const uint8_t *__restrict__ host, uint8_t *__restrict__ dst, const int32_t *__restrict__ rec_idx,
                     int m, uint32_t upe) {
  const uint64_t total = (uint64_t)m * upe, stride = (uint64_t)gridDim.x * blockDim.x;
  for (uint64_t base = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; base < total; base += stride * kFetchUnroll) {
    uint4 v[kFetchUnroll];
    uint8_t *out[kFetchUnroll];
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i) {
      const uint64_t u = base + (uint64_t)i * stride;
      out[i] = nullptr;
      if (u < total) {
        const uint32_t rec = (uint32_t)(u / upe), off = (uint32_t)(u - (uint64_t)rec * upe);
        v[i] = ld_host16(host + ((int64_t)rec_idx[rec] * upe + off) * 16);
        out[i] = dst + u * 16;
      }
    }
#pragma unroll
    for (int i = 0; i < kFetchUnroll; ++i)
      if (out[i]) *reinterpret_cast<uint4 *>(out[i]) = v[i];
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------ host state

struct hisparse {
  DevState d{};
  int device = 0;
  int S = 1, T = kThreads;
  int sm_count = 1;
  size_t resolve_smem = 0, replay_smem = 0;
  std::vector<int64_t> cap, init_len, p2s_off;
  int64_t p2s_total = 0;
  // device allocations (owned)
  std::vector<void *> allocs;
  int64_t *d_cap = nullptr, *d_init_len = nullptr, *d_p2s_off = nullptr;
  uint8_t **d_host = nullptr;
  // streams / events
  cudaStream_t backup = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_wt = nullptr;
  bool wt_pending = false;
  std::vector<cudaEvent_t> ev_plan;   // [G] recorded after each anchor resolve
  std::vector<cudaEvent_t> ev_pref;   // [L] recorded after each prefetch replay
  std::vector<uint8_t> anchor_done;   // [G] the anchor has been resolved at least once
  std::vector<uint8_t> replayed;      // [L] plan replayed (or being replayed) since the anchor's last resolve
  std::vector<uint8_t> pref_unjoined; // [L] a side-stream replay that no stream has waited for yet
  // speculative hints (hisparse_prefetch_hint): discarded outputs, fork / completion events
  int32_t *hint_table = nullptr, *hint_hits = nullptr, *hint_misses = nullptr;
  cudaEvent_t ev_hint_fork = nullptr;
  std::vector<cudaEvent_t> ev_hint;   // [L]
  std::vector<uint8_t> hint_unjoined; // [L]
};

namespace {

template <typename T>
int dev_alloc(hisparse *h, T **out, size_t count) {
  void *p = nullptr;
  HS_CUDA(cudaMalloc(&p, std::max<size_t>(count, 1) * sizeof(T)));
  h->allocs.push_back(p);
  *out = static_cast<T *>(p);
  return HISPARSE_OK;
}

int validate_config(const hisparse_config_t *c) {
  if (!c) return HISPARSE_EINVAL;
  if (c->num_requests < 1 || c->num_layers < 1 || c->layers_per_group < 1) return HISPARSE_EINVAL;
  if (c->num_layers % c->layers_per_group) return HISPARSE_EINVAL;
  if (c->top_k < 1 || c->top_k > HISPARSE_MAX_TOP_K) return HISPARSE_EINVAL;
  if (c->cache_slots < c->top_k || c->cache_slots > HISPARSE_MAX_CACHE_SLOTS) return HISPARSE_EINVAL;
  if (c->entry_bytes < 16 || c->entry_bytes % 16) return HISPARSE_EINVAL;
  if (c->entry_bytes / 16 > 0x7fffffff) return HISPARSE_EINVAL;
  if (!c->capacity || !c->init_len) return HISPARSE_EINVAL;
  for (int r = 0; r < c->num_requests; ++r) {
    if (c->capacity[r] < 1 || c->capacity[r] > 0x7fffffffLL) return HISPARSE_EINVAL;
    if (c->init_len[r] < 0 || c->init_len[r] > c->capacity[r]) return HISPARSE_EINVAL;
  }
  const int s = c->ctas_per_request;
  if (!(s == 0 || s == 1 || s == 2 || s == 4 || s == 8)) return HISPARSE_EINVAL;
  if (c->policy < HISPARSE_POLICY_LRU || c->policy > HISPARSE_POLICY_RANDOM) return HISPARSE_EINVAL;
  return HISPARSE_OK;
}

int hash_size(int k) {
  int H = 256;  // never below 2 KB: the RANDOM policy reuses the table's memory for a 257-word histogram
  while (H < 2 * k) H <<= 1;
  return H;
}

size_t resolve_smem_bytes(int B, int k) {
  const int H = hash_size(k), W = (B + 31) / 32;
  return (size_t)H * 8 + (size_t)4 * k * 4 + (size_t)4 * W * 4 + (size_t)((B + 7) & ~7) * 2 + (size_t)k * 2;
}

cudaStream_t as_stream(void *s) { return static_cast<cudaStream_t>(s); }

const void *resolve_kernel_of(int threads) {
  return threads == kThreadsSmall ? reinterpret_cast<const void *>(&resolve_kernel<kThreadsSmall>)
                                  : reinterpret_cast<const void *>(&resolve_kernel<kThreads>);
}

int launch_resolve(hisparse *h, int layer, const int32_t *sel, int32_t *table, int32_t *hits, int32_t *misses,
                   cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(h->d.N * h->S));
  cfg.blockDim = dim3((unsigned)h->T);
  cfg.dynamicSmemBytes = h->resolve_smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)h->S;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = (h->d.flags & HISPARSE_FLAG_NO_PDL) ? 1 : 2;
  if (h->T == kThreadsSmall)
    HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreadsSmall>, h->d, layer, sel, table, hits, misses, h->S));
  else
    HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreads>, h->d, layer, sel, table, hits, misses, h->S));
  return HISPARSE_OK;
}

int launch_replay(hisparse *h, int layer, cudaStream_t st) {
  replay_kernel<<<h->d.N * h->S, h->T, h->replay_smem, st>>>(h->d, layer, h->S);
  HS_CUDA(cudaGetLastError());
  return HISPARSE_OK;
}

}  // namespace

// ------------------------------------------------------------------------------------------ C-ABI

extern "C" {

const char *hisparse_strerror(int code) {
  switch (code) {
    case HISPARSE_OK: return "ok";
    case HISPARSE_EINVAL: return "invalid argument or geometry";
    case HISPARSE_ENOTPINNED: return "host history is not pinned, device-mapped host memory";
    case HISPARSE_ENOMEM: return "out of memory";
    case HISPARSE_ECUDA: return "CUDA call failed";
    case HISPARSE_ESTATE: return "call not valid in the current state";
    case HISPARSE_ETOOBIG: return "geometry exceeds the fixed scratch of hisparse_resolve_noalloc";
    default: return "unknown error";
  }
}

int hisparse_last_cuda_error(void) { return g_last_cuda_error; }

int hisparse_device_bytes(const hisparse_config_t *c, size_t *kv_bytes, size_t *meta_bytes) {
  const int rc = validate_config(c);
  if (rc) return rc;
  const size_t N = c->num_requests, L = c->num_layers, G = L / c->layers_per_group, B = c->cache_slots, k = c->top_k;
  if (kv_bytes) *kv_bytes = N * L * (B + 1) * (size_t)c->entry_bytes;
  if (meta_bytes) {
    size_t cap_sum = 0;
    for (size_t r = 0; r < N; ++r) cap_sum += (size_t)c->capacity[r];
    *meta_bytes = N * G * B * (4 + 4 + 2)          /* slot_pos, last_use, order */
                  + cap_sum * G * 2                 /* page tables */
                  + N * G * k * 4 * 3               /* plan_pos, plan_slot, anchor_out */
                  + N * G * 4 * 5                   /* t, order_t, plan_n, anchor hits / misses */
                  + N * (8 * 3 + 8) + 16;           /* cap, init_len, p2s_off, host pointers, scalars */
  }
  return HISPARSE_OK;
}

int hisparse_create(const hisparse_config_t *c, hisparse_t **out) {
  if (!out) return HISPARSE_EINVAL;
  *out = nullptr;
  int rc = validate_config(c);
  if (rc) return rc;
  if (!c->host_history) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(c->device));
  const int N = c->num_requests, L = c->num_layers, G = L / c->layers_per_group, B = c->cache_slots, k = c->top_k;

  std::vector<uint8_t *> host_dev(N);
  for (int r = 0; r < N; ++r) {
    if (!c->host_history[r] || ((uintptr_t)c->host_history[r] & 15)) return HISPARSE_EINVAL;
    cudaPointerAttributes a;
    cudaError_t e = cudaPointerGetAttributes(&a, c->host_history[r]);
    if (e != cudaSuccess) { cudaGetLastError(); return HISPARSE_ENOTPINNED; }
    if (a.type != cudaMemoryTypeHost || !a.devicePointer) return HISPARSE_ENOTPINNED;
    host_dev[r] = static_cast<uint8_t *>(a.devicePointer);
  }

  hisparse *h = new (std::nothrow) hisparse();
  if (!h) return HISPARSE_ENOMEM;
  auto fail = [&](int code) { hisparse_destroy(h); return code; };
  h->device = c->device;
  DevState &d = h->d;
  d.N = N; d.L = L; d.lpg = c->layers_per_group; d.G = G; d.B = B; d.k = k;
  d.H = hash_size(k); d.W = (B + 31) / 32;
  d.hshift = 32;
  for (int x = d.H; x > 1; x >>= 1) --d.hshift;
  d.E = c->entry_bytes; d.upe = (uint32_t)(c->entry_bytes / 16); d.flags = c->flags;
  d.policy = c->policy; d.policy_seed = c->policy_seed;
  d.layer_pool_bytes = (int64_t)N * (B + 1) * d.E;
  h->cap.assign(c->capacity, c->capacity + N);
  h->init_len.assign(c->init_len, c->init_len + N);
  h->p2s_off.resize(N);
  int64_t off = 0;
  for (int r = 0; r < N; ++r) { h->p2s_off[r] = off; off += h->cap[r] * G; }
  h->p2s_total = off;
  d.uni_cap = h->cap[0];
  d.uni_init_len = h->init_len[0];
  for (int r = 1; r < N; ++r)
    if (h->cap[r] != h->cap[0] || h->init_len[r] != h->init_len[0]) d.uni_cap = d.uni_init_len = -1;

  int max_optin = 0, smem_per_sm = 0, sm_count = 0;
  if (cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device) != cudaSuccess) return fail(HISPARSE_ECUDA);
  if (cudaDeviceGetAttribute(&smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, c->device) != cudaSuccess) return fail(HISPARSE_ECUDA);
  if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) return fail(HISPARSE_ECUDA);
  h->sm_count = sm_count;
  if (cudaFuncSetAttribute(gather_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 112 * 1024) != cudaSuccess) return fail(HISPARSE_ECUDA);
  // Block size.  One 1024-thread block per SM gives a request the whole SM and all of its shared memory for the
  // fetch ring.  When the grid takes several waves anyway (more blocks than SMs), two 512-thread blocks per SM hide
  // each other's dependent trips to memory; each then gets half of the SM's shared memory.
  int want = c->ctas_per_request;
  if (!want) {
    want = 1;
    while (want < 8 && N * want < 32) want <<= 1;
  }
  d.meta_smem = (int)((resolve_smem_bytes(B, k) + 127) & ~(size_t)127);
  const int64_t budget_small = smem_per_sm / 2 - 1024 - 256;   // per block: 1 KB reserved by the system, static arrays
  const bool fits_small = B <= 16 * kThreadsSmall && k <= 4 * kThreadsSmall &&
                          budget_small - d.meta_smem - kBarBytes >= std::min<int64_t>(d.E, 8192) * 8;
  if ((c->flags & HISPARSE_FLAG_NARROW_BLOCKS) && ((c->flags & HISPARSE_FLAG_WIDE_BLOCKS) || !fits_small)) return fail(HISPARSE_EINVAL);
  const bool small = fits_small && !(c->flags & HISPARSE_FLAG_WIDE_BLOCKS) &&
                     ((c->flags & HISPARSE_FLAG_NARROW_BLOCKS) || (int64_t)N * want > sm_count);
  h->T = small ? kThreadsSmall : kThreads;
  const int64_t budget = small ? budget_small : (int64_t)max_optin - 1024;
  // shared memory: metadata arrays, one mbarrier per thread, then the staging ring of the fetch pipeline,
  // which takes whatever is left (pieces of at most 8 KB; at least one piece must fit)
  const int64_t ring_room = budget - d.meta_smem - kBarBytes;
  if (ring_room < 16) return fail(HISPARSE_EINVAL);
  d.io_chunk = (int)std::min<int64_t>(std::min<int64_t>(d.E, 8192), ring_room & ~(int64_t)15);
  const int slots = (int)(ring_room / d.io_chunk);
  d.io_threads = std::min(slots, h->T);
  d.io_depth = std::min(slots / d.io_threads, 8);
  d.ring_bytes = d.io_threads * d.io_depth * d.io_chunk;
  d.io_ppr = (int)((d.E + d.io_chunk - 1) / d.io_chunk);
  h->resolve_smem = (size_t)d.meta_smem + kBarBytes + (size_t)d.ring_bytes;
  h->replay_smem = h->resolve_smem;   // same offsets, so that both kernels share the pipeline's geometry
  const void *kern = resolve_kernel_of(h->T);
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_optin - 1024) != cudaSuccess) return fail(HISPARSE_ECUDA);
  if (cudaFuncSetAttribute(replay_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, max_optin - 1024) != cudaSuccess) return fail(HISPARSE_ECUDA);

  // Blocks per request: enough of them that about 32 blocks pull on the host link together (measured: fewer
  // leave it under-used when requests are few, more only add launch and barrier cost), as long as all N
  // clusters are resident at once.
  if (c->ctas_per_request) {
    h->S = c->ctas_per_request;
  } else {
    h->S = 1;
    for (int s = want; s > 1; s >>= 1) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)(N * s));
      cfg.blockDim = dim3((unsigned)h->T);
      cfg.dynamicSmemBytes = h->resolve_smem;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeClusterDimension;
      attr[0].val.clusterDim.x = (unsigned)s; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
      cfg.attrs = attr; cfg.numAttrs = 1;
      int nclusters = 0;
      if (cudaOccupancyMaxActiveClusters(&nclusters, kern, &cfg) == cudaSuccess && nclusters >= N) { h->S = s; break; }
      cudaGetLastError();
    }
  }

#define HS_TRY(expr) do { int rc_ = (expr); if (rc_) return fail(rc_); } while (0)
  const size_t NG = (size_t)N * G;
  HS_TRY(dev_alloc(h, &d.pool, (size_t)L * d.layer_pool_bytes));
  HS_TRY(dev_alloc(h, &d.slot_pos, NG * B));
  HS_TRY(dev_alloc(h, &d.last_use, NG * B));
  HS_TRY(dev_alloc(h, &d.order, NG * B));
  HS_TRY(dev_alloc(h, &d.pos2slot, (size_t)h->p2s_total));
  HS_TRY(dev_alloc(h, &h->d_cap, (size_t)N));
  HS_TRY(dev_alloc(h, &h->d_init_len, (size_t)N));
  HS_TRY(dev_alloc(h, &h->d_p2s_off, (size_t)N));
  HS_TRY(dev_alloc(h, &h->d_host, (size_t)N));
  HS_TRY(dev_alloc(h, &d.t, NG));
  if (!(c->flags & HISPARSE_FLAG_EAGER_ORDER)) HS_TRY(dev_alloc(h, &d.order_t, NG));
  HS_TRY(dev_alloc(h, &d.plan_pos, NG * k));
  HS_TRY(dev_alloc(h, &d.plan_slot, NG * k));
  HS_TRY(dev_alloc(h, &d.plan_n, NG));
  HS_TRY(dev_alloc(h, &d.anchor_out, NG * k));
  HS_TRY(dev_alloc(h, &d.anchor_hits, NG));
  HS_TRY(dev_alloc(h, &d.anchor_misses, NG));
  HS_TRY(dev_alloc(h, &d.n_appends, 1));
  HS_TRY(dev_alloc(h, &d.ticket, 1));
  HS_TRY(dev_alloc(h, &d.status, 1));
  HS_TRY(dev_alloc(h, &h->hint_table, (size_t)N * k));
  HS_TRY(dev_alloc(h, &h->hint_hits, (size_t)N));
  HS_TRY(dev_alloc(h, &h->hint_misses, (size_t)N));
  HS_TRY(dev_alloc(h, &d.phase_ns, (size_t)N * 16));
#undef HS_TRY
  d.cap = h->d_cap; d.init_len = h->d_init_len; d.p2s_off = h->d_p2s_off; d.host = h->d_host;

#define HS_TRYC(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { g_last_cuda_error = (int)e_; return fail(HISPARSE_ECUDA); } } while (0)
  HS_TRYC(cudaMemcpy(h->d_cap, h->cap.data(), sizeof(int64_t) * N, cudaMemcpyHostToDevice));
  HS_TRYC(cudaMemcpy(h->d_init_len, h->init_len.data(), sizeof(int64_t) * N, cudaMemcpyHostToDevice));
  HS_TRYC(cudaMemcpy(h->d_p2s_off, h->p2s_off.data(), sizeof(int64_t) * N, cudaMemcpyHostToDevice));
  HS_TRYC(cudaMemcpy(h->d_host, host_dev.data(), sizeof(uint8_t *) * N, cudaMemcpyHostToDevice));
  HS_TRYC(cudaMemset(d.pool, 0, (size_t)L * d.layer_pool_bytes));
  HS_TRYC(cudaMemset(d.slot_pos, 0xff, NG * B * 4));
  HS_TRYC(cudaMemset(d.last_use, 0, NG * B * 4));
  HS_TRYC(cudaMemset(d.pos2slot, 0xff, (size_t)h->p2s_total * 2));
  HS_TRYC(cudaMemset(d.t, 0, NG * 4));
  if (d.order_t) HS_TRYC(cudaMemset(d.order_t, 0, NG * 4));
  HS_TRYC(cudaMemset(d.plan_n, 0, NG * 4));
  HS_TRYC(cudaMemset(d.anchor_out, 0xff, NG * k * 4));
  HS_TRYC(cudaMemset(d.anchor_hits, 0, NG * 4));
  HS_TRYC(cudaMemset(d.anchor_misses, 0, NG * 4));
  HS_TRYC(cudaMemset(d.n_appends, 0, 4));
  HS_TRYC(cudaMemset(d.ticket, 0, 4));
  HS_TRYC(cudaMemset(d.status, 0, 4));
  HS_TRYC(cudaMemset(d.phase_ns, 0, (size_t)N * 16 * 8));
  init_order_kernel<<<296, 256>>>(d.order, (int64_t)NG * B, B);
  HS_TRYC(cudaGetLastError());

  HS_TRYC(cudaStreamCreateWithFlags(&h->backup, cudaStreamNonBlocking));
  HS_TRYC(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
  HS_TRYC(cudaEventCreateWithFlags(&h->ev_wt, cudaEventDisableTiming));
  h->ev_plan.assign(G, nullptr);
  h->ev_pref.assign(L, nullptr);
  for (int g = 0; g < G; ++g) HS_TRYC(cudaEventCreateWithFlags(&h->ev_plan[g], cudaEventDisableTiming));
  for (int l = 0; l < L; ++l) HS_TRYC(cudaEventCreateWithFlags(&h->ev_pref[l], cudaEventDisableTiming));
  HS_TRYC(cudaEventCreateWithFlags(&h->ev_hint_fork, cudaEventDisableTiming));
  h->ev_hint.assign(L, nullptr);
  for (int l = 0; l < L; ++l) HS_TRYC(cudaEventCreateWithFlags(&h->ev_hint[l], cudaEventDisableTiming));
  h->hint_unjoined.assign(L, 0);
  h->anchor_done.assign(G, 0);
  h->replayed.assign(L, 0);
  h->pref_unjoined.assign(L, 0);
  HS_TRYC(cudaDeviceSynchronize());
#undef HS_TRYC
  *out = h;
  return HISPARSE_OK;
}

int hisparse_destroy(hisparse_t *h) {
  if (!h) return HISPARSE_EINVAL;
  cudaSetDevice(h->device);
  cudaDeviceSynchronize();
  for (cudaEvent_t e : h->ev_plan) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_pref) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_hint) if (e) cudaEventDestroy(e);
  if (h->ev_hint_fork) cudaEventDestroy(h->ev_hint_fork);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_wt) cudaEventDestroy(h->ev_wt);
  if (h->backup) cudaStreamDestroy(h->backup);
  for (void *p : h->allocs) cudaFree(p);
  delete h;
  return HISPARSE_OK;
}

int hisparse_join(hisparse_t *h, void *stream) {
  if (!h) return HISPARSE_EINVAL;
  cudaStream_t st = as_stream(stream);
  if (h->wt_pending) {
    HS_CUDA(cudaStreamWaitEvent(st, h->ev_wt, 0));
    h->wt_pending = false;
  }
  for (int l = 0; l < h->d.L; ++l) {
    if (h->pref_unjoined[l]) {
      HS_CUDA(cudaStreamWaitEvent(st, h->ev_pref[l], 0));
      h->pref_unjoined[l] = 0;
    }
    if (h->hint_unjoined[l]) {
      HS_CUDA(cudaStreamWaitEvent(st, h->ev_hint[l], 0));
      h->hint_unjoined[l] = 0;
    }
  }
  return HISPARSE_OK;
}

int hisparse_append(hisparse_t *h, const void *new_kv_dev, void *stream) {
  if (!h || !new_kv_dev) return HISPARSE_EINVAL;
  cudaStream_t st = as_stream(stream);
  const bool inline_wt = h->d.flags & HISPARSE_FLAG_INLINE_WRITE_THROUGH;
  if (h->wt_pending) {  // the previous write-through still reads the reserved slots
    HS_CUDA(cudaStreamWaitEvent(st, h->ev_wt, 0));
    h->wt_pending = false;
  }
  append_kernel<<<h->d.N * h->d.L, 256, 0, st>>>(h->d, static_cast<const uint8_t *>(new_kv_dev), inline_wt ? 1 : 0);
  HS_CUDA(cudaGetLastError());
  if (!inline_wt) {
    HS_CUDA(cudaEventRecord(h->ev_fork, st));
    HS_CUDA(cudaStreamWaitEvent(h->backup, h->ev_fork, 0));
    write_through_kernel<<<h->d.N * h->d.L, 256, 0, h->backup>>>(h->d);
    HS_CUDA(cudaGetLastError());
    HS_CUDA(cudaEventRecord(h->ev_wt, h->backup));
    h->wt_pending = true;
  }
  return HISPARSE_OK;
}

int hisparse_resolve(hisparse_t *h, int layer, const int32_t *sel_dev, int32_t *slot_table_dev, int32_t *hits_dev,
                     int32_t *misses_dev, void *stream) {
  if (!h || layer < 0 || layer >= h->d.L || !slot_table_dev || !hits_dev || !misses_dev) return HISPARSE_EINVAL;
  cudaStream_t st = as_stream(stream);
  const int lpg = h->d.lpg, g = layer / lpg;
  int rc = HISPARSE_OK;
  if (layer % lpg == 0) {
    if (!sel_dev) return HISPARSE_EINVAL;
    if (h->hint_unjoined[layer]) {  // a speculative hint for this layer is still in flight on a side stream
      HS_CUDA(cudaStreamWaitEvent(st, h->ev_hint[layer], 0));
      h->hint_unjoined[layer] = 0;
    }
    // replays of the previous plan of this group must be over before the plan is overwritten
    for (int l = layer + 1; l < layer + lpg; ++l)
      if (h->pref_unjoined[l]) {
        HS_CUDA(cudaStreamWaitEvent(st, h->ev_pref[l], 0));
        h->pref_unjoined[l] = 0;
      }
    rc = launch_resolve(h, layer, sel_dev, slot_table_dev, hits_dev, misses_dev, st);
    if (rc) return rc;
    if (lpg > 1) {
      HS_CUDA(cudaEventRecord(h->ev_plan[g], st));
      for (int l = layer + 1; l < layer + lpg; ++l) h->replayed[l] = 0;
    }
    h->anchor_done[g] = 1;
    if (h->d.flags & HISPARSE_FLAG_DEBUG_VALIDATE) {
      validate_kernel<<<h->d.N, 256, (size_t)h->d.W * 4, st>>>(h->d, g);
      HS_CUDA(cudaGetLastError());
    }
  } else {
    if (!h->anchor_done[g]) return HISPARSE_ESTATE;
    if (h->pref_unjoined[layer]) {
      HS_CUDA(cudaStreamWaitEvent(st, h->ev_pref[layer], 0));
      h->pref_unjoined[layer] = 0;
    } else if (!h->replayed[layer]) {  // no prefetch was issued: synchronous swap-in on the caller's stream
      rc = launch_replay(h, layer, st);
      if (rc) return rc;
      h->replayed[layer] = 1;
    }
    shared_table_kernel<<<h->d.N, 256, 0, st>>>(h->d, layer, slot_table_dev, hits_dev, misses_dev);
    HS_CUDA(cudaGetLastError());
  }
  if (layer == h->d.L - 1 && h->wt_pending) {
    HS_CUDA(cudaStreamWaitEvent(st, h->ev_wt, 0));
    h->wt_pending = false;
  }
  return HISPARSE_OK;
}

int hisparse_prefetch(hisparse_t *h, int layer, void *side_stream) {
  if (!h || layer < 0 || layer >= h->d.L || layer % h->d.lpg == 0) return HISPARSE_EINVAL;
  const int g = layer / h->d.lpg;
  if (!h->anchor_done[g]) return HISPARSE_ESTATE;
  if (h->replayed[layer]) return HISPARSE_OK;
  cudaStream_t st = as_stream(side_stream);
  HS_CUDA(cudaStreamWaitEvent(st, h->ev_plan[g], 0));
  const int rc = launch_replay(h, layer, st);
  if (rc) return rc;
  HS_CUDA(cudaEventRecord(h->ev_pref[layer], st));
  h->replayed[layer] = 1;
  h->pref_unjoined[layer] = 1;
  return HISPARSE_OK;
}

int hisparse_prefetch_hint(hisparse_t *h, int layer, const int32_t *hint_sel_dev, void *stream, void *side_stream) {
  if (!h || layer < 0 || layer >= h->d.L || !hint_sel_dev) return HISPARSE_EINVAL;
  if (h->d.lpg != 1) return HISPARSE_EINVAL;  // shared-selection groups use the exact prefetch instead
  cudaStream_t st = as_stream(stream), side = as_stream(side_stream);
  HS_CUDA(cudaEventRecord(h->ev_hint_fork, st));
  HS_CUDA(cudaStreamWaitEvent(side, h->ev_hint_fork, 0));
  if (h->hint_unjoined[layer]) {  // an earlier hint for the same layer: keep them in order
    HS_CUDA(cudaStreamWaitEvent(side, h->ev_hint[layer], 0));
  }
  const int rc = launch_resolve(h, layer, hint_sel_dev, h->hint_table, h->hint_hits, h->hint_misses, side);
  if (rc) return rc;
  h->anchor_done[layer] = 1;
  HS_CUDA(cudaEventRecord(h->ev_hint[layer], side));
  h->hint_unjoined[layer] = 1;
  return HISPARSE_OK;
}

const void *hisparse_layer_pool(const hisparse_t *h, int layer) {
  if (!h || layer < 0 || layer >= h->d.L) return nullptr;
  return h->d.pool + (int64_t)layer * h->d.layer_pool_bytes;
}

int hisparse_gather(hisparse_t *h, int layer, const int32_t *slot_table_dev, void *out_dev, void *stream) {
  if (!h || layer < 0 || layer >= h->d.L || !slot_table_dev || !out_dev) return HISPARSE_EINVAL;
  if ((uintptr_t)out_dev & 15) return HISPARSE_EINVAL;  // bulk copies need 16-byte aligned addresses
  const int chunk = (int)std::min<int64_t>(h->d.E, 8192);
  const int active = (int)std::min<int64_t>(kGatherThreads, (96 * 1024) / chunk);
  const size_t smem = (size_t)kGatherThreads * 8 + (size_t)chunk + (size_t)active * chunk;
  gather_kernel<<<2 * h->sm_count, kGatherThreads, smem, as_stream(stream)>>>(h->d, layer, slot_table_dev,
                                                                             static_cast<uint8_t *>(out_dev), chunk, active);
  HS_CUDA(cudaGetLastError());
  return HISPARSE_OK;
}

int hisparse_gather_check(hisparse_t *h, int layer, const int32_t *sel_dev, const int32_t *slot_table_dev,
                          int32_t *mismatches_dev, void *stream) {
  if (!h || layer < 0 || layer >= h->d.L || !sel_dev || !slot_table_dev || !mismatches_dev) return HISPARSE_EINVAL;
  const int rc = hisparse_join(h, stream);
  if (rc) return rc;
  // a shared layer is compared against its own history; the selections are its anchor's
  gather_check_kernel<<<592, 256, 0, as_stream(stream)>>>(h->d, layer, sel_dev, slot_table_dev, mismatches_dev);
  HS_CUDA(cudaGetLastError());
  return HISPARSE_OK;
}

int hisparse_status(hisparse_t *h, uint32_t *bits) {
  if (!h || !bits) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemcpy(bits, h->d.status, 4, cudaMemcpyDeviceToHost));
  return HISPARSE_OK;
}

int hisparse_clear_status(hisparse_t *h) {
  if (!h) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemset(h->d.status, 0, 4));
  return HISPARSE_OK;
}

int hisparse_dump_state(hisparse_t *h, int req, int layer, int32_t *slot_pos, uint32_t *last_use, int32_t *lru_order,
                        int32_t *pos2slot, int64_t *len, int64_t *newest, uint32_t *resolves) {
  if (!h || req < 0 || req >= h->d.N || layer < 0 || layer >= h->d.L) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  const int B = h->d.B, g = layer / h->d.lpg;
  const int64_t rg = (int64_t)req * h->d.G + g;
  if (slot_pos) HS_CUDA(cudaMemcpy(slot_pos, h->d.slot_pos + rg * B, (size_t)B * 4, cudaMemcpyDeviceToHost));
  if (last_use) HS_CUDA(cudaMemcpy(last_use, h->d.last_use + rg * B, (size_t)B * 4, cudaMemcpyDeviceToHost));
  if (lru_order) {
    std::vector<uint16_t> tmp(B);
    HS_CUDA(cudaMemcpy(tmp.data(), h->d.order + rg * B, (size_t)B * 2, cudaMemcpyDeviceToHost));
    for (int i = 0; i < B; ++i) lru_order[i] = tmp[i];
  }
  if (pos2slot) {
    std::vector<int16_t> tmp((size_t)h->cap[req]);
    HS_CUDA(cudaMemcpy(tmp.data(), h->d.pos2slot + h->p2s_off[req] + (int64_t)g * h->cap[req], (size_t)h->cap[req] * 2,
                       cudaMemcpyDeviceToHost));
    for (int64_t i = 0; i < h->cap[req]; ++i) pos2slot[i] = tmp[(size_t)i];
  }
  int32_t na = 0;
  HS_CUDA(cudaMemcpy(&na, h->d.n_appends, 4, cudaMemcpyDeviceToHost));
  const int64_t il = h->init_len[req], cap = h->cap[req];
  if (len) *len = std::min(il + na, cap);
  if (newest) *newest = (na > 0 && il + na <= cap) ? il + na - 1 : -1;
  if (resolves) HS_CUDA(cudaMemcpy(resolves, h->d.t + rg, 4, cudaMemcpyDeviceToHost));
  return HISPARSE_OK;
}

int hisparse_order_lag(hisparse_t *h, int req, int layer, uint32_t *lag) {
  if (!h || req < 0 || req >= h->d.N || layer < 0 || layer >= h->d.L || !lag) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  *lag = 0;
  if (!h->d.order_t) return HISPARSE_OK;
  const int64_t rg = (int64_t)req * h->d.G + layer / h->d.lpg;
  uint32_t t = 0, ot = 0;
  HS_CUDA(cudaMemcpy(&t, h->d.t + rg, 4, cudaMemcpyDeviceToHost));
  HS_CUDA(cudaMemcpy(&ot, h->d.order_t + rg, 4, cudaMemcpyDeviceToHost));
  *lag = t - ot;
  return HISPARSE_OK;
}

int hisparse_load_state(hisparse_t *h, int req, int layer, const int32_t *slot_pos, const uint32_t *last_use,
                        uint32_t resolves) {
  if (!h || req < 0 || req >= h->d.N || layer < 0 || layer >= h->d.L || !slot_pos || !last_use) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  const int B = h->d.B, lpg = h->d.lpg, g = layer / lpg;
  const int64_t rg = (int64_t)req * h->d.G + g, cap = h->cap[req];
  int32_t na = 0;
  HS_CUDA(cudaMemcpy(&na, h->d.n_appends, 4, cudaMemcpyDeviceToHost));
  const int64_t len = std::min(h->init_len[req] + na, cap);
  // the page table is the inverse of slot_pos; positions must be distinct and inside the history
  std::vector<int16_t> p2s((size_t)cap, (int16_t)-1);
  for (int s = 0; s < B; ++s) {
    const int32_t p = slot_pos[s];
    if (p == -1) continue;
    if (p < 0 || p >= len || p2s[(size_t)p] != -1) return HISPARSE_EINVAL;
    p2s[(size_t)p] = (int16_t)s;
  }
  // the recency order is the slots sorted by (stamp, slot)
  std::vector<uint16_t> order((size_t)B);
  for (int s = 0; s < B; ++s) order[(size_t)s] = (uint16_t)s;
  std::stable_sort(order.begin(), order.end(), [&](uint16_t a, uint16_t b) { return last_use[a] < last_use[b]; });
  HS_CUDA(cudaMemcpy(h->d.slot_pos + rg * B, slot_pos, (size_t)B * 4, cudaMemcpyHostToDevice));
  HS_CUDA(cudaMemcpy(h->d.last_use + rg * B, last_use, (size_t)B * 4, cudaMemcpyHostToDevice));
  HS_CUDA(cudaMemcpy(h->d.order + rg * B, order.data(), (size_t)B * 2, cudaMemcpyHostToDevice));
  HS_CUDA(cudaMemcpy(h->d.pos2slot + h->p2s_off[req] + (int64_t)g * cap, p2s.data(), (size_t)cap * 2, cudaMemcpyHostToDevice));
  HS_CUDA(cudaMemcpy(h->d.t + rg, &resolves, 4, cudaMemcpyHostToDevice));
  if (h->d.order_t) HS_CUDA(cudaMemcpy(h->d.order_t + rg, &resolves, 4, cudaMemcpyHostToDevice));  // the list is current
  const int32_t zero = 0;
  HS_CUDA(cudaMemcpy(h->d.plan_n + rg, &zero, 4, cudaMemcpyHostToDevice));
  // the host history is authoritative: refill every layer of the group from it (resident records + newest record)
  cudaPointerAttributes a;
  HS_CUDA(cudaPointerGetAttributes(&a, h->d.pool));
  (void)a;
  std::vector<uint8_t *> host(h->d.N);
  HS_CUDA(cudaMemcpy(host.data(), h->d_host, sizeof(uint8_t *) * h->d.N, cudaMemcpyDeviceToHost));
  const int64_t E = h->d.E;
  for (int l = g * lpg; l < (g + 1) * lpg; ++l) {
    uint8_t *pool = h->d.pool + (int64_t)l * h->d.layer_pool_bytes + (int64_t)req * (B + 1) * E;
    const uint8_t *hist = host[req] + (int64_t)l * cap * E;   // device-visible alias of the pinned history
    for (int s = 0; s < B; ++s)
      if (slot_pos[s] >= 0)
        HS_CUDA(cudaMemcpyAsync(pool + (int64_t)s * E, hist + (int64_t)slot_pos[s] * E, (size_t)E, cudaMemcpyDefault, nullptr));
    if (na > 0 && h->init_len[req] + na <= cap)
      HS_CUDA(cudaMemcpyAsync(pool + (int64_t)B * E, hist + (len - 1) * E, (size_t)E, cudaMemcpyDefault, nullptr));
  }
  HS_CUDA(cudaDeviceSynchronize());
  return HISPARSE_OK;
}

int hisparse_load_appends(hisparse_t *h, int32_t appends) {
  if (!h || appends < 0) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemcpy(h->d.n_appends, &appends, 4, cudaMemcpyHostToDevice));
  return HISPARSE_OK;
}

int hisparse_dump_plan(hisparse_t *h, int req, int layer, int32_t *plan_pos, int32_t *plan_slot, int32_t *n) {
  if (!h || req < 0 || req >= h->d.N || layer < 0 || layer >= h->d.L || !n) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  const int64_t rg = (int64_t)req * h->d.G + layer / h->d.lpg;
  HS_CUDA(cudaMemcpy(n, h->d.plan_n + rg, 4, cudaMemcpyDeviceToHost));
  if (plan_pos) HS_CUDA(cudaMemcpy(plan_pos, h->d.plan_pos + rg * h->d.k, (size_t)h->d.k * 4, cudaMemcpyDeviceToHost));
  if (plan_slot) HS_CUDA(cudaMemcpy(plan_slot, h->d.plan_slot + rg * h->d.k, (size_t)h->d.k * 4, cudaMemcpyDeviceToHost));
  return HISPARSE_OK;
}

int hisparse_phase_times(hisparse_t *h, uint64_t *out) {
  if (!h || !out) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemcpy(out, h->d.phase_ns, (size_t)h->d.N * 16 * 8, cudaMemcpyDeviceToHost));
  return HISPARSE_OK;
}

int hisparse_selftest_wait_timeout(hisparse_t *h, uint64_t limit_ns, uint64_t *waited_ns) {
  if (!h || !waited_ns || limit_ns == 0 || limit_ns > 1000000000ull) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(h->device));
  wait_timeout_selftest_kernel<<<1, 32>>>(h->d.status, limit_ns, h->d.phase_ns);
  HS_CUDA(cudaGetLastError());
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemcpy(waited_ns, h->d.phase_ns, 8, cudaMemcpyDeviceToHost));
  return HISPARSE_OK;
}

int hisparse_launch_geometry(const hisparse_t *h, int32_t *ctas_per_request, int32_t *threads, int32_t *smem_bytes) {
  if (!h) return HISPARSE_EINVAL;
  if (ctas_per_request) *ctas_per_request = h->S;
  if (threads) *threads = h->T;
  if (smem_bytes) *smem_bytes = (int32_t)h->resolve_smem;
  return HISPARSE_OK;
}

int hisparse_host_alloc(size_t bytes, void **out) {
  if (!out || !bytes) return HISPARSE_EINVAL;
  *out = nullptr;
  cudaError_t e = cudaHostAlloc(out, bytes, cudaHostAllocPortable | cudaHostAllocMapped);
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; cudaGetLastError(); return HISPARSE_ENOMEM; }
  return HISPARSE_OK;
}

int hisparse_host_free(void *p) {
  if (!p) return HISPARSE_EINVAL;
  HS_CUDA(cudaFreeHost(p));
  return HISPARSE_OK;
}

int hisparse_host_link_probe(int device, size_t bytes, int reps, double *gb_per_s) {
  if (!gb_per_s || !bytes || reps < 1) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(device));
  void *hbuf = nullptr, *dbuf = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  int rc = HISPARSE_OK;
  float best = 0.f;
  cudaError_t e = cudaHostAlloc(&hbuf, bytes, cudaHostAllocPortable);
  if (e == cudaSuccess) e = cudaMalloc(&dbuf, bytes);
  if (e == cudaSuccess) { memset(hbuf, 0x5a, bytes); e = cudaEventCreate(&e0); }
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  for (int i = 0; e == cudaSuccess && i < reps + 1; ++i) {  // the first pass is a warm-up
    cudaEventRecord(e0, nullptr);
    e = cudaMemcpyAsync(dbuf, hbuf, bytes, cudaMemcpyHostToDevice, nullptr);
    cudaEventRecord(e1, nullptr);
    if (e == cudaSuccess) e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e == cudaSuccess && i > 0 && (best == 0.f || ms < best)) best = ms;
  }
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; cudaGetLastError(); rc = e == cudaErrorMemoryAllocation ? HISPARSE_ENOMEM : HISPARSE_ECUDA; }
  else *gb_per_s = (double)bytes / ((double)best * 1e6);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (dbuf) cudaFree(dbuf);
  if (hbuf) cudaFreeHost(hbuf);
  return rc;
}

int hisparse_scatter_read_probe(int device, const void *host_buf, size_t host_bytes, int64_t entry_bytes,
                                int32_t num_records, int32_t num_ctas, int reps, double *gb_per_s) {
  if (!gb_per_s || !host_buf || entry_bytes < 16 || entry_bytes % 16 || num_records < 1 || num_ctas < 1 || reps < 1)
    return HISPARSE_EINVAL;
  const size_t slots = host_bytes / (size_t)entry_bytes;
  if (slots < 1 || slots > 0x7fffffffu) return HISPARSE_EINVAL;
  HS_CUDA(cudaSetDevice(device));
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, host_buf) != cudaSuccess || a.type != cudaMemoryTypeHost || !a.devicePointer) {
    cudaGetLastError();
    return HISPARSE_ENOTPINNED;
  }
  std::vector<int32_t> idx(num_records);
  uint64_t s = 0x2545F4914F6CDD1Dull;
  for (int i = 0; i < num_records; ++i) {
    s ^= s << 13; s ^= s >> 7; s ^= s << 17;
    idx[i] = (int32_t)(s % slots);
  }
  int32_t *d_idx = nullptr;
  uint8_t *d_dst = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  float best = 0.f;
  cudaError_t e = cudaMalloc(&d_idx, (size_t)num_records * 4);
  if (e == cudaSuccess) e = cudaMalloc(&d_dst, (size_t)num_records * entry_bytes);
  if (e == cudaSuccess) e = cudaMemcpy(d_idx, idx.data(), (size_t)num_records * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  for (int i = 0; e == cudaSuccess && i < reps + 2; ++i) {
    cudaEventRecord(e0, nullptr);
    scatter_probe_kernel<<<num_ctas, kThreads>>>(static_cast<const uint8_t *>(a.devicePointer), d_dst, d_idx, num_records,
                                                 (uint32_t)(entry_bytes / 16));
    cudaEventRecord(e1, nullptr);
    e = cudaEventSynchronize(e1);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    if (e == cudaSuccess && i >= 2 && (best == 0.f || ms < best)) best = ms;
  }
  int rc = HISPARSE_OK;
  if (e != cudaSuccess) { g_last_cuda_error = (int)e; cudaGetLastError(); rc = e == cudaErrorMemoryAllocation ? HISPARSE_ENOMEM : HISPARSE_ECUDA; }
  else *gb_per_s = (double)num_records * (double)entry_bytes / ((double)best * 1e6);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (d_dst) cudaFree(d_dst);
  if (d_idx) cudaFree(d_idx);
  return rc;
}


// ------------------------------------------------------------------------------------------ no-allocation entry

}  // extern "C"

namespace {

// Scratch of hisparse_resolve_noalloc, part of the library image: plan positions, plan slots, then per-request
// counters (plan size, hits, misses) and one status word that stands in when the caller passes none.
constexpr size_t kNoAllocPlanBytes = (size_t)HISPARSE_NOALLOC_MAX_SELECTIONS * 4;
constexpr size_t kNoAllocCounterBytes = (size_t)HISPARSE_NOALLOC_MAX_REQUESTS * 4;
constexpr size_t kNoAllocBytes = 2 * kNoAllocPlanBytes + 3 * kNoAllocCounterBytes + 256;
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
unsigned char *g_noalloc_ptr[kMaxDevices] = {};  // device address of the array, looked up once per device
int g_noalloc_optin[kMaxDevices] = {};
std::mutex g_noalloc_mutex;                      // guards the one-time set-up

}  // namespace

extern "C" {

int hisparse_resolve_noalloc(const hisparse_external_state_t *st, const int32_t *sel_dev, int32_t *slot_table_dev,
                             int32_t *hits_dev, int32_t *misses_dev, uint32_t *status_dev, void *stream) {
  if (!st || !sel_dev || !slot_table_dev || !hits_dev || !misses_dev) return HISPARSE_EINVAL;
  const int N = st->num_requests, B = st->cache_slots, k = st->top_k;
  if (N < 1 || k < 1 || k > HISPARSE_MAX_TOP_K || B < k || B > HISPARSE_MAX_CACHE_SLOTS) return HISPARSE_EINVAL;
  if (st->entry_bytes < 16 || st->entry_bytes % 16 || st->entry_bytes / 16 > 0x7fffffff) return HISPARSE_EINVAL;
  if (st->device < 0 || st->device >= kMaxDevices) return HISPARSE_EINVAL;
  if (!st->pool_dev || !st->slot_pos_dev || !st->last_use_dev || !st->lru_order_dev || !st->pos2slot_dev ||
      !st->capacity_dev || !st->init_len_dev || !st->p2s_offset_dev || !st->host_layer_dev || !st->resolves_dev ||
      !st->num_appends_dev)
    return HISPARSE_EINVAL;
  if (N > HISPARSE_NOALLOC_MAX_REQUESTS || (int64_t)N * k > HISPARSE_NOALLOC_MAX_SELECTIONS) return HISPARSE_ETOOBIG;

  const int dev = st->device;
  std::unique_lock<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    // Set-up, once per device, with that device current.  In host code the array's name is only a stand-in for
    // the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
    HS_CUDA(cudaSetDevice(dev));
    void *p = nullptr;
    HS_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    int optin = 0;
    HS_CUDA(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    HS_CUDA(cudaFuncSetAttribute(resolve_kernel<kThreads>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - 1024));
    g_noalloc_optin[dev] = optin;
    g_noalloc_ptr[dev] = static_cast<unsigned char *>(p);
  }
  unsigned char *scratch = g_noalloc_ptr[dev];
  const int optin = g_noalloc_optin[dev];
  lock.unlock();

  DevState d{};  // order_t stays null: the caller's recency list is brought up to date by every call
  d.uni_cap = d.uni_init_len = -1;
  d.N = N; d.L = 1; d.lpg = 1; d.G = 1; d.B = B; d.k = k;
  d.H = hash_size(k); d.W = (B + 31) / 32;
  d.hshift = 32;
  for (int x = d.H; x > 1; x >>= 1) --d.hshift;
  d.E = st->entry_bytes; d.upe = (uint32_t)(st->entry_bytes / 16); d.flags = 0;
  d.layer_pool_bytes = (int64_t)N * (B + 1) * d.E;
  d.pool = static_cast<uint8_t *>(st->pool_dev);
  d.slot_pos = st->slot_pos_dev; d.last_use = st->last_use_dev; d.order = st->lru_order_dev;
  d.pos2slot = st->pos2slot_dev;
  d.cap = st->capacity_dev; d.init_len = st->init_len_dev; d.p2s_off = st->p2s_offset_dev;
  d.host = reinterpret_cast<uint8_t *const *>(st->host_layer_dev);
  d.t = st->resolves_dev;
  d.n_appends = const_cast<int32_t *>(st->num_appends_dev);
  d.plan_pos = reinterpret_cast<int32_t *>(scratch);
  d.plan_slot = reinterpret_cast<int32_t *>(scratch + kNoAllocPlanBytes);
  d.plan_n = reinterpret_cast<int32_t *>(scratch + 2 * kNoAllocPlanBytes);
  d.anchor_hits = reinterpret_cast<int32_t *>(scratch + 2 * kNoAllocPlanBytes + kNoAllocCounterBytes);
  d.anchor_misses = reinterpret_cast<int32_t *>(scratch + 2 * kNoAllocPlanBytes + 2 * kNoAllocCounterBytes);
  d.anchor_out = d.plan_pos;  // only written for shared-selection groups, which this entry point does not have
  d.status = status_dev ? status_dev : reinterpret_cast<uint32_t *>(scratch + 2 * kNoAllocPlanBytes + 3 * kNoAllocCounterBytes);
  d.ticket = nullptr;
  d.phase_ns = nullptr;      // only touched with PHASE_TIMERS, which is off here
  d.meta_smem = (int)((resolve_smem_bytes(B, k) + 127) & ~(size_t)127);
  const int64_t ring_room = (int64_t)optin - 1024 - d.meta_smem - kBarBytes;
  if (ring_room < 16) return HISPARSE_EINVAL;
  d.io_chunk = (int)std::min<int64_t>(std::min<int64_t>(d.E, 8192), ring_room & ~(int64_t)15);
  const int slots = (int)(ring_room / d.io_chunk);
  d.io_threads = std::min(slots, kThreads);
  d.io_depth = std::min(slots / d.io_threads, 8);
  d.ring_bytes = d.io_threads * d.io_depth * d.io_chunk;
  d.io_ppr = (int)((d.E + d.io_chunk - 1) / d.io_chunk);
  const size_t smem = (size_t)d.meta_smem + kBarBytes + (size_t)d.ring_bytes;

  cudaStream_t s = as_stream(stream);
  // the counters other blocks read must not carry the previous call's values into this one
  HS_CUDA(cudaMemsetAsync(scratch + 2 * kNoAllocPlanBytes, 0, 3 * kNoAllocCounterBytes + 256, s));
  const int S = 2;  // two blocks per request: the second one receives the plan through the scratch array
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(N * S));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreads>, d, 0, sel_dev, slot_table_dev, hits_dev, misses_dev, S));
  return HISPARSE_OK;
}

}  // extern "C"
