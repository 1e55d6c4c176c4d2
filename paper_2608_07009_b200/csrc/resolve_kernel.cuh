// Included by hisparse.cu: the Resolve kernel (Sec. 3.4) and its phases.

namespace {

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

}  // namespace
