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

// Block-wide exclusive rank over NB flag bits per thread, thread-major (thread t's bits 0..NB-1 come before thread
// t+1's): returns the number of set bits in all earlier threads.  Ballots and population counts instead of shuffle
// scans; one barrier.  s_warp: 32 ints of scratch, not to be reused before the block has passed another barrier.
template <int NB>
__device__ __forceinline__ int block_rank_bits(const uint32_t bits, int *s_warp, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const uint32_t lt = (1u << lane) - 1u;
  int below = 0, wtot = 0;
#pragma unroll
  for (int i = 0; i < NB; ++i) {
    const uint32_t b = __ballot_sync(0xffffffffu, (bits >> i) & 1u);
    below += __popc(b & lt);
    wtot += __popc(b);
  }
  if (lane == 0) s_warp[warp] = wtot;
  __syncthreads();
  const int w = lane < nw ? s_warp[lane] : 0;
  const int before = __reduce_add_sync(0xffffffffu, lane < warp ? w : 0);
  total = __reduce_add_sync(0xffffffffu, w);
  return before + below;
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

// What a block needs from shared memory, carved out of the dynamic allocation by the offsets fixed at create.
struct SmemView {
  int32_t *sel;                  // the selected row; once consumed, its space holds the recency list (`order`)
  uint16_t *order;
  int32_t *plan_pos, *plan_slot;
  uint16_t *missj;
  uint8_t *marks;                // one byte per slot: == the request's tag when a selection hit the slot
  uint32_t *hitbits, *vicbits;   // hit marks as a bitset (built from `marks` once something missed), victim marks
  int32_t *hitpre, *vicpre;
  int *hist;
  int16_t *got;
  unsigned long long *tab;
  unsigned long long *bars;
  unsigned char *ring;
  int *warp;                     // 32 ints of scratch for block scans
  int *misc;                     // two sets used by alternate requests: [0] a missing position was selected twice
                                 // [1] selections that hit  [2] the newest position was selected  [3] distinct slots hit
};

// `it` = how many requests this block has resolved before the current one (picks the set of flags).
__device__ __forceinline__ SmemView smem_view(const DevState &d, unsigned char *raw, const int it) {
  SmemView v;
  v.sel = reinterpret_cast<int32_t *>(raw);
  v.order = reinterpret_cast<uint16_t *>(raw);
  v.plan_pos = reinterpret_cast<int32_t *>(raw + d.sm_plan_pos);
  v.plan_slot = reinterpret_cast<int32_t *>(raw + d.sm_plan_slot);
  v.missj = reinterpret_cast<uint16_t *>(raw + d.sm_missj);
  const int wpad = (d.W + 3) & ~3;
  v.marks = raw + d.sm_marks;
  v.hitbits = reinterpret_cast<uint32_t *>(raw + d.sm_bits);
  v.vicbits = v.hitbits + wpad;
  v.hitpre = reinterpret_cast<int32_t *>(v.vicbits + wpad);
  v.vicpre = v.hitpre + wpad;
  v.hist = reinterpret_cast<int *>(raw + d.sm_hist);
  v.got = reinterpret_cast<int16_t *>(raw + d.sm_got);
  v.bars = reinterpret_cast<unsigned long long *>(raw + d.meta_smem);
  v.ring = raw + d.meta_smem + d.bar_bytes;
  v.tab = reinterpret_cast<unsigned long long *>(d.sm_tab >= 0 ? raw + d.sm_tab : v.ring);
  v.warp = reinterpret_cast<int *>(raw + d.sm_misc);
  v.misc = v.warp + 32 + (it & 1) * 8;
  return v;
}

// Where a request's slice of the page table is and whether it can be staged in the (still idle) fetch ring.
struct SliceGeom {
  const int16_t *p2s;        // the request's slice (one entry per position)
  uintptr_t aligned;         // its address rounded down to 16 bytes
  int lead;                  // entries between `aligned` and p2s
  int64_t stage_bytes;       // whole 16-byte units that cover the slice
  bool staged;
};

__device__ __forceinline__ SliceGeom slice_geom(const DevState &d, const int g, const int64_t cap_r, const int64_t p2s_off_r) {
  SliceGeom q;
  q.p2s = d.pos2slot + p2s_off_r + (int64_t)g * p2s_stride(cap_r);
  q.aligned = (uintptr_t)q.p2s & ~(uintptr_t)15;
  q.lead = (int)(((uintptr_t)q.p2s - q.aligned) >> 1);
  q.stage_bytes = ((int64_t)q.lead * 2 + cap_r * 2) & ~(int64_t)15;
  q.staged = q.stage_bytes + 16 <= (int64_t)d.ring_bytes;
  return q;
}

// One request's resolve as a block sees it (block-uniform).
struct ReqCtx {
  int r, it, S, layer, g;
  int64_t rg, cap_r, init_len_r, p2s_off_r;
  const int32_t *row;
  int32_t *trow, *arow;
  int32_t *hits_out, *misses_out;
  bool has_next;             // the block takes another request after this one
  int tag;                   // 1..255: what a hit writes into `marks` for this request (so that they need no clearing)
};

__device__ __forceinline__ void request_geom(const DevState &d, const int r, int64_t &cap_r, int64_t &init_len_r,
                                             int64_t &p2s_off_r) {
  const bool uni = d.uni_cap >= 0;  // fixed at create
  cap_r = uni ? d.uni_cap : d.cap[r];
  init_len_r = uni ? d.uni_init_len : d.init_len[r];
  p2s_off_r = uni ? (int64_t)r * d.G * p2s_stride(d.uni_cap) : d.p2s_off[r];
}

// Phase 1: the row and, when it fits the idle fetch ring, the request's slice of the page table start their way to
// shared memory as bulk copies issued by the lanes of the first warp, all completing on one mbarrier (`stage_bar`).
// Staging the slice turns Phase 2's k random lookups into shared-memory reads instead of 32-byte sector reads
// queueing on one SM.  Called by every thread of the block; shapes that bulk copies cannot take (unaligned row, the
// last partial 16-byte unit of the slice) are copied by plain loads, which the consumer orders with a block barrier.
constexpr uint32_t kStagePiece = 16384;  // bytes per bulk copy when a row and a page-table slice are staged (measured:
                                         // 1 KB pieces make the staging slower, not faster)

template <int T>
__device__ __forceinline__ void stage_issue(const DevState &d, const SmemView &v, const SliceGeom &q, const int32_t *row,
                                            const int64_t cap_r, const uint32_t stage_bar) {
  const int tid = threadIdx.x;
  const int k = d.k;
  const bool sel_bulk = (((uintptr_t)row | (uintptr_t)(k * 4)) & 15) == 0;
  if (tid < 32) {
    // pieces of kStagePiece bytes, issued side by side by the lanes of the warp
    const uint32_t row_bytes = sel_bulk ? (uint32_t)k * 4u : 0u, slice_bytes = q.staged ? (uint32_t)q.stage_bytes : 0u;
    if (tid == 0)  // (a copy that lands before this arrival only makes the byte count dip: the phase cannot complete before it)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(stage_bar), "r"(row_bytes + slice_bytes) : "memory");
    const uint32_t row_pieces = (row_bytes + kStagePiece - 1) / kStagePiece, slice_pieces = (slice_bytes + kStagePiece - 1) / kStagePiece;
    for (uint32_t p = (uint32_t)tid; p < row_pieces + slice_pieces; p += 32u) {
      const bool in_row = p < row_pieces;
      const uint32_t o = (in_row ? p : p - row_pieces) * kStagePiece, total = in_row ? row_bytes : slice_bytes;
      const uint32_t n = total - o < kStagePiece ? total - o : kStagePiece;
      const uint32_t dst = (in_row ? smem_u32(v.sel) : smem_u32(v.ring)) + o;
      const char *src = (in_row ? reinterpret_cast<const char *>(row) : reinterpret_cast<const char *>(q.aligned)) + o;
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(dst), "l"(src), "r"(n), "r"(stage_bar) : "memory");
    }
  }
  if (!sel_bulk) stage_async(v.sel, row, k * 4);
  if (q.staged && tid >= 32 && tid < 40) {  // the last, partial 16-byte unit of the slice: plain copies
    const int64_t e = q.stage_bytes / 2 + (tid - 32);
    if (e < q.lead + cap_r) reinterpret_cast<int16_t *>(v.ring)[e] = reinterpret_cast<const int16_t *>(q.aligned)[e];
  }
}

// How a repeated missing position is caught (list_misses): through claims in the staged page-table slice, which
// lookup_phase has already stored (kClaimsStored) or list_misses still has to store (kClaimsPending), or, when the
// slice is not in shared memory, through the table of missing positions (kClaimsNone).
constexpr int kClaimsNone = 0, kClaimsStored = 1, kClaimsPending = 2;

// Phase 2 of Sec. 3.4 as the first block of a cluster runs it, up to the block-wide vote "did anything miss?".
// Thread t owns the KPT consecutive row entries [t*KPT, t*KPT + KPT): it reads them with one vector load, looks them
// up in the page table, marks the slots that hit, and writes its part of the slot table at once (a hit's slot is final;
// an entry that missed gets its slot later, a placeholder for now).  On return pos[] / cls[] hold the thread's
// positions and their classification (slot, B for the newest record, kMiss, or -1), `any_miss` the vote.
// `stage_parity` = phase of the staging barrier that stage_issue's copies for this request complete.
template <int T, int KPT>
__device__ __forceinline__ void lookup_phase(const DevState &d, const SmemView &v, const SliceGeom &q, const ReqCtx &c,
                                             const uint32_t stage_parity, unsigned long long *stamps,
                                             int32_t (&pos)[KPT], int32_t (&cls)[KPT], uint32_t &my_status, bool &any_miss,
                                             uint32_t &t_now, uint32_t &order_t, int &claims) {
  const int tid = threadIdx.x;
  const int k = d.k, B = d.B;
  const int r = c.r, S = c.S;
  const int64_t rg = c.rg, cap_r = c.cap_r, init_len_r = c.init_len_r;
  const int32_t *row = c.row;
  int32_t *trow = c.trow, *arow = c.arow;
  int *s_misc = v.misc;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  const bool coop = !q.staged && S > 1;  // same decision in every block of the cluster (depends on the request only)
  if (coop) cluster_arrive_relaxed();    // phase A, see cluster_lookups
  const uint32_t stage_bar = smem_u32(v.bars + T);
  const bool sel_bulk = (((uintptr_t)row | (uintptr_t)(k * 4)) & 15) == 0;
  // the scalars of this resolve, loaded while the copies fly
  const int64_t na = *(volatile int32_t *)d.n_appends;
  t_now = d.t[rg] + 1u;
  order_t = d.order_t ? d.order_t[rg] : t_now - 1u;  // resolve count the recency list is current for
  const int64_t len = init_len_r + na < cap_r ? init_len_r + na : cap_r;
  const int64_t newest = (na > 0 && init_len_r + na <= cap_r) ? init_len_r + na - 1 : -1;
  if (timers && tid == 0) stamps[8] = clock64();
  if (!sel_bulk) asm volatile("cp.async.wait_all;" ::: "memory");
  // One warp waits for the copies; the others wait for that warp at a block barrier, which costs no issue slots (a
  // block-wide spin on the mbarrier was measured to take most of the instructions of a resolve in which nothing
  // misses, at the expense of the other blocks on the SM).  The barrier also orders the plain copies above.
  bool landed = true;
  if (tid < 32 && !mbar_wait_bounded(stage_bar, stage_parity)) {
    // bounded wait expired: the row cannot be trusted either, so this request resolves nothing in this launch.  The
    // copies get one more bounded chance to land before anything else uses (or the block gives up) their memory.
    mbar_wait_bounded(stage_bar, stage_parity);
    landed = false;
  }
  const bool timed_out = __syncthreads_or(!landed) != 0;
  const bool use_staged = q.staged && !timed_out;
  if (timed_out) my_status |= HISPARSE_STATUS_TIMEOUT;
  if (timers && tid == 0) stamps[9] = clock64();
  int16_t *s_p2s = reinterpret_cast<int16_t *>(v.ring) + q.lead;
  if (coop) cluster_lookups<T>(row, q.p2s, k, len, 0, S, v.got);

  // Phase 2: hit detection through the page table (position -> slot); all of a thread's lookups are issued
  // before the first is used, unconditionally (an entry that is padding or out of range looks up position 0 and
  // discards the answer).
  const int j0 = tid * KPT;
#pragma unroll
  for (int i = 0; i < KPT; ++i) pos[i] = -1;
  if (j0 < k && !timed_out) {
    if constexpr (KPT == 4) {
      const int4 x = *reinterpret_cast<const int4 *>(v.sel + j0);
      pos[0] = x.x; pos[1] = x.y; pos[2] = x.z; pos[3] = x.w;
    } else {
      const int2 x = *reinterpret_cast<const int2 *>(v.sel + j0);
      pos[0] = x.x; pos[1] = x.y;
    }
  }
  int32_t got[KPT];
  const uint32_t ulen = (uint32_t)len;
  int bad = 0;
#pragma unroll
  for (int i = 0; i < KPT; ++i) {
    if (j0 + i >= k) pos[i] = -1;
    const bool ok = (uint32_t)pos[i] < ulen;  // 0 <= p < len (positions and lengths fit 31 bits)
    bad |= (!ok) & (pos[i] != -1);
    const int32_t idx = ok ? pos[i] : 0;
    const int32_t raw = use_staged ? (int32_t)s_p2s[idx] : coop ? (int32_t)v.got[j0 + i < k ? j0 + i : 0] : (int32_t)__ldg(q.p2s + idx);
    pos[i] = ok ? pos[i] : -1;
    got[i] = ok ? raw : -1;
  }
  if (bad) my_status |= HISPARSE_STATUS_OUT_OF_RANGE;
  int miss = 0, nhit = 0;
  int32_t val[KPT];
  const int32_t base = r * (B + 1);
  const uint8_t tag = (uint8_t)c.tag;
  const int32_t inewest = newest >= 0 ? (int32_t)newest : -2;  // -2: no newest record (a discarded entry is -1)
#pragma unroll
  for (int i = 0; i < KPT; ++i) {
    const int32_t p = pos[i];
    int32_t o = -1;
    if (p == inewest) {  // reserved newest-record slot, outside the LRU set
      o = B;
      if (atomicExch(&s_misc[2], 1) != 0) my_status |= HISPARSE_STATUS_DUPLICATE;
    } else if (got[i] >= 0) {
      // A plain byte store marks the slot (shared-memory atomics on a bitset were measured to take about half of
      // a resolve in which nothing misses).  The hit's stamp is written later, in slot order (coalesced), from
      // the marks; a resident position selected twice marks one slot twice, which the counts reveal.
      o = got[i];
      v.marks[o] = tag;
      ++nhit;
    } else if (p >= 0) {
      o = kMiss;
      miss = 1;
      // With the slice in shared memory, a missing position is claimed there by its row index: reading the claim
      // back after the vote tells whether another row entry selected the same position (any negative entry reads
      // as "not resident", so a claim does not disturb a later lookup of that position).
      if (use_staged) s_p2s[p] = (int16_t)(-2 - (j0 + i));
    }
    cls[i] = o;
    val[i] = o < 0 ? -1 : base + o;
  }
  // Phase 5, first part: the thread's entries of the slot table (and of the group's shared table), one vector store
  const bool vec = (((uintptr_t)trow | (uintptr_t)arow) & (KPT * 4 - 1)) == 0 && j0 + KPT <= k;
  if (vec) {
    if constexpr (KPT == 4) {
      *reinterpret_cast<int4 *>(trow + j0) = make_int4(val[0], val[1], val[2], val[3]);
      if (arow) *reinterpret_cast<int4 *>(arow + j0) = make_int4(cls[0] < 0 ? -1 : cls[0], cls[1] < 0 ? -1 : cls[1],
                                                                 cls[2] < 0 ? -1 : cls[2], cls[3] < 0 ? -1 : cls[3]);
    } else {
      *reinterpret_cast<int2 *>(trow + j0) = make_int2(val[0], val[1]);
      if (arow) *reinterpret_cast<int2 *>(arow + j0) = make_int2(cls[0] < 0 ? -1 : cls[0], cls[1] < 0 ? -1 : cls[1]);
    }
  } else {
#pragma unroll
    for (int i = 0; i < KPT; ++i)
      if (j0 + i < k) {
        trow[j0 + i] = val[i];
        if (arow) arow[j0 + i] = cls[i] < 0 ? -1 : cls[i];
      }
  }
  nhit = __reduce_add_sync(0xffffffffu, nhit);
  if ((tid & 31) == 0 && nhit) atomicAdd(&s_misc[1], nhit);
  any_miss = __syncthreads_or(miss) != 0;
  claims = use_staged ? kClaimsStored : kClaimsNone;
  if (timers && tid == 0) stamps[10] = clock64();
}

// The rest of what precedes the fetch when something missed: catch a missing position that was selected twice (it
// must claim one victim, not two), then ONE block-wide rank puts the misses in selection order.  On return
// plan_pos[i] / missj[i] hold the position and the row index of the i-th miss and m their number.
// Repeated positions are a violation of the caller's contract, so the common case is made cheap: every miss has
// claimed its position in the staged slice with its row index (a plain store); a claim that reads back as someone
// else's reveals a repetition, and only then (or when the slice is not in shared memory) do the missing positions go
// through the table (position -> lowest row index), which decides the owner the way the specification does.
template <int T, int KPT>
__device__ __forceinline__ void list_misses(const DevState &d, const SmemView &v, int32_t *trow, int32_t *arow,
                                            unsigned long long *stamps, int *s_misc, int16_t *s_p2s, const int claims,
                                            const int32_t (&pos)[KPT], int32_t (&cls)[KPT], uint32_t &my_status, int &m) {
  const int tid = threadIdx.x;
  const int H = d.H;
  const uint32_t mask = (uint32_t)(H - 1);
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  const int j0 = tid * KPT;
  bool need_table = true;
  if (claims != kClaimsNone) {
    if (claims == kClaimsPending) {
#pragma unroll
      for (int i = 0; i < KPT; ++i)
        if (cls[i] == kMiss) s_p2s[pos[i]] = (int16_t)(-2 - (j0 + i));
      __syncthreads();
    }
    int other = 0;
#pragma unroll
    for (int i = 0; i < KPT; ++i)
      if (cls[i] == kMiss) other |= s_p2s[pos[i]] != (int16_t)(-2 - (j0 + i));
    need_table = __syncthreads_or(other) != 0;  // (also: every claim has been read before the ring is used again)
  }
  if (need_table) {
    if (d.sm_tab < 0) {  // the table shares the ring's memory and is cleared only now that it is needed
      for (int i = tid; i < H; i += T) v.tab[i] = kEmptyEntry;
      __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < KPT; ++i)
      if (cls[i] == kMiss) {
        const int32_t p = pos[i];
        const unsigned long long entry = ((unsigned long long)(uint32_t)p << 32) | (uint32_t)(j0 + i);
        uint32_t h = hash_pos(p, d.hshift);
        for (uint32_t it = 0; it <= mask; ++it) {
          const unsigned long long old = atomicCAS(&v.tab[h], kEmptyEntry, entry);
          if (old == kEmptyEntry) break;
          if ((int32_t)(old >> 32) == p) {  // selected twice: the lowest row index owns the entry
            atomicMin(&v.tab[h], entry);
            s_misc[0] = 1;
            break;
          }
          h = (h + 1u) & mask;
        }
      }
    __syncthreads();
    if (s_misc[0]) {  // every later occurrence of a repeated missing position follows the first one
#pragma unroll
      for (int i = 0; i < KPT; ++i)
        if (cls[i] == kMiss) {
          const int32_t key[1] = {pos[i]};
          int32_t owner[1];
          table_lookup<1>(v.tab, mask, d.hshift, key, owner);
          if (owner[0] != j0 + i) {
            cls[i] = -1;  // not a miss of its own; its table entry is copied from the owner's at the end
            trow[j0 + i] = kDupBase - owner[0];
            if (arow) arow[j0 + i] = kDupBase - owner[0];
            my_status |= HISPARSE_STATUS_DUPLICATE;
          }
        }
    }
  }
  if (timers && tid == 0) stamps[11] = clock64();
  // Phase 3, first half: the misses in selection order.  Their positions are all the fetch needs to start loading;
  // the victims are only needed when a record is stored.
  uint32_t miss_mask = 0;
#pragma unroll
  for (int i = 0; i < KPT; ++i)
    if (cls[i] == kMiss) miss_mask |= 1u << i;
  int mrank = block_rank_bits<KPT>(miss_mask, v.warp, m);
#pragma unroll
  for (int i = 0; i < KPT; ++i)
    if ((miss_mask >> i) & 1u) {
      v.plan_pos[mrank] = pos[i];
      v.missj[mrank] = (uint16_t)(j0 + i);
      ++mrank;
    }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // the ring was written by this block's threads
  if (timers && tid == 0) stamps[12] = clock64();
  __syncthreads();
}

// Phase 3, second half (runs while the first loads are in flight): waits for the recency list (its load was issued
// right after the vote, into the memory the row had used), brings it up to date if it lags, then ONE block scan over
// the non-hit slots in recency order.  Thread t owns IPT consecutive entries of the list.  On return plan_slot[i] holds
// the victim of the i-th miss, vicbits the victims' marks, order the untouched slots compacted at its front and
// n_nonhit the number of slots without a hit.
template <int T, int IPT>
__device__ __forceinline__ void choose_victims(const DevState &d, const SmemView &v, const int r, const int64_t rg,
                                               const int m, unsigned long long *stamps, const uint32_t t_now,
                                               const uint32_t order_t, const bool order_bulk, const uint32_t order_parity,
                                               uint32_t &my_status, int &n_nonhit) {
  const int tid = threadIdx.x;
  const int B = d.B;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  int32_t *s_plan_slot = v.plan_slot;
  uint32_t *s_hitbits = v.hitbits, *s_vicbits = v.vicbits;
  uint16_t *s_order = v.order;
  int *s_warp_pre = v.vicpre;
  int *s_warp = v.warp;
  if (order_bulk) {  // one warp waits for the copy, the others for that warp (see lookup_phase)
    bool landed = true;
    if (tid < 32 && !mbar_wait_bounded(smem_u32(v.bars + T + 1), order_parity)) {
      mbar_wait_bounded(smem_u32(v.bars + T + 1), order_parity);
      landed = false;
    }
    if (__syncthreads_or(!landed)) my_status |= HISPARSE_STATUS_TIMEOUT;
  } else {
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();
  }
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
      select_random_victims<IPT>(B, m, base, t_now, s_hitbits, s_vicbits, v.hist, s_warp);
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

// Everything the first block of a cluster does for a request in which something missed (or whose recency list is kept
// current by every resolve): list the misses, start the fetch, choose the victims while the first loads fly, write the
// metadata back, rewrite the recency list, then drain the fetch.  pos / cls come from lookup_phase.
template <int T, int KPT>
__device__ __forceinline__ void miss_path(const DevState &d, const ReqCtx &c, const int claims, const int32_t (&pos)[KPT],
                                          int32_t (&cls)[KPT], const uint32_t t, const uint32_t order_t,
                                          uint32_t my_status, uint32_t &fetch_parity, uint32_t &order_parity,
                                          bool &gave_up) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SmemView v = smem_view(d, smem_raw, c.it);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int k = d.k, B = d.B, W = d.W, S = c.S, r = c.r;
  const int64_t rg = c.rg;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;
  unsigned long long *stamps = d.phase_ns + (int64_t)r * 16;
  int *s_misc = v.misc;
  int m = 0, n_nonhit = 0;
  int16_t *s_p2s = reinterpret_cast<int16_t *>(v.ring) + slice_geom(d, c.g, c.cap_r, c.p2s_off_r).lead;
  list_misses<T, KPT>(d, v, c.trow, c.arow, stamps, s_misc, s_p2s, claims, pos, cls, my_status, m);
  if (timers && tid == 0) { stamps[3] = global_ns(); stamps[7] = stamps[3]; }
  // Phase 4 starts here, with the positions of the misses: the first batch of host loads is in flight while the
  // victims are chosen (a record's slot is only needed when it is stored) and the metadata is written back
  TmaFetch fetch;
  fetch.init(d, r, c.layer, m, v.plan_pos, v.plan_slot, v.ring, v.bars, 0, S, fetch_parity);
  fetch.issue(d);
  // The recency list starts its way into the memory the row occupied (every thread consumed its row entries before
  // the vote); it is needed only once the first loads are in flight.
  const uint16_t *order_g = d.order + rg * B;
  const bool order_bulk = (((uintptr_t)order_g | (uintptr_t)(B * 2)) & 15) == 0;
  if (order_bulk) {
    if (tid == 0) {
      const uint32_t bar = smem_u32(v.bars + T + 1);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)B * 2u) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(v.order)), "l"(order_g), "r"((uint32_t)B * 2u), "r"(bar) : "memory");
    }
  } else {
    stage_async(v.order, order_g, B * 2);
  }
  // With the loads on their way: the victim marks cleared and the hit marks turned into a bitset, which the victim
  // choice and the list rewrite work on (every mark was written before the vote; the loop bound is uniform, so
  // every lane takes part in the ballot).  Both are ordered before their first use by choose_victims' barrier.
  // (Before the loads, this cost the fetch 1100 cycles of waiting.)
  for (int i = tid; i < W; i += T) v.vicbits[i] = 0u;
  for (int sb = 0; sb < B; sb += T) {
    const int s = sb + tid;
    const uint32_t word = __ballot_sync(0xffffffffu, s < B && v.marks[s] == (uint8_t)c.tag);
    if (lane == 0 && (s >> 5) < W) v.hitbits[s >> 5] = word;
  }
#define HS_VICT(IPT) choose_victims<T, IPT>(d, v, r, rg, m, stamps, t, order_t, order_bulk, order_parity, my_status, n_nonhit)
  if constexpr (T == kThreads) {
    if (B <= 4 * T) HS_VICT(4);
    else if (B <= 8 * T) HS_VICT(8);
    else HS_VICT(16);
  } else {
    if (B <= 8 * T) HS_VICT(8);
    else HS_VICT(16);
  }
#undef HS_VICT
  if (order_bulk) order_parity ^= 1u;
  // same state as right after the first issue, recomputed instead of kept in registers across the victim choice
  fetch.init(d, r, c.layer, m, v.plan_pos, v.plan_slot, v.ring, v.bars, 0, S, fetch_parity);
  fetch.active = fetch.active && fetch.piece_of(d, 0) < fetch.total;
  // Phase 5, metadata half: page table, slot array, stamps, plan, and the slot-table entries of the misses
  {
    int32_t *slot_pos = d.slot_pos + rg * B;
    uint32_t *last_use = d.last_use + rg * B;
    int16_t *p2s = d.pos2slot + c.p2s_off_r + (int64_t)c.g * p2s_stride(c.cap_r);
    int32_t *plan_pos_g = d.plan_pos + rg * k, *plan_slot_g = d.plan_slot + rg * k;
    const int32_t base = r * (B + 1);
    const uint32_t miss_stamp = 2u * t;
    for (int i = tid; i < m; i += T) {
      const int vs = v.plan_slot[i];
      const int32_t p = v.plan_pos[i];
      const int j = v.missj[i];
      const int32_t old = slot_pos[vs];
      if (old >= 0) p2s[old] = -1;
      slot_pos[vs] = p;
      p2s[p] = (int16_t)vs;
      last_use[vs] = miss_stamp;
      plan_pos_g[i] = p;
      plan_slot_g[i] = vs;
      c.trow[j] = base + vs;
      if (c.arow) c.arow[j] = vs;
    }
    if (tid == 0) d.plan_n[rg] = m;
  }
  if (my_status) atomicOr(d.status, my_status);
  if (my_status & HISPARSE_STATUS_TIMEOUT) gave_up = true;
  // The plan is public: the other blocks of the cluster start fetching while this one publishes.  Every thread
  // arrives with release semantics after its own plan writes and every reader waits with acquire semantics, which
  // orders them at cluster scope: no separate fence.
  if (S > 1) cluster_arrive();
  {
    uint16_t *order = d.order + rg * B;
    uint32_t *s_hitbits = v.hitbits, *s_vicbits = v.vicbits;
    int32_t *s_hitpre = v.hitpre, *s_vicpre = v.vicpre;
    uint16_t *s_order = v.order;
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
    __syncthreads();
    if (s_misc[0]) {
      // rare: a row entry that repeats a missing position takes the table entry of its first occurrence, which this
      // block wrote above (block-scope ordering through the barrier)
      for (int j = tid; j < k; j += T) {
        const int32_t o = c.trow[j];
        if (o <= kDupBase) {
          c.trow[j] = c.trow[kDupBase - o];
          if (c.arow) c.arow[j] = c.arow[kDupBase - o];
        }
      }
    }
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
    for (int qq = tid; qq < B; qq += T) order[qq] = s_order[qq];
    if (tid == 0) {
      // distinct hits = slots whose hit bit is set (+ the reserved slot if the newest position was selected); more
      // selections that hit than slots hit = a resident position was selected twice
      const int nhits = (B - n_nonhit) + (s_misc[2] ? 1 : 0);
      if (s_misc[1] != B - n_nonhit) atomicOr(d.status, HISPARSE_STATUS_DUPLICATE);
      s_misc[0] = s_misc[1] = s_misc[2] = s_misc[3] = 0;  // this set serves the request after the next
      c.hits_out[r] = nhits;
      c.misses_out[r] = m;
      d.anchor_hits[rg] = nhits;
      d.anchor_misses[rg] = m;
      d.t[rg] = t;
      if (d.order_t) d.order_t[rg] = t;
    }
    if (timers && tid == 0) stamps[4] = global_ns();
  }
  if (S > 1) cluster_wait();
  // Phase 4, rest: wait for the batches, store them into the cache slots, issue what is left.  Whatever follows
  // in the stream may be scheduled from here on (it still waits for this grid to finish before it reads).
  if (!c.has_next) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!fetch.drain(d, d.status)) gave_up = true;
  fetch_parity = fetch.parity;
  if (timers) {
    __syncthreads();
    if (tid == 0) {
      const unsigned long long now = global_ns();
      stamps[5] = now;
      atomicMax(&stamps[6], now);
      atomicMax(d.layer_ns + d.L + c.layer, now);
    }
  }
}

// The same, kept out of line for blocks that loop over requests: the loop's short path (nothing missed) then keeps
// its few registers, and only a request with misses pays for the call.  The thread's row entries and their
// classification travel through shared memory (the victim array is idle until the victims are chosen).
template <int T, int KPT>
__device__ __noinline__ void miss_path_cold(const DevState &d, const ReqCtx &c, const uint32_t t, const uint32_t order_t,
                                            const uint32_t my_status, uint32_t &fetch_parity, uint32_t &order_parity,
                                            bool &gave_up) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  static_assert(KPT == 4, "the stash holds one position per row entry");
  int32_t pos[KPT], cls[KPT];
  int4 x = make_int4(-1, -1, -1, -1);
  if ((int)threadIdx.x * KPT < d.k) x = reinterpret_cast<const int4 *>(smem_raw + d.sm_plan_slot)[threadIdx.x];
  pos[0] = x.x; pos[1] = x.y; pos[2] = x.z; pos[3] = x.w;
#pragma unroll
  for (int i = 0; i < KPT; ++i) cls[i] = pos[i] >= 0 ? kMiss : -1;  // only the misses matter from here on
  // (the array gets its real content only after several block barriers: every thread has its entries by then)
  const int claims = slice_geom(d, c.g, c.cap_r, c.p2s_off_r).staged ? kClaimsPending : kClaimsNone;
  miss_path<T, KPT>(d, c, claims, pos, cls, t, order_t, my_status, fetch_parity, order_parity, gave_up);
}

// A block of a cluster other than the first: shares the page-table lookups when the slice cannot be staged, then
// takes its share of the recorded plan through the fetch pipeline.
template <int T>
__device__ __forceinline__ void helper_block(const DevState &d, const ReqCtx &c, const int part, uint32_t &fetch_parity,
                                             bool &gave_up) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SmemView v = smem_view(d, smem_raw, 0);
  const int tid = threadIdx.x, k = d.k;
  const SliceGeom q = slice_geom(d, c.g, c.cap_r, c.p2s_off_r);
  if (!q.staged) {  // the request's page-table slice is too large to be staged: the cluster shares the lookups
    const int64_t na = *(volatile int32_t *)d.n_appends;
    const int64_t len = c.init_len_r + na < c.cap_r ? c.init_len_r + na : c.cap_r;
    cluster_arrive_relaxed();  // phase A
    cluster_lookups<T>(c.row, q.p2s, k, len, part, c.S, v.got);
  }
  cluster_arrive();
  cluster_wait();
  const int m = __ldcg(d.plan_n + c.rg);
  const int32_t *pp = d.plan_pos + c.rg * k, *ps = d.plan_slot + c.rg * k;
  for (int i = tid; i < m; i += T) { v.plan_pos[i] = __ldcg(pp + i); v.plan_slot[i] = __ldcg(ps + i); }
  __syncthreads();
  TmaFetch fetch;
  fetch.init(d, c.r, c.layer, m, v.plan_pos, v.plan_slot, v.ring, v.bars, part, c.S, fetch_parity);
  fetch.issue(d);
  if (!fetch.drain(d, d.status)) gave_up = true;
  fetch_parity = fetch.parity;
  if (d.flags & HISPARSE_FLAG_PHASE_TIMERS) {
    __syncthreads();
    if (tid == 0) {
      const unsigned long long now = global_ns();
      atomicMax(&d.phase_ns[(int64_t)c.r * 16 + 6], now);
      atomicMax(d.layer_ns + d.L + c.layer, now);
    }
  }
}

// The loop of a resident wave of narrow blocks, written out for the shape it is meant for: every request has the
// same capacity, the rows / table rows / page-table slices are 16-byte aligned whole units, the slice fits the ring.
// Same steps and same results as the general code below (lookup_phase + the short path of resolve_kernel), with
// everything that does not depend on the request hoisted out of the loop, 32-bit lengths, and no per-request geometry
// structs: the general code spends ~840 instructions per thread and request, which made a resolve in which nothing
// misses issue-bound; this loop spends about a fifth of that.  The first request with a miss ends the loop: the general
// loop takes that request, and the block's later ones, from there (see lean_loop).
__device__ __forceinline__ bool lean_shape(const DevState &d, const int32_t *sel, const int32_t *table, const int threads) {
  return !(d.flags & HISPARSE_FLAG_PHASE_TIMERS) && d.uni_cap >= 0 && d.order_t != nullptr &&
         (((uintptr_t)sel | (uintptr_t)table | (uintptr_t)d.pos2slot | (uintptr_t)d.anchor_out) & 15) == 0 &&
         (d.k & 3) == 0 && d.k <= 4 * threads && p2s_stride(d.uni_cap) * 2 + 16 <= (int64_t)d.ring_bytes;
}

template <int T>
__device__ __forceinline__ void lean_stage_issue(const DevState &d, const int32_t *sel, const int g, const int r,
                                                 const uint32_t s_sel_addr, const uint32_t ring_addr, const uint32_t stage_bar) {
  const uint32_t lane = threadIdx.x;  // called by the first warp only
  const uint32_t row_bytes = (uint32_t)d.k * 4u;
  const uint32_t slice_bytes = (uint32_t)p2s_stride(d.uni_cap) * 2u;  // whole 16-byte units (the padding is -1)
  if (lane == 0)
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(stage_bar), "r"(row_bytes + slice_bytes) : "memory");
  const char *row = reinterpret_cast<const char *>(sel + (int64_t)r * d.k);
  const char *slice = reinterpret_cast<const char *>(d.pos2slot + ((int64_t)r * d.G + g) * p2s_stride(d.uni_cap));
  const uint32_t row_pieces = (row_bytes + kStagePiece - 1) / kStagePiece, slice_pieces = (slice_bytes + kStagePiece - 1) / kStagePiece;
  for (uint32_t p = lane; p < row_pieces + slice_pieces; p += 32u) {  // small pieces, side by side: see stage_issue
    const bool in_row = p < row_pieces;
    const uint32_t o = (in_row ? p : p - row_pieces) * kStagePiece, total = in_row ? row_bytes : slice_bytes;
    const uint32_t n = total - o < kStagePiece ? total - o : kStagePiece;
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"((in_row ? s_sel_addr : ring_addr) + o), "l"((in_row ? row : slice) + o), "r"(n), "r"(stage_bar) : "memory");
  }
}

// Shared-memory accesses of the lean loop by 32-bit shared address (no generic-address arithmetic).
__device__ __forceinline__ int4 lds_v4(uint32_t a) {
  int4 v;
  asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ int32_t lds_s16(uint32_t a) {
  int32_t v;
  asm volatile("ld.shared.s16 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds_u8(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void sts_u8(uint32_t a, uint32_t v) { asm volatile("st.shared.u8 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ int32_t lds_s32(uint32_t a) {
  int32_t v;
  asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void sts_s32(uint32_t a, int32_t v) { asm volatile("st.shared.s32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void red_add_s32(uint32_t a, int32_t v) { asm volatile("red.shared.add.s32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ int32_t atom_add_s32(uint32_t a, int32_t v) {
  int32_t o;
  asm volatile("atom.shared.add.s32 %0, [%1], %2;" : "=r"(o) : "r"(a), "r"(v) : "memory");
  return o;
}

// Returns -1 when the block has nothing left to do; otherwise the number of requests it has finished, with `r` the
// request in which something missed: that request's row and slice are still staged (its barrier's phase is over), its
// marks are written and its counters cleared, and the caller's general loop takes it from the lookups on.  (Calling the
// out-of-line miss path from inside this loop made the compiler keep the loop's state in local memory around the call
// site: ~17 spill instructions per warp and request on a path that never made the call; as a function of its own,
// out of line, the loop spilled even more.)
template <int T>
__device__ __forceinline__ int lean_loop(const DevState &d, const int g, const int32_t *__restrict__ sel,
                                         int32_t *__restrict__ table, int32_t *__restrict__ hits_out,
                                         int32_t *__restrict__ misses_out, int &r, const int stride) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31;
  const int k = d.k, B = d.B, N = d.N;
  const uint32_t a_base = smem_u32(smem_raw);
  const uint32_t a_ring = a_base + (uint32_t)(d.meta_smem + d.bar_bytes);   // the staged page-table slice
  const uint32_t a_marks = a_base + (uint32_t)d.sm_marks;
  const uint32_t a_spare = a_marks + (uint32_t)d.marks_spare;                // a byte that no slot owns
  const uint32_t a_misc = a_base + (uint32_t)d.sm_misc + 128u;              // two sets of 8 ints
  const uint32_t stage_bar = a_base + (uint32_t)d.meta_smem + (uint32_t)T * 8u;
  const uint32_t a_row = a_base + (uint32_t)tid * 16u;                      // this thread's four row entries
  const int cap = (int)d.uni_cap, il = (int)d.uni_init_len;
  const bool mine = tid * 4 < k;
  const bool stamp_hits = d.policy != HISPARSE_POLICY_FIFO;
  const int G = d.G;
  int tag = 0, it = 0;
  // The counters of a request are read, reported and cleared by the first thread one request later, behind the block
  // barrier that follows the staging wait (the two sets of counters alternate): that saves the barrier the counts
  // would otherwise need right after the stamp pass, one of three per request.
  int r_prev = -1;
  uint32_t t_prev = 0, set_prev = 0;
  auto finish = [&](const int rf, const uint32_t tf, const uint32_t set) {   // first thread only
    const int rgf = rf * G + g;
    const int distinct = lds_s32(set + 12u), selected = lds_s32(set + 4u), isnew = lds_s32(set + 8u);
    if (distinct != selected) atomicOr(d.status, HISPARSE_STATUS_DUPLICATE);  // a resident position was selected twice
    const int nhits = distinct + (isnew ? 1 : 0);
    sts_s32(set, 0); sts_s32(set + 4u, 0); sts_s32(set + 8u, 0); sts_s32(set + 12u, 0);  // for the request after the next
    hits_out[rf] = nhits;
    misses_out[rf] = 0;
    d.anchor_hits[rgf] = nhits;
    d.anchor_misses[rgf] = 0;
    d.plan_n[rgf] = 0;
    d.t[rgf] = tf;
    if (!stamp_hits) d.order_t[rgf] = tf;
  };
  // a request's resolve count is loaded one request ahead (with the next request's inputs), so that the trip to
  // memory is over when the count is needed
  uint32_t t_ahead = r < N ? d.t[r * G + g] : 0u;
  // nothing appends while a resolve runs (stream order): the lengths are the same for every request of the launch
  const int na = *(volatile int32_t *)d.n_appends;
  int len = il + na, newest = na > 0 ? il + na - 1 : -2;  // -2: no newest record (a discarded entry is -1)
  if (len > cap) { len = cap; newest = -2; }
  bool more = r < N;
  for (; more; ++it) {
    const int rg = r * G + g;                       // N * G fits 32 bits (the metadata arrays are indexed by it)
    const uint32_t parity = (uint32_t)it & 1u;
    const uint32_t a_set = a_misc + parity * 32u;
    if (tag == 255) {
      // the tags start over: forget the old marks, once every thread is done with the previous request's
      tag = 0;
      __syncthreads();
      for (int i = tid * 16; i < B; i += T * 16) *reinterpret_cast<uint4 *>(smem_raw + d.sm_marks + i) = make_uint4(0, 0, 0, 0);
      __syncthreads();
    }
    ++tag;
    const uint32_t t = t_ahead + 1u;
    if (tid >= T - 2 && r + 2 * stride < N) {
      // the request after the next: its row and slice start their way from HBM to L2 now, two requests ahead of
      // their use (the staging copy of one request ahead then reads L2)
      const int r2 = r + 2 * stride;
      const bool is_row = tid == T - 2;
      const char *p = is_row ? reinterpret_cast<const char *>(sel + (int64_t)r2 * k)
                             : reinterpret_cast<const char *>(d.pos2slot + ((int64_t)r2 * G + g) * p2s_stride(cap));
      const uint32_t n = is_row ? (uint32_t)k * 4u : (uint32_t)p2s_stride(cap) * 2u;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(n) : "memory");
    }
    bool landed = true;
    if (tid < 32 && !mbar_wait_bounded(stage_bar, parity)) {
      mbar_wait_bounded(stage_bar, parity);
      landed = false;
    }
    uint32_t st = 0;
    bool gave_up = false;
    if (__syncthreads_or(!landed)) { st = HISPARSE_STATUS_TIMEOUT; gave_up = true; }
    if (tid == 0 && r_prev >= 0) finish(r_prev, t_prev, set_prev);   // (its stamp pass is over)
    int4 x = make_int4(-1, -1, -1, -1);
    if (mine && !gave_up) x = lds_v4(a_row);
    int32_t pos[4] = {x.x, x.y, x.z, x.w};
    int32_t got[4];
    int bad = 0;
    // every access below is unconditional (an entry that is padding or out of range looks up position 0 and discards
    // the answer; an entry that did not hit marks a spare byte): branches around them cost more than they save
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bool ok = (uint32_t)pos[i] < (uint32_t)len;  // 0 <= p < len
      bad |= (!ok) & (pos[i] != -1);
      const int32_t g16 = lds_s16(a_ring + 2u * (uint32_t)(ok ? pos[i] : 0));
      pos[i] = ok ? pos[i] : -1;
      got[i] = ok ? g16 : -1;
    }
    if (bad) st |= HISPARSE_STATUS_OUT_OF_RANGE;
    const int32_t base = r * (B + 1);
    int nhit = 0, nnew = 0;
    bool miss = false;
    int32_t val[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const bool isnew = pos[i] == newest, hit = got[i] >= 0 && !isnew;
      miss |= pos[i] >= 0 && !isnew && !hit;
      sts_u8(hit ? a_marks + (uint32_t)got[i] : a_spare, (uint32_t)tag);
      nhit += hit;
      nnew += isnew;
      val[i] = hit ? base + got[i] : (isnew ? base + B : -1);
    }
    if (nnew) {  // the reserved newest-record slot, outside the LRU set; selected twice = a repeated position
      if (atom_add_s32(a_set + 8u, nnew) + nnew > 1) st |= HISPARSE_STATUS_DUPLICATE;
    }
    if (mine) {
      *reinterpret_cast<int4 *>(table + (int64_t)r * k + tid * 4) = make_int4(val[0], val[1], val[2], val[3]);
      if (d.lpg > 1)
        *reinterpret_cast<int4 *>(d.anchor_out + (int64_t)rg * k + tid * 4) =
            make_int4(val[0] < 0 ? -1 : val[0] - base, val[1] < 0 ? -1 : val[1] - base, val[2] < 0 ? -1 : val[2] - base,
                      val[3] < 0 ? -1 : val[3] - base);
    }
    nhit = __reduce_add_sync(0xffffffffu, nhit);
    if (lane == 0 && nhit) red_add_s32(a_set + 4u, nhit);
    const bool any_miss = __syncthreads_or(miss) != 0;
    const int rn = r + stride;        // the request this block takes next
    const bool has_next = rn < N;
    if (has_next) t_ahead = d.t[rn * G + g];
    if (any_miss) {
      // something missed: the general loop takes this request again from its lookups on (the staged row and slice are
      // untouched, the marks carry this request's tag either way); what this pass counted is forgotten
      if (tid == 0) { sts_s32(a_set, 0); sts_s32(a_set + 4u, 0); sts_s32(a_set + 8u, 0); sts_s32(a_set + 12u, 0); }
      return it;
    }
    if (has_next && !gave_up) {
      // the row and the ring are free (every thread consumed its entries before the vote): the next request's inputs
      // travel while this one's stamps are written
      if (tid < 32) lean_stage_issue<T>(d, sel, g, rn, a_base, a_ring, stage_bar);
    } else {
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    {
      uint32_t *lu = d.last_use + (int64_t)rg * B + tid;
      const uint32_t hit_stamp = 2u * t + 1u;
      const uint32_t a_m = a_marks + (uint32_t)tid;
      int cnt = 0;
      if (stamp_hits) {
        // four slots per round, written out in PTX: four loads, four compares, four predicated stores, the count
        // (the marks are padded to whole rounds of this loop, padding = 0)
        for (int s0 = 0; s0 < B; s0 += 4 * T) {
          uint32_t c4;
          asm volatile(
              "{\n"
              ".reg .pred p0, p1, p2, p3;\n"
              ".reg .u32 m0, m1, m2, m3, c0, c1, c2, c3;\n"
              "ld.shared.u8 m0, [%1];\n"
              "ld.shared.u8 m1, [%1+%5];\n"
              "ld.shared.u8 m2, [%1+%6];\n"
              "ld.shared.u8 m3, [%1+%7];\n"
              "setp.eq.u32 p0, m0, %2;\n"
              "setp.eq.u32 p1, m1, %2;\n"
              "setp.eq.u32 p2, m2, %2;\n"
              "setp.eq.u32 p3, m3, %2;\n"
              "@p0 st.global.u32 [%3], %4;\n"
              "@p1 st.global.u32 [%3+%8], %4;\n"
              "@p2 st.global.u32 [%3+%9], %4;\n"
              "@p3 st.global.u32 [%3+%10], %4;\n"
              "selp.u32 c0, 1, 0, p0;\n"
              "selp.u32 c1, 1, 0, p1;\n"
              "selp.u32 c2, 1, 0, p2;\n"
              "selp.u32 c3, 1, 0, p3;\n"
              "add.u32 c0, c0, c1;\n"
              "add.u32 c2, c2, c3;\n"
              "add.u32 %0, c0, c2;\n"
              "}"
              : "=r"(c4)
              : "r"(a_m + (uint32_t)s0), "r"((uint32_t)tag), "l"(lu + s0), "r"(hit_stamp), "n"(T), "n"(2 * T), "n"(3 * T),
                "n"(4 * T), "n"(8 * T), "n"(12 * T)
              : "memory");
          cnt += (int)c4;
        }
      } else {   // FIFO: a hit changes no stamp; only the distinct slots are counted
        for (int s0 = 0; s0 < B; s0 += T) cnt += lds_u8(a_m + (uint32_t)s0) == (uint32_t)tag;
      }
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (lane == 0 && cnt) red_add_s32(a_set + 12u, cnt);
    }
    if (st) atomicOr(d.status, st);
    r_prev = r;
    t_prev = t;
    set_prev = a_set;
    if (gave_up) break;
    more = has_next;
    r = rn;
  }
  if (r_prev >= 0) {   // the block's last request
    __syncthreads();
    if (tid == 0) finish(r_prev, t_prev, set_prev);
  }
  return -1;
}

// MINB = thread blocks of this size that must fit one SM (bounds the registers per thread).
// Grid: one cluster of S blocks per request, or fewer clusters than requests, in which case a cluster takes the
// requests c, c + clusters, c + 2 clusters, .. one after the other (LOOP, only with S = 1: a grid of several waves is
// launched as one resident wave of looping blocks, so that no block pays for another launch and the next request's
// row and page-table slice are already on their way while the current one is finished).
template <int T, int MINB, bool LOOP>
__global__ void __launch_bounds__(T, MINB)
resolve_kernel(const __grid_constant__ DevState d, const int layer, const int32_t *__restrict__ sel,
               int32_t *__restrict__ table, int32_t *__restrict__ hits_out, int32_t *__restrict__ misses_out, const int S) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int tid = threadIdx.x, lane = tid & 31;
  const int part = blockIdx.x % S, stride = gridDim.x / S;
  const int g = layer / d.lpg;
  const int k = d.k, B = d.B;
  const bool timers = d.flags & HISPARSE_FLAG_PHASE_TIMERS;

  // Prologue that depends on nothing an earlier kernel wrote: barriers, cleared marks (and table, when it has memory
  // of its own), the addresses of everything Phase 1 will load.  With programmatic dependent launch it overlaps the
  // tail of whatever runs before this kernel in the stream.
  int r = blockIdx.x / S;
  {
    const SmemView v = smem_view(d, smem_raw, 0);
    fetch_barriers_init(v.bars, d.io_threads);
    if (part == 0) {
      if (d.sm_tab >= 0)
        for (int i = tid; i < d.H; i += T) v.tab[i] = kEmptyEntry;
      for (int i = tid * 16; i < d.marks_spare + 16; i += T * 16) *reinterpret_cast<uint4 *>(v.marks + i) = make_uint4(0, 0, 0, 0);
      if (tid < 16) v.misc[tid] = 0;
      if (tid < 2) {
        // Warm L2 with what Phase 1 will stage (row, page-table slice).  A prefetch consumes nothing, and L2 is where
        // earlier kernels' writes land, so this is safe before the dependency wait; when the previous kernel lets its
        // dependents start early, the staging after the wait then reads L2 instead of HBM.
        int64_t cap_r, init_len_r, p2s_off_r;
        request_geom(d, r, cap_r, init_len_r, p2s_off_r);
        const SliceGeom q = slice_geom(d, g, cap_r, p2s_off_r);
        const char *p = tid == 0 ? reinterpret_cast<const char *>(sel + (int64_t)r * k) : reinterpret_cast<const char *>(q.p2s);
        int64_t n = tid == 0 ? (int64_t)k * 4 : cap_r * 2;
        const uintptr_t a = ((uintptr_t)p + 15) & ~(uintptr_t)15;   // whole 16-byte units inside the array only
        n = (n - (int64_t)(a - (uintptr_t)p)) & ~(int64_t)15;
        if (n > (1 << 20)) n = 1 << 20;                             // no point warming more than the ring could stage
        if (n > 0 && (tid == 0 || q.staged))
          asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a), "r"((uint32_t)n) : "memory");
      }
    }
    __syncthreads();  // the barriers are initialised and the marks cleared before anything uses them
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (part != 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!LOOP && part == 0 && tid == 96 && r < d.N) {
      // A request whose previous resolve on this group missed nothing will most likely miss nothing now: whatever
      // follows in the stream may be scheduled at once, so that its launch latency and prologue run under this
      // whole kernel instead of under its last third (a resolve that does fetch releases its dependents only once
      // its loads are in flight: earlier costs the fetch ~2 us, which a wrong guess here pays once).  One thread of a
      // warp that takes no part in the staging reads the flag, so nothing waits for the load.
      if (__ldcg(d.anchor_misses + (int64_t)r * d.G + g) == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    if (part == 0) {
      int64_t cap_r, init_len_r, p2s_off_r;
      request_geom(d, r, cap_r, init_len_r, p2s_off_r);
      stage_issue<T>(d, v, slice_geom(d, g, cap_r, p2s_off_r), sel + (int64_t)r * k, cap_r, smem_u32(v.bars + T));
    }
  }
  uint32_t fetch_parity = 0, order_parity = 0;  // phases of this thread's fetch barrier / of the list's staging barrier
  bool gave_up = false;                          // a bounded wait expired: the block takes no further request

  int it = 0;
  if constexpr (LOOP) {
    if (S == 1 && lean_shape(d, sel, table, T)) {
      it = lean_loop<T>(d, g, sel, table, hits_out, misses_out, r, stride);
      if (it < 0) return;
    }
  }
  // (the wide block never loops: one pass, so that nothing has to stay in registers across requests)
  for (; r < d.N && !gave_up && (LOOP || it == 0); r += stride, ++it) {
    ReqCtx c;
    c.r = r; c.it = it; c.S = S; c.layer = layer; c.g = g;
    c.rg = (int64_t)r * d.G + g;
    request_geom(d, r, c.cap_r, c.init_len_r, c.p2s_off_r);
    c.row = sel + (int64_t)r * k;
    c.trow = table + (int64_t)r * k;
    c.arow = d.lpg > 1 ? d.anchor_out + c.rg * k : nullptr;
    c.hits_out = hits_out; c.misses_out = misses_out;
    c.has_next = LOOP && r + stride < d.N;
    if (part != 0) {
      helper_block<T>(d, c, part, fetch_parity, gave_up);
      continue;
    }
    const SmemView v = smem_view(d, smem_raw, it);
    const SliceGeom q = slice_geom(d, g, c.cap_r, c.p2s_off_r);
    unsigned long long *stamps = d.phase_ns + (int64_t)r * 16;
    if (timers && tid == 0) {
      stamps[0] = global_ns(); stamps[6] = 0ull; stamps[15] = clock64();
      atomicMin(d.layer_ns + layer, stamps[0]);
    }
    c.tag = it % 255 + 1;
    if (LOOP && it > 0 && c.tag == 1) {
      // the tags start over: forget the old marks (every thread is done with the previous request's)
      for (int i = tid * 16; i < B; i += T * 16) *reinterpret_cast<uint4 *>(v.marks + i) = make_uint4(0, 0, 0, 0);
      __syncthreads();
    }
    uint32_t my_status = 0, order_t = 0, t = 0;
    bool any_miss = false;
    int claims = kClaimsNone;
    // row entries per thread: k <= 4 * T by construction (create refuses other shapes for this block size)
    constexpr int KPT = 4;
    int32_t pos[KPT], cls[KPT];
    if (!LOOP && k <= 2 * T) {
      int32_t pos2[2], cls2[2];
      lookup_phase<T, 2>(d, v, q, c, (uint32_t)(it & 1), stamps, pos2, cls2, my_status, any_miss, t, order_t, claims);
      if (any_miss || d.order_t == nullptr) {
        miss_path<T, 2>(d, c, claims, pos2, cls2, t, order_t, my_status, fetch_parity, order_parity, gave_up);
        continue;
      }
    } else {
      lookup_phase<T, KPT>(d, v, q, c, (uint32_t)(it & 1), stamps, pos, cls, my_status, any_miss, t, order_t, claims);
      if (any_miss || d.order_t == nullptr) {
        if (LOOP) {
          // stash the thread's missing positions for the out-of-line path
          if (tid * KPT < k)
            reinterpret_cast<int4 *>(v.plan_slot)[tid] = make_int4(cls[0] == kMiss ? pos[0] : -1, cls[1] == kMiss ? pos[1] : -1,
                                                                  cls[2] == kMiss ? pos[2] : -1, cls[3] == kMiss ? pos[3] : -1);
          const ReqCtx cc = c;  // the copy that lives in memory for the call; `c` itself stays in registers
          miss_path_cold<T, KPT>(d, cc, t, order_t, my_status, fetch_parity, order_parity, gave_up);
          if (c.has_next) {
            // after a fetch, the next request's inputs can only start once every thread is done with the ring
            gave_up = __syncthreads_or(gave_up) != 0;
            if (!gave_up) {
              const int rn = r + stride;
              int64_t cap_n, il_n, off_n;
              request_geom(d, rn, cap_n, il_n, off_n);
              stage_issue<T>(d, v, slice_geom(d, g, cap_n, off_n), sel + (int64_t)rn * k, cap_n, smem_u32(v.bars + T));
            }
          }
        } else {
          miss_path<T, KPT>(d, c, claims, pos, cls, t, order_t, my_status, fetch_parity, order_parity, gave_up);
        }
        continue;
      }
    }
    // Short path.  Every valid selection is resident (or the newest record): nothing to fetch, no victim to choose.
    // The slot table is written; what is left are the hit stamps, in slot order (coalesced), and the counters.  The
    // recency list is not touched and order_t stays behind (rebuild_order brings it up to date in the next resolve
    // that needs victims); under FIFO a hit changes nothing, so the list stays current.
    if (my_status & HISPARSE_STATUS_TIMEOUT) gave_up = true;
    if (c.has_next && !gave_up) {
      // the row and the ring are free (every thread consumed its entries before the vote): the next request's
      // inputs travel while this one's stamps are written
      const int rn = r + stride;
      int64_t cap_n, il_n, off_n;
      request_geom(d, rn, cap_n, il_n, off_n);
      stage_issue<T>(d, v, slice_geom(d, g, cap_n, off_n), sel + (int64_t)rn * k, cap_n, smem_u32(v.bars + T));
    } else {
      // let whatever follows in the stream start its prologue now (measured: with a fetch ahead, releasing the
      // dependents before the first loads are issued costs the fetch about 2 us, so that path releases them only
      // once its metadata is written back)
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    if (timers && tid == 0) { stamps[3] = global_ns(); stamps[7] = stamps[3]; }
    {
      uint32_t *last_use = d.last_use + c.rg * B;
      const uint32_t hit_stamp = 2u * t + 1u;
      const bool stamp = d.policy != HISPARSE_POLICY_FIFO;
      const uint8_t tag = (uint8_t)c.tag;
      int cnt = 0;
      for (int s = tid; s < B; s += T)
        if (v.marks[s] == tag) {
          if (stamp) last_use[s] = hit_stamp;
          ++cnt;
        }
      cnt = __reduce_add_sync(0xffffffffu, cnt);
      if (lane == 0 && cnt) atomicAdd(&v.misc[3], cnt);
    }
    // the counts are complete, and the marks may be written again (a looping block's next request)
    __syncthreads();
    if (tid == 0) {
      const int distinct = v.misc[3];
      if (distinct != v.misc[1]) my_status |= HISPARSE_STATUS_DUPLICATE;  // a resident position was selected twice
      const int nhits = distinct + (v.misc[2] ? 1 : 0);
      v.misc[0] = v.misc[1] = v.misc[2] = v.misc[3] = 0;  // this set serves the request after the next
      hits_out[r] = nhits;
      misses_out[r] = 0;
      d.anchor_hits[c.rg] = nhits;
      d.anchor_misses[c.rg] = 0;
      d.plan_n[c.rg] = 0;
      d.t[c.rg] = t;
      if (d.policy == HISPARSE_POLICY_FIFO) d.order_t[c.rg] = t;
      if (timers) { stamps[4] = global_ns(); atomicMax(d.layer_ns + d.L + layer, stamps[4]); }
    }
    if (my_status) atomicOr(d.status, my_status);
    if (S > 1) {  // the other blocks of the cluster find an empty plan
      cluster_arrive();
      cluster_wait();
    }
  }
}

}  // namespace
