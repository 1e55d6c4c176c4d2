// Included by hisparse.cu: plan replay (Sec. 3.5), append and write-through (Sec. 3.3 step 4), the consumer
// stand-ins, the validation and self-test kernels and the copy-only probe.

namespace {

// ------------------------------------------------------------------------------------------ plan replay (Sec. 3.5)

// Copy-only kernel: replays the anchor's miss plan into a shared layer's cache.  grid = N * S blocks.
__global__ void __launch_bounds__(kThreads, 1) replay_kernel(const DevState d, const int layer, const int S) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  int32_t *s_plan_pos = reinterpret_cast<int32_t *>(smem_raw);
  int32_t *s_plan_slot = s_plan_pos + d.k;
  unsigned long long *s_bars = reinterpret_cast<unsigned long long *>(smem_raw + d.meta_smem);
  unsigned char *s_ring = smem_raw + d.meta_smem + d.bar_bytes;
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
  const int16_t *p2s = d.pos2slot + d.p2s_off[r] + (int64_t)g * p2s_stride(d.cap[r]);
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
