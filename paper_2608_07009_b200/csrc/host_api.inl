// Included by hisparse.cu: host-side handle and the C-ABI entry points declared in hisparse.h.

// ------------------------------------------------------------------------------------------ host state

struct hisparse {
  DevState d{};
  int device = 0;
  int S = 1, T = kThreads, minb = 1;   // blocks per request, threads per block, blocks of that size per SM
  int clusters = 1;                    // clusters in a resolve launch: N, or one resident wave that loops over the requests
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

// Lays out the dynamic shared memory of the resolve / replay kernels for blocks of `threads` threads.  `coop` =
// the blocks of a cluster may share the page-table lookups (needs the answers array); `tab_in_ring` = the table of
// missing positions shares the ring's memory instead of having its own.
void layout_smem(DevState &d, int threads, bool coop, bool tab_in_ring) {
  auto pad = [](size_t x) { return (x + 15) & ~(size_t)15; };
  const size_t k = (size_t)d.k, B = (size_t)d.B, wpad = ((size_t)d.W + 3) & ~(size_t)3;
  size_t o = std::max(pad(k * 4), pad(B * 2));   // the row, later the recency list
  d.sm_plan_pos = (int)o;  o += pad(k * 4);
  d.sm_plan_slot = (int)o; o += pad(k * 4);
  d.sm_missj = (int)o;     o += pad(k * 2);
  d.sm_marks = (int)o;     d.marks_spare = (int)((B + 2047) & ~(size_t)2047); o += (size_t)d.marks_spare + 16;
  d.sm_bits = (int)o;      o += 4 * wpad * 4;   // hit and victim bitsets, two prefix arrays
  d.sm_hist = (int)o;      o += 1040;
  d.sm_misc = (int)o;      o += 256;
  d.sm_got = coop ? (int)o : 0; o += coop ? pad(k * 2) : 0;
  d.sm_tab = tab_in_ring ? -1 : (int)o; o += tab_in_ring ? 0 : (size_t)d.H * 8;
  d.meta_smem = (int)((o + 127) & ~(size_t)127);
  d.bar_bytes = (threads + 2) * 8;
}

// Geometry of the fetch pipeline for `ring_room` bytes of staging ring.  False when not even one piece fits (or, with
// the table inside the ring, when the ring cannot hold it).
bool layout_ring(DevState &d, int threads, int64_t ring_room) {
  if (ring_room < 16) return false;
  d.io_chunk = (int)std::min<int64_t>(std::min<int64_t>(d.E, 8192), ring_room & ~(int64_t)15);
  const int slots = (int)(ring_room / d.io_chunk);
  d.io_threads = std::min(slots, threads);
  d.io_depth = std::min(slots / d.io_threads, 8);
  d.ring_bytes = d.io_threads * d.io_depth * d.io_chunk;
  d.io_ppr = (int)((d.E + d.io_chunk - 1) / d.io_chunk);
  if (d.sm_tab < 0 && (int64_t)d.H * 8 > ring_room) return false;
  return true;
}

size_t kernel_smem_bytes(const DevState &d) {
  // with the table inside the ring, the allocation covers the larger of the two
  const size_t ring = d.sm_tab < 0 ? std::max<size_t>((size_t)d.ring_bytes, (size_t)d.H * 8) : (size_t)d.ring_bytes;
  return (size_t)d.meta_smem + (size_t)d.bar_bytes + ring;
}

cudaStream_t as_stream(void *s) { return static_cast<cudaStream_t>(s); }

const void *resolve_kernel_of(int threads, int minb) {
  if (threads == kThreadsSmall)
    return minb >= 3 ? reinterpret_cast<const void *>(&resolve_kernel<kThreadsSmall, 3, true>)
                     : reinterpret_cast<const void *>(&resolve_kernel<kThreadsSmall, 2, true>);
  return reinterpret_cast<const void *>(&resolve_kernel<kThreads, 1, false>);
}

int launch_resolve(hisparse *h, int layer, const int32_t *sel, int32_t *table, int32_t *hits, int32_t *misses,
                   cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(h->clusters * h->S));
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
  if (h->T == kThreadsSmall && h->minb >= 3)
    HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreadsSmall, 3, true>, h->d, layer, sel, table, hits, misses, h->S));
  else if (h->T == kThreadsSmall)
    HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreadsSmall, 2, true>, h->d, layer, sel, table, hits, misses, h->S));
  else
    HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreads, 1, false>, h->d, layer, sel, table, hits, misses, h->S));
  return HISPARSE_OK;
}

int launch_replay(hisparse *h, int layer, cudaStream_t st) {
  replay_kernel<<<h->d.N * h->S, h->T, h->replay_smem, st>>>(h->d, layer, h->S);
  HS_CUDA(cudaGetLastError());
  return HISPARSE_OK;
}

}  // namespace

// ---- the sparse-attention consumer (attention_kernel.cuh) ----

namespace {

struct AttGeom { int splits, tiles_per_split; size_t smem, workspace; };

// Splits of a row's k entries such that the launch fills the GPU once at two blocks per SM, in whole tiles.
int attention_geometry(const hisparse *h, int num_heads, int value_dims, AttGeom *g) {
  const int64_t E = h->d.E;
  if (num_heads < kAttHeads || num_heads % kAttHeads) return HISPARSE_EINVAL;
  if (E % 32 || E > 2 * 64 * kAttMaxQuerySteps || !(value_dims == 128 || value_dims == 256 || value_dims == 512) ||
      value_dims > E / 2)
    return HISPARSE_EINVAL;
  const int tiles = (h->d.k + kAttTile - 1) / kAttTile;
  const int64_t groups = (int64_t)h->d.N * (num_heads / kAttHeads);
  int want = (int)std::max<int64_t>(1, (2 * (int64_t)h->sm_count) / groups);
  want = std::min(want, tiles);
  g->tiles_per_split = (tiles + want - 1) / want;
  g->splits = (tiles + g->tiles_per_split - 1) / g->tiles_per_split;
  const size_t row = (size_t)E + kAttPad;
  g->smem = kAttHeads * row + kAttStages * kAttTile * row + kAttHeads * (kAttTile * 2 + kAttPad) + kAttGroups * 16 * 4 +
            kAttWarps * 64 * 16 + (kAttStages + 1) / 2 * 16 + (size_t)g->tiles_per_split * kAttTile * 4;
  g->workspace = (size_t)h->d.N * num_heads * g->splits * (value_dims + 4) * sizeof(float);
  return HISPARSE_OK;
}

template <int NV, int KQ>
int launch_attention_kq(hisparse *h, const AttGeom &g, const uint8_t *pool, const int32_t *table, const __nv_bfloat16 *q,
                        int num_heads, float scale, float *partial, cudaStream_t st) {
  int optin = 0;
  HS_CUDA(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device));
  if (g.smem > (size_t)optin) return HISPARSE_EINVAL;
  HS_CUDA(cudaFuncSetAttribute(sparse_attention_kernel<NV, KQ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)g.smem));
  const dim3 grid((unsigned)(h->d.N * g.splits), (unsigned)(num_heads / kAttHeads));
  sparse_attention_kernel<NV, KQ><<<grid, kAttThreads, g.smem, st>>>(pool, h->d.E, table, h->d.k, q, num_heads,
                                                                     scale * 1.4426950408889634f, g.splits, partial, h->d.status);
  HS_CUDA(cudaGetLastError());
  return HISPARSE_OK;
}

// The kernel keeps a quarter of the query's k-steps (16 numbers each) per warp in registers: the instantiation with the
// smallest array that holds them.
template <int NV>
int launch_attention(hisparse *h, const AttGeom &g, const uint8_t *pool, const int32_t *table, const __nv_bfloat16 *q,
                     int num_heads, float scale, float *partial, cudaStream_t st) {
  const int steps = (int)(h->d.E / 32), per_warp = (steps + 3) / 4;
  if (per_warp <= 3) return launch_attention_kq<NV, 3>(h, g, pool, table, q, num_heads, scale, partial, st);
  if (per_warp <= 5) return launch_attention_kq<NV, 5>(h, g, pool, table, q, num_heads, scale, partial, st);
  return launch_attention_kq<NV, kAttMaxQuerySteps>(h, g, pool, table, q, num_heads, scale, partial, st);
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
    for (size_t r = 0; r < N; ++r) cap_sum += (size_t)p2s_stride(c->capacity[r]);
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
  for (int r = 0; r < N; ++r) { h->p2s_off[r] = off; off += p2s_stride(h->cap[r]) * G; }
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
  int want = c->ctas_per_request;
  if (!want) {
    want = 1;
    while (want < 8 && N * want < 32) want <<= 1;
  }
  // Block size and shared memory.  One 1024-thread block per SM gives a request the whole SM: the table of missing
  // positions has memory of its own (cleared before the dependency wait) and the fetch ring takes all the rest.
  // When the grid takes several waves anyway (more blocks than SMs), three or two 512-thread blocks share an SM and
  // hide each other's dependent trips to memory; the table then borrows the ring's memory and the ring is as large
  // as a third (half) of the SM allows.
  const bool coop = want > 1;
  const int64_t piece = std::min<int64_t>(d.E, 8192);
  auto try_small = [&](int per_sm) {
    if (!(B <= 16 * kThreadsSmall && k <= 4 * kThreadsSmall)) return false;
    layout_smem(d, kThreadsSmall, coop, true);
    const int64_t budget = smem_per_sm / per_sm - 1024 - 256;   // per block: 1 KB reserved by the system, static arrays
    const int64_t room = budget - d.meta_smem - d.bar_bytes;
    return room >= piece * 4 && layout_ring(d, kThreadsSmall, room);
  };
  const bool want_small = !(c->flags & HISPARSE_FLAG_WIDE_BLOCKS) &&
                          ((c->flags & HISPARSE_FLAG_NARROW_BLOCKS) || (int64_t)N * want > sm_count);
  if ((c->flags & HISPARSE_FLAG_NARROW_BLOCKS) && (c->flags & HISPARSE_FLAG_WIDE_BLOCKS)) return fail(HISPARSE_EINVAL);
  h->T = kThreads; h->minb = 1;
  if (want_small) {
    // Three narrow blocks per SM (40 registers) only for shapes whose blocks can run the short loop (the kernel's
    // lean_shape: one block per request, every request the same capacity, whole 16-byte rows, a page-table slice that
    // fits the ring of a third of an SM); otherwise two (64 registers).  Measured on batches of 200 / 256 / 600
    // C2-shaped requests, whose slices are too long to stage: with two blocks per SM a launch with misses takes
    // 482 / 615 / 1420 us instead of 490 / 620 / 1432 and a launch without misses 12.3 / 13.3 / 23.6 us instead of
    // 19.3 / 22.4 / 37.5; on the short loop's shapes three per SM take 61.6 us per 8192 requests instead of 65.8.
    for (int per_sm = 3; per_sm >= 2 && h->T == kThreads; --per_sm) {
      if (!try_small(per_sm)) continue;
      const bool short_loop = want == 1 && d.uni_cap >= 0 && (k & 3) == 0 &&
                              !(c->flags & (HISPARSE_FLAG_EAGER_ORDER | HISPARSE_FLAG_PHASE_TIMERS)) &&
                              p2s_stride(d.uni_cap) * 2 + 16 <= (int64_t)d.ring_bytes;
      if (per_sm == 3 && !short_loop) continue;
      h->T = kThreadsSmall; h->minb = per_sm;
    }
    if (h->T == kThreads && (c->flags & HISPARSE_FLAG_NARROW_BLOCKS)) return fail(HISPARSE_EINVAL);
  }
  if (h->T == kThreads) {
    layout_smem(d, kThreads, coop, false);
    if (!layout_ring(d, kThreads, (int64_t)max_optin - 1024 - d.meta_smem - d.bar_bytes)) return fail(HISPARSE_EINVAL);
  }
  h->resolve_smem = kernel_smem_bytes(d);
  h->replay_smem = h->resolve_smem;   // same offsets, so that both kernels share the pipeline's geometry
  const void *kern = resolve_kernel_of(h->T, h->minb);
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

  // A grid of several waves of narrow blocks is launched as ONE resident wave whose blocks loop over the requests.
  h->clusters = N;
  if (h->S == 1 && h->T == kThreadsSmall) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, h->T, h->resolve_smem) != cudaSuccess) return fail(HISPARSE_ECUDA);
    if (per_sm >= 1) h->clusters = std::min(N, per_sm * sm_count);
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
  HS_TRY(dev_alloc(h, &d.layer_ns, (size_t)L * 2));
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
  HS_TRYC(cudaMemset(d.layer_ns, 0xff, (size_t)L * 8));
  HS_TRYC(cudaMemset(d.layer_ns + L, 0, (size_t)L * 8));
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
  if ((uintptr_t)new_kv_dev & 15) return HISPARSE_EINVAL;  // the records are read as 16-byte vectors
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

int hisparse_attention_workspace_bytes(const hisparse_t *h, int num_heads, int value_dims, size_t *bytes) {
  if (!h || !bytes) return HISPARSE_EINVAL;
  AttGeom g;
  const int rc = attention_geometry(h, num_heads, value_dims, &g);
  if (rc) return rc;
  *bytes = g.workspace;
  return HISPARSE_OK;
}

int hisparse_sparse_attention(hisparse_t *h, int layer, const void *q_dev, int num_heads, int value_dims,
                              const int32_t *slot_table_dev, float scale, float *out_dev, float *lse_dev,
                              void *workspace_dev, size_t workspace_bytes, void *stream) {
  if (!h || layer < 0 || layer >= h->d.L || !q_dev || !slot_table_dev || !out_dev || !lse_dev || !workspace_dev)
    return HISPARSE_EINVAL;
  if (((uintptr_t)q_dev | (uintptr_t)workspace_dev | (uintptr_t)out_dev) & 15) return HISPARSE_EINVAL;
  AttGeom g;
  int rc = attention_geometry(h, num_heads, value_dims, &g);
  if (rc) return rc;
  if (workspace_bytes < g.workspace) return HISPARSE_EINVAL;
  rc = hisparse_join(h, stream);   // a prefetch replay or a write-through may still be filling this layer's cache
  if (rc) return rc;
  cudaStream_t st = as_stream(stream);
  const uint8_t *pool = h->d.pool + (int64_t)layer * h->d.layer_pool_bytes;
  const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(q_dev);
  float *partial = static_cast<float *>(workspace_dev);
  switch (value_dims) {
    case 128: rc = launch_attention<2>(h, g, pool, slot_table_dev, q, num_heads, scale, partial, st); break;
    case 256: rc = launch_attention<4>(h, g, pool, slot_table_dev, q, num_heads, scale, partial, st); break;
    default: rc = launch_attention<8>(h, g, pool, slot_table_dev, q, num_heads, scale, partial, st); break;
  }
  if (rc) return rc;
  {
    // programmatic dependent launch: the combine kernel is scheduled while the attention kernel drains (it waits for
    // the partial results with griddepcontrol.wait), which hides its launch latency
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(h->d.N * num_heads));
    cfg.blockDim = dim3(128);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const float *partial_c = partial;
    const int splits = g.splits;
    HS_CUDA(cudaLaunchKernelEx(&cfg, sparse_attention_combine_kernel, partial_c, splits, value_dims, out_dev, lse_dev));
  }
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
    HS_CUDA(cudaMemcpy(tmp.data(), h->d.pos2slot + h->p2s_off[req] + (int64_t)g * p2s_stride(h->cap[req]), (size_t)h->cap[req] * 2,
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
  HS_CUDA(cudaMemcpy(h->d.pos2slot + h->p2s_off[req] + (int64_t)g * p2s_stride(cap), p2s.data(), (size_t)cap * 2, cudaMemcpyHostToDevice));
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

int hisparse_layer_times(hisparse_t *h, uint64_t *out) {
  if (!h || !out) return HISPARSE_EINVAL;
  const size_t L = (size_t)h->d.L;
  HS_CUDA(cudaSetDevice(h->device));
  HS_CUDA(cudaDeviceSynchronize());
  HS_CUDA(cudaMemcpy(out, h->d.layer_ns, L * 2 * 8, cudaMemcpyDeviceToHost));
  HS_CUDA(cudaMemset(h->d.layer_ns, 0xff, L * 8));   // start = "none yet"
  HS_CUDA(cudaMemset(h->d.layer_ns + L, 0, L * 8));
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


}  // extern "C"
