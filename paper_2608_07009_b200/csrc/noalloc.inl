// Included by hisparse.cu: hisparse_resolve_noalloc, the entry point that allocates nothing.

// ------------------------------------------------------------------------------------------ no-allocation entry

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

  // bulk copies write the fetched records straight into the pool: its base must be 16-byte aligned, like the
  // histories (whose addresses live in device memory and cannot be checked here)
  if ((uintptr_t)st->pool_dev & 15) return HISPARSE_EINVAL;

  // Every call runs with the state's device current and leaves the caller's current device as it found it.
  const int dev = st->device;
  int caller_dev = -1;
  HS_CUDA(cudaGetDevice(&caller_dev));
  struct DeviceGuard {
    int restore;
    ~DeviceGuard() { if (restore >= 0) cudaSetDevice(restore); }
  } guard{-1};
  if (caller_dev != dev) {
    HS_CUDA(cudaSetDevice(dev));
    guard.restore = caller_dev;
  }
  std::unique_lock<std::mutex> lock(g_noalloc_mutex);
  if (!g_noalloc_ptr[dev]) {
    // Set-up, once per device, with that device current.  In host code the array's name is only a stand-in for
    // the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
    void *p = nullptr;
    HS_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    int optin = 0;
    HS_CUDA(cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    HS_CUDA(cudaFuncSetAttribute(resolve_kernel<kThreads, 1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - 1024));
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
  d.layer_ns = nullptr;
  layout_smem(d, kThreads, true, false);   // a request's two blocks may share the page-table lookups
  if (!layout_ring(d, kThreads, (int64_t)optin - 1024 - d.meta_smem - d.bar_bytes)) return HISPARSE_EINVAL;
  const size_t smem = kernel_smem_bytes(d);

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
  HS_CUDA(cudaLaunchKernelEx(&cfg, resolve_kernel<kThreads, 1, false>, d, 0, sel_dev, slot_table_dev, hits_dev, misses_dev, S));
  return HISPARSE_OK;
}

}  // extern "C"
