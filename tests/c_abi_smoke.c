/* Plain-C user of the library: shows that the boundary needs nothing but pointers and sizes.
 * Two requests, one layer, B = 8 slots, k = 4 selections, 32-byte records; two resolves and a byte check. */
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "hisparse.h"

#define CHECK(x) do { int rc_ = (x); if (rc_ != 0) { printf("FAIL %s -> %d (%s)\n", #x, rc_, hisparse_strerror(rc_)); return 1; } } while (0)
#define CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { printf("FAIL %s -> %s\n", #x, cudaGetErrorString(e_)); return 1; } } while (0)

int main(void) {
  enum { N = 2, L = 1, B = 8, K = 4, E = 32, CAP = 64, LEN = 40 };
  void *hist[N];
  for (int r = 0; r < N; ++r) {
    CHECK(hisparse_host_alloc((size_t)L * CAP * E, &hist[r]));
    for (int p = 0; p < CAP; ++p) memset((char *)hist[r] + (size_t)p * E, (r << 6) | p, E);
  }
  int64_t cap[N] = {CAP, CAP}, len[N] = {LEN, LEN};
  hisparse_config_t cfg;
  memset(&cfg, 0, sizeof cfg);
  cfg.num_requests = N; cfg.num_layers = L; cfg.layers_per_group = 1; cfg.cache_slots = B; cfg.top_k = K;
  cfg.entry_bytes = E; cfg.capacity = cap; cfg.init_len = len; cfg.host_history = hist; cfg.device = 0;
  hisparse_t *h = NULL;
  CHECK(hisparse_create(&cfg, &h));

  int32_t sel1[N * K] = {5, 6, 7, 8, 30, 31, 32, 33}, sel2[N * K] = {8, 9, 5, -1, 33, 1, 2, 30};
  int32_t *d_sel, *d_tab, *d_hits, *d_miss, *d_bad;
  uint8_t *d_out;
  CUDA(cudaMalloc((void **)&d_sel, sizeof sel1)); CUDA(cudaMalloc((void **)&d_tab, sizeof sel1));
  CUDA(cudaMalloc((void **)&d_hits, N * 4)); CUDA(cudaMalloc((void **)&d_miss, N * 4));
  CUDA(cudaMalloc((void **)&d_bad, 4)); CUDA(cudaMemset(d_bad, 0, 4));
  CUDA(cudaMalloc((void **)&d_out, (size_t)N * K * E));
  int32_t tab[N * K], hits[N], miss[N], bad = -1;

  CUDA(cudaMemcpy(d_sel, sel1, sizeof sel1, cudaMemcpyHostToDevice));
  CHECK(hisparse_resolve(h, 0, d_sel, d_tab, d_hits, d_miss, NULL));
  CHECK(hisparse_gather_check(h, 0, d_sel, d_tab, d_bad, NULL));
  CUDA(cudaMemcpy(tab, d_tab, sizeof tab, cudaMemcpyDeviceToHost));
  CUDA(cudaMemcpy(miss, d_miss, sizeof miss, cudaMemcpyDeviceToHost));
  for (int i = 0; i < N * K; ++i)               /* cold caches fill slots 0,1,2,3 of each request in selection order */
    if (tab[i] != (i / K) * (B + 1) + i % K) { printf("FAIL cold table[%d] = %d\n", i, tab[i]); return 1; }
  if (miss[0] != K || miss[1] != K) { printf("FAIL cold misses\n"); return 1; }

  CUDA(cudaMemcpy(d_sel, sel2, sizeof sel2, cudaMemcpyHostToDevice));
  CHECK(hisparse_resolve(h, 0, d_sel, d_tab, d_hits, d_miss, NULL));
  CHECK(hisparse_gather_check(h, 0, d_sel, d_tab, d_bad, NULL));
  CHECK(hisparse_gather(h, 0, d_tab, d_out, NULL));
  CUDA(cudaMemcpy(tab, d_tab, sizeof tab, cudaMemcpyDeviceToHost));
  CUDA(cudaMemcpy(hits, d_hits, sizeof hits, cudaMemcpyDeviceToHost));
  CUDA(cudaMemcpy(miss, d_miss, sizeof miss, cudaMemcpyDeviceToHost));
  CUDA(cudaMemcpy(&bad, d_bad, 4, cudaMemcpyDeviceToHost));
  /* request 0: 8 and 5 hit (slots 3 and 0), 9 misses -> slot 4, padding -> -1; request 1: 33 and 30 hit, 1 and 2 miss */
  const int32_t want[N * K] = {3, 4, 0, -1, 9 + 3, 9 + 4, 9 + 5, 9 + 0};
  for (int i = 0; i < N * K; ++i)
    if (tab[i] != want[i]) { printf("FAIL table[%d] = %d, want %d\n", i, tab[i], want[i]); return 1; }
  if (hits[0] != 2 || miss[0] != 1 || hits[1] != 2 || miss[1] != 2) { printf("FAIL counts\n"); return 1; }
  if (bad != 0) { printf("FAIL %d selections address wrong bytes\n", bad); return 1; }
  uint8_t out[N * K * E];
  CUDA(cudaMemcpy(out, d_out, sizeof out, cudaMemcpyDeviceToHost));
  for (int i = 0; i < N * K; ++i) {
    const uint8_t expect = sel2[i] < 0 ? 0 : (uint8_t)(((i / K) << 6) | sel2[i]);
    for (int b = 0; b < E; ++b)
      if (out[i * E + b] != expect) { printf("FAIL gathered byte of entry %d\n", i); return 1; }
  }
  uint32_t status = 99;
  CHECK(hisparse_status(h, &status));
  if (status != 0) { printf("FAIL status %u\n", status); return 1; }
  CHECK(hisparse_destroy(h));
  for (int r = 0; r < N; ++r) CHECK(hisparse_host_free(hist[r]));
  printf("C-ABI OK\n");
  return 0;
}
