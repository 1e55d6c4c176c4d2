// Included by hisparse.cu: the sparse-attention consumer of the slot table (Sec. 3.4 Phase 5: the attention kernel
// reads the selected records out of the GPU cache through the emitted slots; Sec. 2.1: attention is exact over the
// selected set).  Decode attention in the absorbed form of multi-head latent attention, the record layout of the DSA
// configurations: a record is D bf16 numbers (E = 2 D bytes), its key all D of them, its value the first Dv.
//
//   out[n, h, :] = sum_j softmax_j(scale * q[n, h, :] . rec[n, j]) * rec[n, j][:Dv]      over table[n, j] >= 0
//
// This IS a dense contraction (a [16 heads x D] query block against the gathered records), so it runs on the tensor
// cores (mma.sync m16n8k16, bf16 inputs, fp32 accumulation); but at 16 heads per GPU it moves 1152 bytes per record
// for 35 KFLOP, far below the machine's ridge, so the design is the one for an HBM-bound kernel: records are gathered
// by bulk copies (cp.async.bulk, one per record, mbarrier completion) into a double-buffered shared-memory tile while
// the previous tile is multiplied, the selection is split over enough thread blocks to fill the GPU in one wave, two
// blocks per SM, and a second small kernel combines the splits.
//
// Block = 8 warps, one request, one group of 16 heads, one contiguous split of the row's k entries, tiles of 32
// records.  Per tile: S = Q K^T (warp w: records 16 (w & 1) .. + 15 over quarter w >> 1 of D, with its slice of the
// query held in registers as A fragments and ONE ldmatrix.x4 of records per k-step; the four quarters are added through
// shared memory), running row maximum across the record groups through shared memory, P = exp(S - m) rounded to bf16
// into shared memory, O = alpha O + P V (warp w: value dims [Dv/8 w, Dv/8 (w+1)), fp32 accumulators in registers).
// Eight warps rather than four: a tile is a serial chain of ldmatrix -> mma -> maximum -> exp -> mma with block
// barriers in between.  Rows of the tile are padded by 16 bytes in shared memory, which makes every ldmatrix phase
// hit 8 different bank groups (a 1152-byte stride would put all rows on one).  The combine kernel is launched with
// programmatic dependent launch, so that its launch latency hides under this kernel's tail.

namespace {

constexpr int kAttTile = 32;        // records per tile
constexpr int kAttWarps = 8;
constexpr int kAttGroups = kAttTile / 8;   // groups of 8 records (one n-tile of the score MMA) per tile
constexpr int kAttThreads = kAttWarps * 32;
constexpr int kAttHeads = 16;       // heads per block (one m16 row block)
constexpr int kAttPad = 16;         // bytes of padding per staged row
constexpr int kAttStages = 2;       // tiles in the gather ring
constexpr int kAttMaxQuerySteps = 9;   // k-steps of the query per warp at most: records of up to 4 x 9 x 16 = 576 numbers

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Partial result of one (request, head, split): Dv unnormalised output numbers, then the running maximum (base 2) and
// the sum of the weights, padded to Dv + 4 floats so that rows stay 16-byte aligned.
// NV = Dv / 64 = 8-wide output tiles per warp (Dv = 512 -> 8).  KQ = k-steps (of 16 numbers) of the query that a warp
// keeps in registers = ceil(D / 64) at most (D = 576 -> 9).
template <int NV, int KQ>
__global__ void __launch_bounds__(kAttThreads, 2)
sparse_attention_kernel(const uint8_t *__restrict__ pool, const int64_t E, const int32_t *__restrict__ table, const int k,
                        const __nv_bfloat16 *__restrict__ q, const int H, const float scale_log2e, const int splits,
                        float *__restrict__ partial, uint32_t *status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int Dv = NV * 8 * kAttWarps;
  const int D = (int)(E / 2);
  const int row_bytes = (int)E + kAttPad;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = blockIdx.x / splits, split = blockIdx.x - n * splits, hg = blockIdx.y;
  // this split's entries of the row: [lo, hi), whole tiles except for the row's end
  const int per = ((k + splits - 1) / splits + kAttTile - 1) / kAttTile * kAttTile;
  const int lo = split * per, hi = lo + per < k ? lo + per : k;
  const int ntiles = hi > lo ? (hi - lo + kAttTile - 1) / kAttTile : 0;

  unsigned char *s_q = smem_raw;                                         // [16][row_bytes]
  unsigned char *s_kv = s_q + kAttHeads * row_bytes;                     // [2][kAttTile][row_bytes]
  unsigned char *s_p = s_kv + kAttStages * kAttTile * row_bytes;         // [16][kAttTile * 2 + 16] bf16 weights
  float *s_red = reinterpret_cast<float *>(s_p + kAttHeads * (kAttTile * 2 + kAttPad));   // [kAttGroups][16]
  float4 *s_part = reinterpret_cast<float4 *>(s_red + kAttGroups * 16);                    // [kAttWarps][2][32]: partial scores
  unsigned long long *s_bar = reinterpret_cast<unsigned long long *>(s_part + kAttWarps * 64);   // [kAttStages]
  int32_t *s_tab = reinterpret_cast<int32_t *>(s_bar + (kAttStages + 1) / 2 * 2);   // [per]: this split's table entries
  constexpr int p_stride = kAttTile * 2 + kAttPad;

  if (tid < kAttStages) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(s_bar + tid)), "r"(kAttTile) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  // this split's slice of the row (-1 past its end): read once, so that neither the gather nor the masking waits
  // for global memory inside the tile loop
  for (int i = tid; i < per; i += kAttThreads) s_tab[i] = lo + i < hi ? table[(int64_t)n * k + lo + i] : -1;
  // the query block of this head group: 16 rows of D bf16, padded
  {
    const uint4 *src = reinterpret_cast<const uint4 *>(q + ((int64_t)n * H + (int64_t)hg * kAttHeads) * D);
    const int per_row = (int)(E / 16);
    for (int i = tid; i < kAttHeads * per_row; i += kAttThreads) {
      const int r = i / per_row, c = i - r * per_row;
      *reinterpret_cast<uint4 *>(s_q + r * row_bytes + c * 16) = src[i];
    }
  }
  __syncthreads();

  // Gather of tile t into buffer t % kAttStages: the first four lanes of every warp bring one record each.  A valid
  // entry is one bulk copy; padding (or an entry past the split's end) is zero-filled by plain stores, so that 0 weight
  // times the row is 0, not NaN.  Four per warp rather than 32 lanes of one warp: a warp issues the bulk copies of its
  // lanes one after the other (the instruction takes its operands from uniform registers), ~65 cycles each, so one
  // warp spent ~2100 cycles per tile issuing, as long as the tile's whole arithmetic, with the other warps waiting for
  // it at the next barrier.
  // (16-byte cp.async copies by all threads instead: 32.7 us against 30 us; asking the later tiles' records into L2
  // with one prefetch each at the start: 37 us; a ninth warp that only gathers: with bulk copies 38 us, with cp.async
  // 59 us, against 26.5 us; requesting the first tiles before the table slice and the query are loaded: no change.
  // All measured on the C2 shape, none kept.)
  constexpr int kPerWarp = kAttTile / kAttWarps;   // records each warp brings
  auto gather = [&](const int t) {
    if (lane >= kPerWarp || t >= ntiles) return;
    const int j = warp * kPerWarp + lane;
    const int32_t rec = s_tab[t * kAttTile + j];
    unsigned char *dst = s_kv + ((t % kAttStages) * kAttTile + j) * row_bytes;
    const uint32_t bar = smem_u32(s_bar + (t % kAttStages));
    if (rec >= 0) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)E) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(dst)), "l"(pool + (int64_t)rec * E), "r"((uint32_t)E), "r"(bar) : "memory");
    } else {
      for (int o = 0; o < (int)E; o += 16) *reinterpret_cast<uint4 *>(dst + o) = make_uint4(0, 0, 0, 0);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // a later tile's bulk copy writes the same bytes
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
    }
  };
#pragma unroll
  for (int i = 0; i < kAttStages; ++i) gather(i);

  const int r0 = lane >> 2;                 // this thread's accumulator rows are r0 and r0 + 8
  // Scores: warp w multiplies the records 16 (w & 1) .. + 15 of a tile (two n-tiles) with the query over the k-steps
  // [ks_lo, ks_hi) = quarter w >> 1 of D; its slice of the query never changes, so it lives in registers as A
  // fragments (read from shared memory every tile, the query made up half of the kernel's shared-memory traffic).
  const int rh = warp & 1, dq = warp >> 1;
  const int KS = D / 16, ks_lo = KS * dq / 4, ks_hi = KS * (dq + 1) / 4;
  uint32_t qa[KQ][4];
  {
    const uint32_t a_addr = smem_u32(s_q) + (uint32_t)((lane & 15) * row_bytes + (lane >> 4) * 16);
#pragma unroll
    for (int i = 0; i < KQ; ++i) {
      if (ks_lo + i < ks_hi) ldsm_x4(qa[i], a_addr + (uint32_t)(ks_lo + i) * 32u);
      else qa[i][0] = qa[i][1] = qa[i][2] = qa[i][3] = 0u;
    }
  }
  // Softmax: warp w owns n-tile w & 3 of the summed scores (the warps w and w + 4 hold the same numbers; the lower
  // four write the weights)
  const int grp = warp & (kAttGroups - 1);
  const bool half = warp >= kAttGroups;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float acc[NV][4];
#pragma unroll
  for (int i = 0; i < NV; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  bool timed_out = false;

  for (int t = 0; t < ntiles; ++t) {
    if (!mbar_wait_bounded(smem_u32(s_bar + (t % kAttStages)), (uint32_t)((t / kAttStages) & 1))) timed_out = true;
    const unsigned char *kv = s_kv + (t % kAttStages) * kAttTile * row_bytes;
    // S = Q K^T for this warp's 16 records over its quarter of D: two 16 x 8 n-tiles, k-steps of 16, two accumulators
    // per n-tile (one would make the MMAs one dependent chain).  One ldmatrix.x4 per k-step: records 0-7 / 8-15 of the
    // warp's half, lower / upper 8 numbers of the k-step.
    float sc[4];
    {
      float part[2][2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) part[i][j][0] = part[i][j][1] = part[i][j][2] = part[i][j][3] = 0.f;
      const uint32_t b_addr = smem_u32(kv) + (uint32_t)((rh * 16 + (lane & 7) + (lane >> 4) * 8) * row_bytes + ((lane >> 3) & 1) * 16) +
                              (uint32_t)ks_lo * 32u;
#pragma unroll
      for (int i = 0; i < KQ; ++i) {
        if (ks_lo + i < ks_hi) {   // (uniform in the warp)
          uint32_t b[4];
          ldsm_x4(b, b_addr + (uint32_t)i * 32u);
          mma_bf16(part[0][i & 1], qa[i], b[0], b[1]);
          mma_bf16(part[1][i & 1], qa[i], b[2], b[3]);
        }
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
        s_part[(warp * 2 + nt) * 32 + lane] = make_float4(part[nt][0][0] + part[nt][1][0], part[nt][0][1] + part[nt][1][1],
                                                         part[nt][0][2] + part[nt][1][2], part[nt][0][3] + part[nt][1][3]);
      __syncthreads();
      // n-tile grp = records 8 grp .. + 7 was scored by the warps (grp >> 1) + 2 dq as their n-tile grp & 1: the four
      // quarters of D, added in a fixed order (so that both warps that own the n-tile hold bit-identical scores)
      const int src = grp * 32 + lane;
      const float4 p0 = s_part[src], p1 = s_part[src + 4 * 32], p2 = s_part[src + 8 * 32], p3 = s_part[src + 12 * 32];
      sc[0] = (p0.x + p1.x) + (p2.x + p3.x); sc[1] = (p0.y + p1.y) + (p2.y + p3.y);
      sc[2] = (p0.z + p1.z) + (p2.z + p3.z); sc[3] = (p0.w + p1.w) + (p2.w + p3.w);
    }
    // mask padding, scale into the base-2 domain, row maxima over the tile
    const int jbase = t * kAttTile + grp * 8 + 2 * (lane & 3);
    float s2[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) s2[i] = s_tab[jbase + (i & 1)] >= 0 ? sc[i] * scale_log2e : -INFINITY;
    float mx[2] = {fmaxf(s2[0], s2[1]), fmaxf(s2[2], s2[3])};
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 1));
      mx[i] = fmaxf(mx[i], __shfl_xor_sync(0xffffffffu, mx[i], 2));
    }
    if ((lane & 3) == 0 && !half) { s_red[grp * 16 + r0] = mx[0]; s_red[grp * 16 + r0 + 8] = mx[1]; }
    __syncthreads();
    float alpha[2], m_use[2];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = r0 + 8 * i;
      float mt = s_red[row];
#pragma unroll
      for (int w = 1; w < kAttGroups; ++w) mt = fmaxf(mt, s_red[w * 16 + row]);
      const float m_new = fmaxf(m_run[i], mt);
      alpha[i] = m_run[i] == -INFINITY ? 0.f : exp2f(m_run[i] - m_new);
      m_use[i] = m_new == -INFINITY ? 0.f : m_new;     // a row that is all padding so far: weights 0, no NaN
      m_run[i] = m_new;
    }
    float pr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[i] = exp2f(s2[i] - m_use[i >> 1]);
    l_run[0] = l_run[0] * alpha[0] + pr[0] + pr[1];
    l_run[1] = l_run[1] * alpha[1] + pr[2] + pr[3];
    // the weights as bf16, where every warp can read them as the A operand of P V
    if (!half) {
      const int col = grp * 8 + 2 * (lane & 3);
      *reinterpret_cast<uint32_t *>(s_p + r0 * p_stride + col * 2) = pack_bf16(pr[0], pr[1]);
      *reinterpret_cast<uint32_t *>(s_p + (r0 + 8) * p_stride + col * 2) = pack_bf16(pr[2], pr[3]);
    }
    if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {   // (a maximum moved: rescale what was summed so far)
#pragma unroll
      for (int i = 0; i < NV; ++i) { acc[i][0] *= alpha[0]; acc[i][1] *= alpha[0]; acc[i][2] *= alpha[1]; acc[i][3] *= alpha[1]; }
    }
    __syncthreads();
    // O += P V: this warp's value dims [warp * NV * 8, (warp + 1) * NV * 8), k-steps of 16 records
    {
      const uint32_t p_addr = smem_u32(s_p) + (uint32_t)((lane & 15) * p_stride + (lane >> 4) * 16);
      const uint32_t v_addr = smem_u32(kv) + (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * row_bytes + (lane >> 4) * 16) +
                              (uint32_t)(warp * NV * 16);
#pragma unroll
      for (int ks = 0; ks < kAttTile / 16; ++ks) {
        uint32_t a[4];
        ldsm_x4(a, p_addr + (uint32_t)ks * 32u);
#pragma unroll
        for (int nt = 0; nt < NV; nt += 2) {
          uint32_t b[4];
          ldsm_x4_trans(b, v_addr + (uint32_t)(ks * 16 * row_bytes) + (uint32_t)nt * 16u);
          mma_bf16(acc[nt], a, b[0], b[1]);
          mma_bf16(acc[nt + 1], a, b[2], b[3]);
        }
      }
    }
    __syncthreads();   // every warp is done with this tile's buffer, the weights and the maxima
    gather(t + kAttStages);
  }

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the combine kernel may be scheduled from here on
  // partial sums of the weights: across the quad, then across the record groups (one warp of each pair reports)
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 1);
    l_run[i] += __shfl_xor_sync(0xffffffffu, l_run[i], 2);
  }
  if ((lane & 3) == 0 && !half) { s_red[grp * 16 + r0] = l_run[0]; s_red[grp * 16 + r0 + 8] = l_run[1]; }
  __syncthreads();
  float *out = partial + (((int64_t)n * H + (int64_t)hg * kAttHeads) * splits + split) * (Dv + 4);
  const int64_t head_stride = (int64_t)splits * (Dv + 4);
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int col = warp * NV * 8 + i * 8 + 2 * (lane & 3);
    *reinterpret_cast<float2 *>(out + (int64_t)r0 * head_stride + col) = make_float2(acc[i][0], acc[i][1]);
    *reinterpret_cast<float2 *>(out + (int64_t)(r0 + 8) * head_stride + col) = make_float2(acc[i][2], acc[i][3]);
  }
  if (warp == 0 && (lane & 3) == 0) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int row = r0 + 8 * i;
      float l = 0.f;
#pragma unroll
      for (int w = 0; w < kAttGroups; ++w) l += s_red[w * 16 + row];
      out[(int64_t)row * head_stride + Dv] = m_run[i];
      out[(int64_t)row * head_stride + Dv + 1] = l;
    }
  }
  if (timed_out && tid == 0) atomicOr(status, HISPARSE_STATUS_TIMEOUT);
}

// out[n, h, :] = sum_s 2^(m_s - M) o_s / sum_s 2^(m_s - M) l_s,  lse = ln 2 * (M + log2 L).  One block of 128 threads
// per (n, h); splits <= 128 (one per tile of a row of at most 4096 entries).
__global__ void __launch_bounds__(128)
sparse_attention_combine_kernel(const float *__restrict__ partial, const int splits, const int Dv,
                                float *__restrict__ out, float *__restrict__ lse) {
  __shared__ float s_w[128];
  __shared__ float s_red[8];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t nh = blockIdx.x;
  const int stride = Dv + 4;
  const float *p = partial + nh * splits * stride;
  asm volatile("griddepcontrol.wait;" ::: "memory");   // the attention kernel's partial results are complete and visible
  const float m = tid < splits ? p[(int64_t)tid * stride + Dv] : -INFINITY;
  const float l = tid < splits ? p[(int64_t)tid * stride + Dv + 1] : 0.f;
  float M = m;
#pragma unroll
  for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  if (lane == 0) s_red[warp] = M;
  __syncthreads();
  M = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  const float w = m == -INFINITY ? 0.f : exp2f(m - M);
  s_w[tid] = w;
  float L = w * l;
#pragma unroll
  for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  if (lane == 0) s_red[4 + warp] = L;
  __syncthreads();
  L = (s_red[4] + s_red[5]) + (s_red[6] + s_red[7]);
  const float inv = L > 0.f ? 1.f / L : 0.f;
  for (int c = tid * 4; c < Dv; c += 128 * 4) {
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int s = 0; s < splits; ++s) {
      const float4 v = *reinterpret_cast<const float4 *>(p + (int64_t)s * stride + c);
      const float ws = s_w[s];
      o.x += ws * v.x; o.y += ws * v.y; o.z += ws * v.z; o.w += ws * v.w;
    }
    *reinterpret_cast<float4 *>(out + nh * Dv + c) = make_float4(o.x * inv, o.y * inv, o.z * inv, o.w * inv);
  }
  if (tid == 0) lse[nh] = L > 0.f ? 0.6931471805599453f * (M + log2f(L)) : -INFINITY;
}

}  // namespace
