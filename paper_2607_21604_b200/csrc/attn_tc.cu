// GQA attention of the recomputed rows over the assembled K/V on the tcgen05 tensor cores
// (head_dim 128, 16-bit models).
//
// One CTA = one kv head x a block of BR = 128 / g query rows (g = q heads per kv head): the
// g heads of a row that share the kv head are stacked along M, so one K/V tile in shared
// memory serves all of them.  Per key tile of 128 keys:
//     S  = Q K^T          tcgen05.mma 128x128x16 x8, float in tensor memory
//     P  = exp2(S*c - m)  4 softmax warps, one M row per thread (no shuffles); the 16-bit
//                         probabilities go back into the first 64 columns of the S buffer
//                         (tcgen05.st), two per 32-bit column
//     O_j = P V           tcgen05.mma 128x128x16 x8 with P read from tensor memory as the A
//                         operand and V from shared memory as an MN-major B operand
//     O  = O*corr + O_j   accumulated in registers by 4 more warps (no TMEM read-modify-write)
// S/P and O_j are double-buffered in tensor memory (4 x 128 columns): the tensor pipe computes
// S(j+1) and O(j-1) while the softmax of tile j runs; the in-order tensor pipe itself keeps
// S(j+2) from overwriting P(j) before P(j) V(j) has read it.  Keeping P out of shared memory
// leaves room for three K and three V stages and halves the shared-memory traffic of P V.
// Warp 0 feeds K and V tiles by TMA, warp 1 issues the MMAs, warps 2-5 do the softmax,
// warps 6-9 fold the P V products into the output rows they keep in registers; the per-tile
// rescale factors travel through shared memory.
// Row blocks are taken longest first across all kv heads (the last rows see the most keys).
// Query row r sees keys k_lo[r] <= j <= k_hi[r]; both arrays are non-decreasing in r.
#include "tc_common.cuh"

namespace {

constexpr int HD = 128;              // head dimension
constexpr int BN = 128;              // keys per tile
constexpr int SLAB = 128 * 64 * 2;   // one 64-wide slab of a 128-row tile: 16 KB
constexpr int TILE = 2 * SLAB;       // 32 KB
constexpr int ATT_THREADS = 320;
constexpr int KV_STAGES = 3;
// shared memory: Q | K[3] | V[3] | barriers | rescale factors
constexpr int OFF_Q = 0, OFF_K = TILE, OFF_V = 4 * TILE, OFF_BAR = 7 * TILE;
constexpr int OFF_CORR = OFF_BAR + 256;      // float corr[4][128], float l_final[128]
constexpr int ATT_SMEM = OFF_CORR + 5 * 128 * 4;   // 232192 of the 232448 bytes a CTA may own: no slack for
                                                   // re-aligning, the buffer itself is declared 1024-byte aligned

struct AttnParams {
  int R, T, n_q, n_kv, g, BR, row_blocks;
  const int32_t* k_lo;
  const int32_t* k_hi;
  void* out;
  float scale_log2;            // log2(e) / sqrt(head_dim)
  uint32_t idesc_qk, idesc_pv;
  int32_t* status;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = 4, B_VFULL = 7, B_VEMPTY = 10, B_SFULL = 13, B_PFULL = 15, B_OFULL = 17,
       B_OEMPTY = 19, B_COUNT = 21 };

template <typename T>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if (tc::smem_u32(smem) & 1023u) {               // swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) set_status(p.status, AKVS_ERR_UNSUPPORTED);
    return;
  }
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // 1-D grid, kv head fastest: CTAs are handed out longest row block first across ALL heads
  // (the last rows see the most keys), so the tail of the launch is made of short CTAs
  const int hk = blockIdx.x % p.n_kv;
  const int r0 = (p.row_blocks - 1 - blockIdx.x / p.n_kv) * p.BR;
  const int n_rows = min(p.BR, p.R - r0);
  const int key_lo = p.k_lo[r0];
  const int key_hi = p.k_hi[r0 + n_rows - 1];
  const int n_tiles = key_hi >= key_lo ? (key_hi - key_lo) / BN + 1 : 0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < B_COUNT; ++i) {
      const bool four = (i >= B_PFULL && i < B_PFULL + 2) || (i >= B_OEMPTY && i < B_OEMPTY + 2);
      tc::mbar_init(&bar[i], four ? 4 : 1);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::fence_proxy_async();
  }
  if (warp == 1) {
    tc::tmem_alloc(tmem_slot, 512);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  // tensor-memory columns: S0 0..127, S1 128..255, O0 256..383, O1 384..511

  if (warp == 0) {
    // -------------------------------------------------------------------- TMA producer
    if (lane == 0 && n_tiles > 0) {
      tc::prefetch_tmap(&tmQ);
      tc::prefetch_tmap(&tmK);
      tc::prefetch_tmap(&tmV);
      const uint32_t q_bytes = (uint32_t)(2 * p.BR * p.g * 128);
      tc::mbar_expect_tx(&bar[B_QFULL], q_bytes);
      tc::tma_load_3d(smem + OFF_Q, &tmQ, 0, hk * p.g, r0, &bar[B_QFULL]);
      tc::tma_load_3d(smem + OFF_Q + SLAB, &tmQ, 64, hk * p.g, r0, &bar[B_QFULL]);
      bool ok = true;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j % KV_STAGES;
        const uint32_t ph = ((j / KV_STAGES) & 1) ^ 1;
        const int y = key_lo + j * BN;
        if (!tc::mbar_wait(&bar[B_KEMPTY + s], ph, abort_flag)) { ok = false; break; }
        tc::mbar_expect_tx(&bar[B_KFULL + s], TILE);
        tc::tma_load_2d(smem + OFF_K + s * TILE, &tmK, hk * HD, y, &bar[B_KFULL + s]);
        tc::tma_load_2d(smem + OFF_K + s * TILE + SLAB, &tmK, hk * HD + 64, y, &bar[B_KFULL + s]);
        if (!tc::mbar_wait(&bar[B_VEMPTY + s], ph, abort_flag)) { ok = false; break; }
        tc::mbar_expect_tx(&bar[B_VFULL + s], TILE);
        tc::tma_load_2d(smem + OFF_V + s * TILE, &tmV, hk * HD, y, &bar[B_VFULL + s]);
        tc::tma_load_2d(smem + OFF_V + s * TILE + SLAB, &tmV, hk * HD + 64, y, &bar[B_VFULL + s]);
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // -------------------------------------------------------------------- MMA issuer
    if (lane == 0 && n_tiles > 0) {
      bool ok = tc::mbar_wait(&bar[B_QFULL], 0, abort_flag);
      const uint32_t q_addr = tc::smem_u32(smem + OFF_Q);
      // S(j) may overwrite the buffer that held S(j-2)/P(j-2): the tensor pipe runs the MMAs of
      // this thread in order and P(j-2) V(j-2) was issued before, so no barrier is needed
      auto issue_qk = [&](int j) -> bool {
        const int s = j & 1, ks = j % KV_STAGES;
        if (!tc::mbar_wait(&bar[B_KFULL + ks], (j / KV_STAGES) & 1, abort_flag)) return false;
        tc::fence_after_sync();
        const uint32_t k_addr = tc::smem_u32(smem + OFF_K + ks * TILE);
#pragma unroll
        for (int k = 0; k < HD / 16; ++k) {
          const uint32_t off = (k >> 2) * SLAB + (k & 3) * 32;
          tc::mma_f16(tmem_base + s * BN, tc::smem_desc_k_sw128(q_addr + off), tc::smem_desc_k_sw128(k_addr + off),
                      p.idesc_qk, k != 0);
        }
        tc::mma_commit(&bar[B_SFULL + s]);
        tc::mma_commit(&bar[B_KEMPTY + ks]);
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int s = j & 1;
        const uint32_t ph = (j >> 1) & 1;
        if (j + 1 < n_tiles && !issue_qk(j + 1)) { ok = false; break; }
        const int vs = j % KV_STAGES;
        if (!tc::mbar_wait(&bar[B_VFULL + vs], (j / KV_STAGES) & 1, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(&bar[B_PFULL + s], ph, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(&bar[B_OEMPTY + s], ph ^ 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t v_addr = tc::smem_u32(smem + OFF_V + vs * TILE);
#pragma unroll
        for (int k = 0; k < BN / 16; ++k) {
          // 16 keys of P = 8 packed 32-bit columns of the S/P buffer
          const uint64_t db = tc::smem_desc_mn_sw128(v_addr + k * 2048, SLAB);
          tc::mma_f16_ts(tmem_base + 2 * BN + s * HD, tmem_base + s * BN + k * 8, db, p.idesc_pv, k != 0);
        }
        tc::mma_commit(&bar[B_OFULL + s]);
        tc::mma_commit(&bar[B_VEMPTY + vs]);
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else if (warp < 6) {
    // -------------------------------------------------------------------- softmax
    const int quad = warp & 3;
    const int m = quad * 32 + lane;                 // row of the M tile owned by this thread
    const int r_local = m / p.g;
    const int r = r0 + r_local;
    const bool valid = r_local < p.BR && r < p.R;
    const int hi = valid ? p.k_hi[r] : -1;
    const int lo = valid && p.k_lo[r] <= hi ? p.k_lo[r] : 0x40000000;   // nothing visible: no key reaches lo
    // key visible  <=>  lo <= key <= hi  <=>  (unsigned)(key - lo) <= hi - lo: one compare and a
    // select per element (a per-element && / || compiles to divergent branches, measured 2x slower)
    const unsigned span = hi >= lo ? (unsigned)(hi - lo) : 0u;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    float* corr_ring = reinterpret_cast<float*>(smem + OFF_CORR);
    float m_run = -1.0e30f, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j & 1;
      const uint32_t ph = (j >> 1) & 1;
      const int j0 = key_lo + j * BN;
      if (!tc::mbar_wait(&bar[B_SFULL + s], ph, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      float t[BN];
      tc::tmem_ld32(lane_addr + s * BN + 0, *reinterpret_cast<float(*)[32]>(&t[0]));
      tc::tmem_ld32(lane_addr + s * BN + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
      tc::tmem_ld32(lane_addr + s * BN + 64, *reinterpret_cast<float(*)[32]>(&t[64]));
      tc::tmem_ld32(lane_addr + s * BN + 96, *reinterpret_cast<float(*)[32]>(&t[96]));
      tc::tmem_ld_wait();
      const bool full_tile = lo <= j0 && j0 + BN - 1 <= hi;
      if (!full_tile) {
#pragma unroll
        for (int i = 0; i < BN; ++i) {
          t[i] = ((unsigned)(j0 + i - lo) <= span) ? t[i] : -INFINITY;
        }
      }
      // four independent chains each for the maximum and the sum: a scheduler that runs one
      // softmax warp cannot hide a 128-long dependent chain
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < BN; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], t[i]);
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float m_new = fmaxf(m_run, mx * p.scale_log2);
      const float corr = ex2(m_run - m_new);
      m_run = m_new;
      corr_ring[(j & 3) * 128 + m] = corr;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int i = 0; i < BN; ++i) {
        t[i] = ex2(fmaf(t[i], p.scale_log2, -m_new));          // exp2(-inf) = 0 for masked keys
        sum4[i & 3] += t[i];
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l_run = fmaf(l_run, corr, sum);
      if (j == n_tiles - 1) corr_ring[4 * 128 + m] = l_run;
      // P overwrites the first 64 columns of this S buffer: two 16-bit probabilities per column
      uint32_t pk[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) pk[i] = pack2<T>(t[2 * i], t[2 * i + 1]);
      tc::tmem_st32(lane_addr + s * BN, pk);
#pragma unroll
      for (int i = 0; i < 32; ++i) pk[i] = pack2<T>(t[64 + 2 * i], t[64 + 2 * i + 1]);
      tc::tmem_st32(lane_addr + s * BN + 32, pk);
      tc::tmem_st_wait();
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&bar[B_PFULL + s]);
    }
    if (!ok && lane == 0) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
  } else {
    // -------------------------------------------------------------------- output accumulation
    const int quad = warp & 3;
    const int m = quad * 32 + lane;
    const int r_local = m / p.g, head = m - r_local * p.g;
    const int r = r0 + r_local;
    const bool valid = r_local < p.BR && r < p.R;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float* corr_ring = reinterpret_cast<const float*>(smem + OFF_CORR);
    float o[HD];
#pragma unroll
    for (int i = 0; i < HD; ++i) o[i] = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles && ok; ++j) {
      const int s = j & 1;
      if (!tc::mbar_wait(&bar[B_OFULL + s], (j >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      const float corr = corr_ring[(j & 3) * 128 + m];
#pragma unroll
      for (int c = 0; c < HD / 64; ++c) {
        float t[64];
        tc::tmem_ld32(lane_addr + 2 * BN + s * HD + c * 64, *reinterpret_cast<float(*)[32]>(&t[0]));
        tc::tmem_ld32(lane_addr + 2 * BN + s * HD + c * 64 + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
        tc::tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 64; ++i) o[c * 64 + i] = fmaf(o[c * 64 + i], corr, t[i]);
      }
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&bar[B_OEMPTY + s]);
    }
    if (!ok && lane == 0) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    if (valid) {
      const float l = n_tiles > 0 ? corr_ring[4 * 128 + m] : 0.f;
      const float inv = l > 0.f ? 1.f / l : 0.f;
      T* op = reinterpret_cast<T*>(p.out) + ((size_t)r * p.n_q + (size_t)hk * p.g + head) * HD;
#pragma unroll
      for (int v = 0; v < HD / 8; ++v) {
        float t[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) t[i] = o[v * 8 + i] * inv;
        st16(op + v * 8, t);
      }
    }
  }

  if (*abort_flag) __nanosleep(200000);
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

}  // namespace

// q [R][n_q][128], k/v [T][n_kv][128], out [R][n_q][128], all of the 16-bit type `dtype`.
int32_t launch_attention_tc(int dtype, const void* q, const void* k, const void* v, void* out, const int32_t* k_lo,
                            const int32_t* k_hi, int R, int T, int n_q, int n_kv, int32_t* status, cudaStream_t st) {
  if (R == 0) return AKVS_OK;
  if (dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  if (n_kv <= 0 || n_q % n_kv != 0 || n_q / n_kv > 128 || T <= 0) return AKVS_ERR_SHAPE;
  static bool attr_set = false;
  if (!attr_set) {
    AKVS_CUDA(cudaFuncSetAttribute(attention_tc_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM));
    AKVS_CUDA(cudaFuncSetAttribute(attention_tc_kernel<f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, ATT_SMEM));
    attr_set = true;
  }
  AttnParams p;
  p.R = R; p.T = T; p.n_q = n_q; p.n_kv = n_kv;
  p.g = n_q / n_kv;
  p.BR = 128 / p.g;
  p.k_lo = k_lo; p.k_hi = k_hi; p.out = out; p.status = status;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  const uint32_t fmt = dtype == AKVS_F16 ? tc::kF16 : tc::kBF16;
  p.idesc_qk = tc::idesc_f16(fmt, fmt, 128, BN, 0);
  p.idesc_pv = tc::idesc_f16(fmt, fmt, 128, HD, 1);
  CUtensorMap tmQ, tmK, tmV;
  AKVS_TRY(encode_tmap_3d_16bit(&tmQ, q, HD, n_q, R, HD, (uint64_t)n_q * HD, p.g, p.BR));
  AKVS_TRY(encode_tmap_2d_16bit(&tmK, k, T, (uint64_t)n_kv * HD, (uint64_t)n_kv * HD, BN));
  AKVS_TRY(encode_tmap_2d_16bit(&tmV, v, T, (uint64_t)n_kv * HD, (uint64_t)n_kv * HD, BN));
  p.row_blocks = akvs_cdiv(R, p.BR);
  const dim3 grid((unsigned)p.row_blocks * n_kv);
  double flops = 0;   // filled by the caller's accounting when profiling attention
  ProfScope prof(3, 0, flops, st);
  if (dtype == AKVS_BF16) attention_tc_kernel<bf16><<<grid, ATT_THREADS, ATT_SMEM, st>>>(tmQ, tmK, tmV, p);
  else attention_tc_kernel<f16><<<grid, ATT_THREADS, ATT_SMEM, st>>>(tmQ, tmK, tmV, p);
  AKVS_LAUNCHED();
  return AKVS_OK;
}
