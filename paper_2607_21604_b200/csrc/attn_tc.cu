// GQA attention of the recomputed rows over the assembled K/V on the tcgen05 tensor cores
// (head_dim 128, 16-bit models).
//
// One CTA = one kv head x a block of BR = 128 / g query rows (g = q heads per kv head): the
// g heads of a row that share the kv head are stacked along M, so one K/V tile in shared
// memory serves all of them.  Per key tile of 128 keys:
//     S  = Q K^T          tcgen05.mma 128x128x16 x8, float in tensor memory; Q is the A operand
//                         read from tensor memory (written there once per CTA), K comes from
//                         shared memory
//     P  = exp2(S*c - m)  one M row per thread (no shuffles); the 16-bit probabilities go to a
//                         64-column buffer in tensor memory (tcgen05.st), two per column
//     O += P V            tcgen05.mma 128x128x16 x8 with P as the A operand from tensor memory
//                         and V from shared memory as an MN-major B operand; O stays in tensor
//                         memory for the whole key loop
// Tensor-memory columns: O 0..127 | Q 128..191 | P 192..255 | S0, S1 256..511.  With Q and P in
// tensor memory the MMAs read only K and V from shared memory, and shared memory holds three
// K and four V stages.
// The exponentials bound the kernel (the special-function unit of a scheduler needs ~1030
// cycles for the 32 x 128 values of its rows, as long as the 16 MMAs of the tile), so the
// softmax of consecutive tiles overlaps: two warp groups take the even and the odd key tiles,
// each with its own S buffer, which it hands back as soon as the scores sit in registers; the
// tensor pipe then works two tiles ahead of the softmax.
// Both groups scale their probabilities to one reference maximum m per row, kept in shared
// memory and handed from tile to tile (the group of tile j takes it over from the group of
// tile j-1 through an mbarrier per warp pair).  m is raised only when a tile's maximum
// exceeds it by more than 8 (in log2 units): the probabilities then stay below 2^8, and the
// rows of O in tensor memory are rescaled by that warp before its P V is issued - a rare
// event after the first tiles.  Each group keeps the row sums of its own tiles; the two
// halves are combined after the last tile and the groups write half of the columns each.
// Warp 0 feeds K tiles by TMA, warp 2 the V tiles; warp 1 issues Q K^T and warp 3 P V, so
// that each issuing thread hides the other's barrier round trips (MMAs of different threads
// are not ordered: every reuse of a tensor-memory buffer goes through an mbarrier).
// Row blocks are taken longest first across all kv heads (the last rows see the most keys).
// Query row r sees keys k_lo[r] <= j <= k_hi[r]; both arrays are non-decreasing in r.
// With second-range arrays (batched requests: a query row sees its own context and, not
// adjacent to it, its own query tokens) a row also sees k_lo2[r] <= j <= k_hi2[r]; the key
// tiles of a CTA then walk the hull of its rows' first ranges and after it the hull of the
// second ranges, each tile masked with the range of its segment.
#include "tc_common.cuh"

namespace {

constexpr int HD = 128;              // head dimension
constexpr int BN = 128;              // keys per tile
constexpr int SLAB = 128 * 64 * 2;   // one 64-wide slab of a 128-row tile: 16 KB
constexpr int TILE = 2 * SLAB;       // 32 KB
constexpr int ATT_THREADS = 384;     // warp group 0: TMA / MMA, warp groups 1 and 2: softmax
constexpr int K_STAGES = 3, V_STAGES = 4;
constexpr float RESCALE_STEP = 8.f;  // the reference maximum may lag a tile's maximum by this much
// shared memory: K[3] | V[4] | barriers | reference maxima and row sums
constexpr int OFF_K = 0, OFF_V = K_STAGES * TILE, OFF_BAR = (K_STAGES + V_STAGES) * TILE;
constexpr int OFF_ROW = OFF_BAR + 512;       // float m_ref[128], l_part[2][128], m_part[2][128]
constexpr int ATT_SMEM = OFF_ROW + 5 * 128 * 4;    // 232448 bytes is all a CTA may own: no slack for
                                                   // re-aligning, the buffer itself is declared 1024-byte aligned
// tensor-memory columns
constexpr uint32_t COL_O = 0, COL_Q = 128, COL_P = 192, COL_S = 256;

struct AttnParams {
  int R, T, n_q, n_kv, g, BR, row_blocks;
  const void* q;
  const int32_t* k_lo;
  const int32_t* k_hi;
  const int32_t* k_lo2;        // second visible range per row, or null
  const int32_t* k_hi2;
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

// Packed float pairs (one instruction for two lanes of arithmetic, the sm_100 float2 builtins:
// a pair stays in an aligned register pair, no moves around the instruction) and the 3-input
// maximum: the softmax loop is bound by issue slots shared between two warps of a scheduler.
__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

enum { B_QFULL = 0,     // Q sits in tensor memory (4 warps)
       B_KFULL = 1, B_KEMPTY = B_KFULL + K_STAGES, B_VFULL = B_KEMPTY + K_STAGES, B_VEMPTY = B_VFULL + V_STAGES,
       B_SFULL = B_VEMPTY + V_STAGES,   // [2] S of an even / odd tile is complete
       B_SEMPTY = B_SFULL + 2,          // [2] the group has taken S into registers (4 warps)
       B_PFULL = B_SEMPTY + 2,          // P of the next tile is in tensor memory (4 warps)
       B_ODONE = B_PFULL + 1,           // [4] P V of tile j (slot j mod 4) has completed
       B_OFINAL = B_ODONE + 4,          // the last P V has completed
       B_DEC = B_OFINAL + 1,            // [2][4] the warp of this quad has settled the reference maximum of an even / odd tile
       B_FIN = B_DEC + 8,               // [4] both warps of this quad have published their row sums
       B_COUNT = B_FIN + 4 };
static_assert(B_COUNT * 8 + 16 <= 512, "barriers, the tensor-memory slot and the abort flag share 512 bytes");
static_assert((K_STAGES + V_STAGES) * TILE + 512 + 5 * 128 * 4 <= 232448, "shared memory of one CTA");

template <typename T>
__global__ void __launch_bounds__(ATT_THREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                    const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  if (tc::smem_u32(smem) & 1023u) {               // swizzled tiles need 1024-byte alignment
    if (threadIdx.x == 0) set_status(p.status, AKVS_ERR_UNSUPPORTED);
    return;
  }
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bar + B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* m_ref = reinterpret_cast<float*>(smem + OFF_ROW);       // [128]
  float* l_part = m_ref + 128;                                    // [2][128]
  float* m_part = m_ref + 3 * 128;                                // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  pdl_trigger();
  if (threadIdx.x == 0) {
    for (int i = 0; i < B_COUNT; ++i) {
      int count = 1;
      if (i == B_QFULL || i == B_PFULL || (i >= B_SEMPTY && i < B_SEMPTY + 2)) count = 4;   // the warps of a group
      if (i >= B_FIN && i < B_FIN + 4) count = 2;                                           // one warp of each group
      tc::mbar_init(&bar[i], count);
    }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::fence_proxy_async();
  }
  if (threadIdx.x < 128) m_ref[threadIdx.x] = -1.0e30f;
  if (warp == 1) {
    tc::tmem_alloc(tmem_slot, 512);
    tc::tmem_relinquish();
  }
  pdl_wait();                       // the key ranges below are the first global memory this kernel reads
  // 1-D grid, kv head fastest: CTAs are handed out longest row block first across ALL heads
  // (the last rows see the most keys), so the tail of the launch is made of short CTAs
  const int hk = blockIdx.x % p.n_kv;
  const int r0 = (p.row_blocks - 1 - blockIdx.x / p.n_kv) * p.BR;
  const int n_rows = min(p.BR, p.R - r0);
  int key_lo = p.k_lo[r0];
  int key_hi = p.k_hi[r0 + n_rows - 1];
  int key_lo2 = 1, key_hi2 = 0;
  if (p.k_lo2) {
    // two ranges per row: neither is monotone across the rows of a block, take the hulls
    int a = 0x7fffffff, b = -1, c = 0x7fffffff, d = -1;
    for (int i = lane; i < n_rows; i += 32) {
      const int l1 = p.k_lo[r0 + i], h1 = p.k_hi[r0 + i], l2 = p.k_lo2[r0 + i], h2 = p.k_hi2[r0 + i];
      if (l1 <= h1) { a = min(a, l1); b = max(b, h1); }
      if (l2 <= h2) { c = min(c, l2); d = max(d, h2); }
    }
    key_lo = __reduce_min_sync(0xffffffffu, a);
    key_hi = __reduce_max_sync(0xffffffffu, b);
    key_lo2 = __reduce_min_sync(0xffffffffu, c);
    key_hi2 = __reduce_max_sync(0xffffffffu, d);
  }
  const int n_tiles1 = key_hi >= key_lo ? (key_hi - key_lo) / BN + 1 : 0;
  const int n_tiles = n_tiles1 + (key_hi2 >= key_lo2 ? (key_hi2 - key_lo2) / BN + 1 : 0);
  // first key of tile j
  auto tile_key = [&](int j) { return j < n_tiles1 ? key_lo + j * BN : key_lo2 + (j - n_tiles1) * BN; };

  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // Registers move from the TMA / MMA warp group to the two softmax groups (128 values of a
  // row live in each thread): 40 + 2 x 232 = 504 of the 512 per thread column.  Every role
  // branch starts with its own setmaxnreg so that the compiler budgets each region by itself.
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    if (warp == 0) {
      // ------------------------------------------------------------------ TMA producer: K
      if (lane == 0 && n_tiles > 0) {
        tc::prefetch_tmap(&tmK);
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
          const int s = j % K_STAGES;
          const uint32_t ph = ((j / K_STAGES) & 1) ^ 1;
          const int y = tile_key(j);
          if (!tc::mbar_wait(&bar[B_KEMPTY + s], ph, abort_flag)) { ok = false; break; }
          tc::mbar_expect_tx(&bar[B_KFULL + s], TILE);
          tc::tma_load_2d(smem + OFF_K + s * TILE, &tmK, hk * HD, y, &bar[B_KFULL + s]);
          tc::tma_load_2d(smem + OFF_K + s * TILE + SLAB, &tmK, hk * HD + 64, y, &bar[B_KFULL + s]);
        }
        if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
      }
    } else if (warp == 2) {
      // ------------------------------------------------------------------ TMA producer: V
      if (lane == 0 && n_tiles > 0) {
        tc::prefetch_tmap(&tmV);
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
          const int s = j % V_STAGES;
          const uint32_t ph = ((j / V_STAGES) & 1) ^ 1;
          const int y = tile_key(j);
          if (!tc::mbar_wait(&bar[B_VEMPTY + s], ph, abort_flag)) { ok = false; break; }
          tc::mbar_expect_tx(&bar[B_VFULL + s], TILE);
          tc::tma_load_2d(smem + OFF_V + s * TILE, &tmV, hk * HD, y, &bar[B_VFULL + s]);
          tc::tma_load_2d(smem + OFF_V + s * TILE + SLAB, &tmV, hk * HD + 64, y, &bar[B_VFULL + s]);
        }
        if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
      }
    } else if (warp == 1) {
      // ------------------------------------------------------------------ MMA issuer: S = Q K^T
      // Two threads feed the tensor pipe (this one and warp 3 for P V): each hides the other's
      // barrier round trips.  MMAs of different threads are not ordered: every reuse of a
      // tensor-memory buffer goes through an mbarrier.
      if (lane == 0 && n_tiles > 0) {
        bool ok = tc::mbar_wait(&bar[B_QFULL], 0, abort_flag);
        for (int j = 0; j < n_tiles && ok; ++j) {
          const int g = j & 1, ks = j % K_STAGES;
          if (j >= 2 && !tc::mbar_wait(&bar[B_SEMPTY + g], ((j >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
          if (!tc::mbar_wait(&bar[B_KFULL + ks], (j / K_STAGES) & 1, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t k_addr = tc::smem_u32(smem + OFF_K + ks * TILE);
#pragma unroll
          for (int k = 0; k < HD / 16; ++k) {
            // 16 elements of a Q row = 8 packed 32-bit columns
            const uint32_t off = (k >> 2) * SLAB + (k & 3) * 32;
            tc::mma_f16_ts(tmem_base + COL_S + g * BN, tmem_base + COL_Q + k * 8, tc::smem_desc_k_sw128(k_addr + off),
                           p.idesc_qk, k != 0);
          }
          tc::mma_commit(&bar[B_SFULL + g]);
          tc::mma_commit(&bar[B_KEMPTY + ks]);
        }
        if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
      }
    } else {
      // ------------------------------------------------------------------ MMA issuer: O += P V
      if (lane == 0 && n_tiles > 0) {
        bool ok = true;
        for (int j = 0; j < n_tiles && ok; ++j) {
          const int vs = j % V_STAGES;
          if (!tc::mbar_wait(&bar[B_VFULL + vs], (j / V_STAGES) & 1, abort_flag)) { ok = false; break; }
          if (!tc::mbar_wait(&bar[B_PFULL], j & 1, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t v_addr = tc::smem_u32(smem + OFF_V + vs * TILE);
#pragma unroll
          for (int k = 0; k < BN / 16; ++k) {
            // 16 keys of P = 8 packed 32-bit columns
            const uint64_t db = tc::smem_desc_mn_sw128(v_addr + k * 2048, SLAB);
            tc::mma_f16_ts(tmem_base + COL_O, tmem_base + COL_P + k * 8, db, p.idesc_pv, (j | k) != 0);
          }
          tc::mma_commit(&bar[B_ODONE + (j & 3)]);
          tc::mma_commit(&bar[B_VEMPTY + vs]);
          if (j == n_tiles - 1) tc::mma_commit(&bar[B_OFINAL]);
        }
        if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
      }
    }
  } else {
    // ---------------------------------------------------------------------- softmax groups
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
    const int quad = warp & 3;
    const int grp = (warp >> 2) - 1;                // 0: tiles 0, 2, 4, ...   1: tiles 1, 3, 5, ...
    const int m = quad * 32 + lane;                 // row of the M tile owned by this thread
    const int r_local = m / p.g, head = m - r_local * p.g;
    const int r = r0 + r_local;
    const bool valid = r_local < p.BR && r < p.R;
    // Rows of the M tile that belong to no query row (g does not divide 128, or the last row
    // block is short) have Q = 0 and are never written: they take every key as visible, so that
    // their warp does not run the masking pass on every tile for their sake.
    const int hi1 = valid ? p.k_hi[r] : 0x3fffffff;
    const int lo1 = !valid ? -0x40000000 : (p.k_lo[r] <= hi1 ? p.k_lo[r] : 0x40000000);   // nothing visible: no key reaches lo
    const int hi2 = !valid ? 0x3fffffff : (p.k_lo2 ? p.k_hi2[r] : -1);
    const int lo2 = !valid ? -0x40000000 : (p.k_lo2 && p.k_lo2[r] <= hi2 ? p.k_lo2[r] : 0x40000000);
    // key visible  <=>  lo <= key <= hi  <=>  (unsigned)(key - lo) <= hi - lo: one compare and a
    // select per element (a per-element && / || compiles to divergent branches, measured 2x slower)
    const unsigned span1 = hi1 >= lo1 ? (unsigned)(hi1 - lo1) : 0u;
    const unsigned span2 = hi2 >= lo2 ? (unsigned)(hi2 - lo2) : 0u;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    if (grp == 0 && n_tiles > 0) {
      // Q row of this thread: global -> registers -> tensor memory, 16-bit pairs as they lie in memory
      const uint4* qp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(p.q) +
                                                       ((size_t)r * p.n_q + (size_t)hk * p.g + head) * HD);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        uint32_t w[32];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 x = valid ? __ldg(qp + c * 8 + i) : make_uint4(0u, 0u, 0u, 0u);
          w[4 * i] = x.x; w[4 * i + 1] = x.y; w[4 * i + 2] = x.z; w[4 * i + 3] = x.w;
        }
        tc::tmem_st32(lane_addr + COL_Q + c * 32, w);
      }
      tc::tmem_st_wait();
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&bar[B_QFULL]);
    }
    const uint32_t s_addr = lane_addr + COL_S + grp * BN;
    float m_mine = -1.0e30f;                        // reference maximum this thread's row sum is scaled to
    float l_mine = 0.f;                             // row sum over this group's tiles
    bool ok = true;
    for (int j = grp; j < n_tiles && ok; j += 2) {
      const int j0 = tile_key(j);
      const bool seg2 = j >= n_tiles1;              // the tile belongs to the second ranges
      const int lo = seg2 ? lo2 : lo1, hi = seg2 ? hi2 : hi1;
      const unsigned span = seg2 ? span2 : span1;
      if (!tc::mbar_wait(&bar[B_SFULL + grp], (j >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      float t[BN];
      tc::tmem_ld32(s_addr + 0, *reinterpret_cast<float(*)[32]>(&t[0]));
      tc::tmem_ld32(s_addr + 32, *reinterpret_cast<float(*)[32]>(&t[32]));
      tc::tmem_ld32(s_addr + 64, *reinterpret_cast<float(*)[32]>(&t[64]));
      tc::tmem_ld32(s_addr + 96, *reinterpret_cast<float(*)[32]>(&t[96]));
      tc::tmem_ld_wait();
      // S is in registers: the buffer may take the group's next tile already
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&bar[B_SEMPTY + grp]);
      const bool full_tile = lo <= j0 && j0 + BN - 1 <= hi;
      if (!full_tile) {
#pragma unroll
        for (int i = 0; i < BN; ++i) {
          t[i] = ((unsigned)(j0 + i - lo) <= span) ? t[i] : -INFINITY;
        }
      }
      // four independent chains each for the maximum and the sum: a 128-long dependent chain
      // would leave the scheduler waiting on latency
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int i = 0; i < BN; i += 2) mx4[(i >> 1) & 3] = max3(mx4[(i >> 1) & 3], t[i], t[i + 1]);
      const float cand = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
      // take the reference maximum over from tile j-1 (the other group's warp of this quad)
      if (j > 0 && !tc::mbar_wait(&bar[B_DEC + ((j - 1) & 1) * 4 + quad], ((j - 1) >> 1) & 1, abort_flag)) {
        ok = false;
        break;
      }
      const float m_old = m_ref[m];
      const bool raise = cand > m_old + RESCALE_STEP;
      const float m_new = raise ? cand : m_old;
      if (raise) m_ref[m] = m_new;
      __syncwarp();
      if (lane == 0 && j + 1 < n_tiles) tc::mbar_arrive(&bar[B_DEC + (j & 1) * 4 + quad]);
      if (m_mine != m_new) l_mine *= ex2(m_mine - m_new);       // rare: keeps a special-function round trip off the usual path
      m_mine = m_new;
      if (j > 0 && __any_sync(0xffffffffu, raise)) {
        // rows of O accumulated so far move to the new maximum, once P(j-1) V(j-1) has landed
        if (!tc::mbar_wait(&bar[B_ODONE + ((j - 1) & 3)], ((j - 1) >> 2) & 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        const float f = ex2(m_old - m_new);         // exactly 1 for the rows that keep their maximum
#pragma unroll 1
        for (int c = 0; c < HD / 32; ++c) {
          float o[32];
          tc::tmem_ld32(lane_addr + COL_O + c * 32, o);
          tc::tmem_ld_wait();
          uint32_t ob[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) ob[i] = __float_as_uint(o[i] * f);
          tc::tmem_st32(lane_addr + COL_O + c * 32, ob);
        }
      }
      const float2 scale2 = make_float2(p.scale_log2, p.scale_log2), shift2 = make_float2(-m_new, -m_new);
      float2 sum2[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};      // two packed pairs of partial sums
#pragma unroll
      for (int i = 0; i < BN; i += 2) {
        const float2 x = __ffma2_rn(make_float2(t[i], t[i + 1]), scale2, shift2);
        t[i] = ex2(x.x);                                        // exp2(-inf) = 0 for masked keys
        t[i + 1] = ex2(x.y);
        sum2[(i >> 1) & 1] = __fadd2_rn(sum2[(i >> 1) & 1], make_float2(t[i], t[i + 1]));
      }
      l_mine += (sum2[0].x + sum2[0].y) + (sum2[1].x + sum2[1].y);
      // two 16-bit probabilities per 32-bit column, packed before the wait below: only the two
      // stores stay on the chain P(j-1) ready -> P(j-1) V(j-1) -> P(j) stored
      uint32_t pk[64];
#pragma unroll
      for (int i = 0; i < 64; ++i) pk[i] = pack2<T>(t[2 * i], t[2 * i + 1]);
      // the P buffer is free once P(j-1) V(j-1) has read it
      if (j > 0) {
        if (!tc::mbar_wait(&bar[B_ODONE + ((j - 1) & 3)], ((j - 1) >> 2) & 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
      }
      tc::tmem_st32(lane_addr + COL_P, *reinterpret_cast<uint32_t(*)[32]>(&pk[0]));
      tc::tmem_st32(lane_addr + COL_P + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk[32]));
      tc::tmem_st_wait();
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&bar[B_PFULL]);
    }
    // ---- epilogue: combine the two groups' row sums, normalise, write half of the columns each
    l_part[grp * 128 + m] = l_mine;
    m_part[grp * 128 + m] = m_mine;
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(&bar[B_FIN + quad]);
    if (ok && !tc::mbar_wait(&bar[B_FIN + quad], 0, abort_flag)) ok = false;
    if (ok && n_tiles > 0 && !tc::mbar_wait(&bar[B_OFINAL], 0, abort_flag)) ok = false;
    if (!ok && lane == 0) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    if (ok) {
      tc::fence_after_sync();
      const float ma = m_part[m], mb = m_part[128 + m];
      const float m_fin = fmaxf(ma, mb);            // the maximum only grows: the later tile's is final
      const float l = l_part[m] * ex2(ma - m_fin) + l_part[128 + m] * ex2(mb - m_fin);
      const float inv = l > 0.f ? 1.f / l : 0.f;
      float o[64];
      if (n_tiles > 0) {
        tc::tmem_ld32(lane_addr + COL_O + grp * 64, *reinterpret_cast<float(*)[32]>(&o[0]));
        tc::tmem_ld32(lane_addr + COL_O + grp * 64 + 32, *reinterpret_cast<float(*)[32]>(&o[32]));
        tc::tmem_ld_wait();
      } else {
#pragma unroll
        for (int i = 0; i < 64; ++i) o[i] = 0.f;
      }
      if (valid) {
        T* op = reinterpret_cast<T*>(p.out) + ((size_t)r * p.n_q + (size_t)hk * p.g + head) * HD + grp * 64;
#pragma unroll
        for (int v = 0; v < 8; ++v) {
          float w[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) w[i] = o[v * 8 + i] * inv;
          st16(op + v * 8, w);
        }
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
                            const int32_t* k_hi, const int32_t* k_lo2, const int32_t* k_hi2, int R, int T, int n_q,
                            int n_kv, int32_t* status, cudaStream_t st) {
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
  p.q = q; p.k_lo = k_lo; p.k_hi = k_hi; p.k_lo2 = k_lo2; p.k_hi2 = k_lo2 ? k_hi2 : nullptr; p.out = out; p.status = status;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  const uint32_t fmt = dtype == AKVS_F16 ? tc::kF16 : tc::kBF16;
  p.idesc_qk = tc::idesc_f16(fmt, 128, BN, 0);
  p.idesc_pv = tc::idesc_f16(fmt, 128, HD, 1);
  CUtensorMap tmK, tmV;
  AKVS_TRY(encode_tmap_2d_16bit(&tmK, k, T, (uint64_t)n_kv * HD, (uint64_t)n_kv * HD, BN));
  AKVS_TRY(encode_tmap_2d_16bit(&tmV, v, T, (uint64_t)n_kv * HD, (uint64_t)n_kv * HD, BN));
  p.row_blocks = akvs_cdiv(R, p.BR);
  const dim3 grid((unsigned)p.row_blocks * n_kv);
  double flops = 0;   // filled by the caller's accounting when profiling attention
  ProfScope prof(3, 0, flops, st);
  if (dtype == AKVS_BF16) AKVS_CUDA(launch_pdl(attention_tc_kernel<bf16>, grid, dim3(ATT_THREADS), ATT_SMEM, st, tmK, tmV, p));
  else AKVS_CUDA(launch_pdl(attention_tc_kernel<f16>, grid, dim3(ATT_THREADS), ATT_SMEM, st, tmK, tmV, p));
  AKVS_LAUNCHED();
  return AKVS_OK;
}
