// Linear layers of the 16-bit models (bfloat16 or float16, both operands the same type) on
// the 5th-generation tensor cores (tcgen05), float accumulation in tensor memory.  y = x W^T with
// x [M][K] and W [N][K], both K-major, staged by TMA in
// 128-byte-swizzled 64-wide k slabs.
//
// Persistent kernel, one CTA per SM, 6 warps:
//   warp 0      TMA producer (one elected lane), 4-stage ring of (A 128x64, B 256x64) slabs
//   warp 1      tensor-memory allocation + MMA issue (one lane): 128x256x16 tcgen05.mma
//   warps 2-5   epilogue: tcgen05.ld the 128x256 float accumulator (row per thread), fuse
//               the layer's elementwise tail, store.  Two accumulators (2 x 256 columns)
//               let the epilogue of tile i overlap the main loop of tile i+1.
// The 256 accumulator columns are two 128-row blocks of B that may come from different
// weight matrices: (Wq | Wk | Wv) share one launch, and (W_gate, W_up) land side by side
// so that silu(gate) * up is formed in registers and only the activation is written.
// Epilogues: store (16-bit; a 128-column block that is one attention head gets its RoPE rotation
// in registers), residual (h += acc as a vector reduction at the L2, nothing is read back),
// SwiGLU.  A launch whose 128x256 tiles would occupy well under all SMs runs 128x128 tiles
// (one B block per tile, `nh` = 1); every other launch of more than 128 rows runs on CTA pairs
// with 256x256 tiles (gemm_tc_pair_kernel below, tcgen05.mma.cta_group::2).  The kernels are launched as
// programmatic dependents: set-up and the first weight tiles overlap the tail of the kernel before.
#include <unordered_map>

#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BNH = 128, BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, BH_BYTES = BNH * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + 2 * BH_BYTES;        // 49152
constexpr int EPI_PITCH = 144;                             // bytes between staged rows: 128 of payload + 16
constexpr int EPI_STAGE_BYTES = 32 * EPI_PITCH;            // staging tile of one epilogue warp
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + 4 * EPI_STAGE_BYTES;
static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of the GEMM");
constexpr int THREADS = 192;

enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2 };

struct GemmParams {
  int M, K, tiles_m, tiles_n;
  int nh;                 // 128-column blocks of B per tile: 2 (128x256 tiles) or 1 (128x128, when 256-wide
                          // tiles would leave most SMs without work)
  int n_seg;
  int seg_blocks[3];      // 128-row blocks of each B matrix
  void* seg_out[3];       // output of each segment (16-bit [M][ldc], or float for EPI_RESID)
  int seg_ldc[3];
  int32_t* status;
  uint32_t idesc;         // tcgen05 instruction descriptor (operand formats, M, N)
  // fused RoPE (EPI_STORE only): segments whose bit is set in rope_mask hold heads of 128
  // columns; row r is rotated through rope[pos[r]] (rotate-half pairs (i, i + 64)) before the store
  const float2* rope;     // [positions][64] (cos, sin)
  const int32_t* pos;     // [M]
  int rope_mask;
  int n_pos;              // rows of the rope table: a position outside [0, n_pos) (positions may be caller
                          // data) raises AKVS_ERR_INVALID_ARG and is rotated as position 0
  // split-K (EPI_RESID only: its epilogue adds into h at the L2, so partial sums over k ranges
  // need no second pass): work item i = (split i / n_tiles, tile i % n_tiles); a split covers
  // k slabs [split * kb_split, min(KB, (split + 1) * kb_split)), never empty
  int splits, kb_split;
  // Ordered partial sums: the epilogue warps of split s of a tile start adding only when all
  // split_warps epilogue warps of every earlier split of that tile have added theirs (a counter
  // per tile, back at zero when the launch ends), so every element receives its partial sums in
  // the same order on every run.
  unsigned int* split_count;
  int split_warps;
};

constexpr int SPLITK_MAX_TILES = 8192;
#ifndef AKVS_SPLIT_MIN_KB
#define AKVS_SPLIT_MIN_KB 32
#endif
// One counter per output tile of the split launch in flight.  File-scope device memory, so a
// single-step call needs no workspace; like the rest of the library's process-wide state it
// assumes one stream of launches per device at a time.
__device__ unsigned int g_splitk_count[SPLITK_MAX_TILES];

// Bounded wait until *c >= target.  False when the limit ran out or the CTA is aborting.
__device__ __forceinline__ bool wait_count(const unsigned int* c, unsigned int target, volatile int* abort_flag) {
  const long long t0 = clock64();
  for (uint32_t it = 0;; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(c) : "memory");
    if (v >= target) return true;
    __nanosleep(64);
    if ((it & 63) == 63 && (*abort_flag || clock64() - t0 > tc::kWaitCycles)) return false;
  }
}

// Before the epilogue of a split work item: wait for the tile's earlier splits.
__device__ __forceinline__ bool split_turn(const GemmParams& p, int item, int n_tiles, int lane, volatile int* abort_flag) {
  const int split = item / n_tiles;
  if (split == 0) return true;
  int got = 1;
  if (lane == 0) got = wait_count(p.split_count + (item - split * n_tiles), (unsigned)(split * p.split_warps), abort_flag);
  return __shfl_sync(0xffffffffu, got, 0) != 0;
}
// After it: this warp's reductions are performed, then the tile's count moves; the launch's last
// arrival puts it back to zero.
__device__ __forceinline__ void split_done(const GemmParams& p, int tile, int lane) {
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    unsigned int* c = p.split_count + tile;
    const unsigned int old = atomicAdd(c, 1u);
    if (old + 1u == (unsigned)(p.splits * p.split_warps)) atomicExch(c, 0u);
  }
}

// Tile and k-slab range of work item `item`.
__device__ __forceinline__ void item_range(const GemmParams& p, int item, int n_tiles, int KB, int& tile, int& kb0,
                                           int& kb1) {
  const int split = item / n_tiles;
  tile = item - split * n_tiles;
  kb0 = split * p.kb_split;
  kb1 = kb0 + p.kb_split < KB ? kb0 + p.kb_split : KB;
}

// Which weight matrix and which of its rows the 128-row block `block` of the concatenated
// output columns comes from.  Past the last matrix the row lies beyond its extent and the
// TMA load fills zeros.
__device__ __forceinline__ void locate(const GemmParams& p, int block, int& seg, int& row) {
  seg = 0;
  while (seg < p.n_seg - 1 && block >= p.seg_blocks[seg]) {
    block -= p.seg_blocks[seg];
    ++seg;
  }
  row = block * BNH;
}

// SwiGLU epilogue of one accumulator tile for one thread: its row `row` of the output, tile column
// `tn`; t_addr = the accumulator's tensor-memory address in the warp's lane quadrant.  Stores
// straight from the row-per-thread layout of tcgen05.ld (64 contiguous bytes per thread and
// chunk).  Staging these through shared memory like the other epilogues measured 4 % SLOWER on
// the 14-round W_gate/W_up launch: every tile but the last overlaps the next tile's main loop,
// whose MMAs want the shared-memory bandwidth to themselves, and the tail is short here.
template <typename T>
__device__ __forceinline__ void epilogue_swiglu_row(const GemmParams& p, uint32_t t_addr, int row, int tn) {
  T* out = reinterpret_cast<T*>(p.seg_out[0]);
  const int ldc = p.seg_ldc[0];
  const int n_valid = p.seg_blocks[0] * BNH;
#pragma unroll 1
  for (int c = 0; c < BNH / 32; ++c) {
    float g[32], u[32];
    tc::tmem_ld32(t_addr + c * 32, g);
    tc::tmem_ld32(t_addr + BNH + c * 32, u);
    tc::tmem_ld_wait();
    const int col = tn * BNH + c * 32;
    if (row < p.M && col < n_valid) {
      T* o = out + (size_t)row * ldc + col;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        float r[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float x = g[v * 8 + i];
          r[i] = x / (1.f + __expf(-x)) * u[v * 8 + i];
        }
        st16(o + v * 8, r);
      }
    }
  }
}

// Store and residual epilogues of one accumulator tile for one warp: the 32 rows row0 .. row0+31
// of the output, the 2 (or `nh`) 128-column blocks of tile column `tn`.  tcgen05.ld hands each
// thread ONE ROW (32 columns per load); storing from that layout sends 32 rows x 16 bytes per
// instruction - 32 separate lines - and the last tile's epilogue is the exposed tail of the
// launch.  So each chunk goes through a per-warp staging tile in shared memory (32 rows x 128
// bytes, row pitch 144 bytes so that 16-byte accesses of a quarter warp fall on distinct banks)
// and leaves it as whole 128-byte (64 for the rotated heads) row segments, 8 lanes per row
// (measured on the 8B shapes: QKV -5 us, W_o -10 us, W_down -7 us per launch).
template <int EPI, typename T>
__device__ __forceinline__ void epilogue_warp(const GemmParams& p, uint32_t t_addr, int row0, int lane, int tn, int nh,
                                              uint8_t* stage) {
  const int row = row0 + lane;                  // the row this thread holds after tcgen05.ld
  uint8_t* mine = stage + lane * EPI_PITCH;
  const int q = lane & 7, rsub = lane >> 3;     // on the way out: 16-byte piece q of staged row 4 i + rsub
#pragma unroll 1
  for (int hf = 0; hf < nh; ++hf) {
    int seg, brow;
    locate(p, nh * tn + hf, seg, brow);
    const bool valid = brow < p.seg_blocks[seg] * BNH;
    const int ldc = p.seg_ldc[seg];
    if (EPI == EPI_STORE && ((p.rope_mask >> seg) & 1)) {
      // this 128-column block is one head: rotate the pairs (i, i + 64) in registers
      int ps = row < p.M ? p.pos[row] : 0;
      if ((unsigned)ps >= (unsigned)p.n_pos) {
        set_status(p.status, AKVS_ERR_INVALID_ARG);
        ps = 0;
      }
      const float2* rt = p.rope + (size_t)ps * 64;
      T* out = reinterpret_cast<T*>(p.seg_out[seg]);
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        float lo[32], hi[32];
        tc::tmem_ld32(t_addr + hf * BNH + c * 32, lo);
        tc::tmem_ld32(t_addr + hf * BNH + 64 + c * 32, hi);
        tc::tmem_ld_wait();
        __syncwarp();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float rl[8], rh[8];
#pragma unroll
          for (int i = 0; i < 8; i += 2) {
            const float4 cs = *reinterpret_cast<const float4*>(rt + c * 32 + v * 8 + i);   // two (cos, sin)
            rl[i] = lo[v * 8 + i] * cs.x - hi[v * 8 + i] * cs.y;
            rh[i] = hi[v * 8 + i] * cs.x + lo[v * 8 + i] * cs.y;
            rl[i + 1] = lo[v * 8 + i + 1] * cs.z - hi[v * 8 + i + 1] * cs.w;
            rh[i + 1] = hi[v * 8 + i + 1] * cs.z + lo[v * 8 + i + 1] * cs.w;
          }
          st16(reinterpret_cast<T*>(mine + v * 16), rl);          // bytes 0..63: columns c*32 .. +31
          st16(reinterpret_cast<T*>(mine + 64 + v * 16), rh);     // bytes 64..127: columns 64 + c*32 .. +31
        }
        __syncwarp();
        const int col = brow + (q < 4 ? c * 32 + q * 8 : 64 + c * 32 + (q - 4) * 8);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rr = 4 * i + rsub, grow = row0 + rr;
          if (grow < p.M && valid)
            *reinterpret_cast<uint4*>(out + (size_t)grow * ldc + col) =
                *reinterpret_cast<const uint4*>(stage + rr * EPI_PITCH + q * 16);
        }
      }
      continue;
    }
    if (EPI == EPI_RESID) {
      float* out = reinterpret_cast<float*>(p.seg_out[seg]);
#pragma unroll 1
      for (int c = 0; c < BNH / 32; ++c) {
        float a[32];
        tc::tmem_ld32(t_addr + hf * BNH + c * 32, a);
        tc::tmem_ld_wait();
        __syncwarp();
#pragma unroll
        for (int v = 0; v < 8; ++v)
          *reinterpret_cast<float4*>(mine + v * 16) = make_float4(a[v * 4], a[v * 4 + 1], a[v * 4 + 2], a[v * 4 + 3]);
        __syncwarp();
        const int col = brow + c * 32 + q * 4;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int rr = 4 * i + rsub, grow = row0 + rr;
          if (grow < p.M && valid) {
            // h += acc as a reduction at the L2: one add per element (every element belongs to
            // exactly one tile) and nothing comes back to the SM, so the epilogue does not sit
            // through a load round trip per chunk
            const float4 a4 = *reinterpret_cast<const float4*>(stage + rr * EPI_PITCH + q * 16);
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(out + (size_t)grow * ldc + col), "f"(a4.x),
                         "f"(a4.y), "f"(a4.z), "f"(a4.w) : "memory");
          }
        }
      }
    } else {
      T* out = reinterpret_cast<T*>(p.seg_out[seg]);
#pragma unroll 1
      for (int c = 0; c < BNH / 32; ++c) {
        float a[32];
        tc::tmem_ld32(t_addr + hf * BNH + c * 32, a);
        tc::tmem_ld_wait();
        if ((c & 1) == 0) __syncwarp();
#pragma unroll
        for (int v = 0; v < 4; ++v) {
          float r[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) r[i] = a[v * 8 + i];
          st16(reinterpret_cast<T*>(mine + (c & 1) * 64 + v * 16), r);
        }
        if (c & 1) {
          __syncwarp();
          const int col = brow + (c - 1) * 32 + q * 8;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int rr = 4 * i + rsub, grow = row0 + rr;
            if (grow < p.M && valid)
              *reinterpret_cast<uint4*>(out + (size_t)grow * ldc + col) =
                  *reinterpret_cast<const uint4*>(stage + rr * EPI_PITCH + q * 16);
          }
        }
      }
    }
  }
}

template <int EPI, typename T>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
               const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint64_t* full = bars;                    // [STAGES]
  uint64_t* empty = bars + STAGES;          // [STAGES]
  uint64_t* acc_full = bars + 2 * STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;       // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = (p.K + BK - 1) / BK;
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int n_items = n_tiles * p.splits;
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { tc::mbar_init(&full[i], 1); tc::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], 4); }
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
  // Everything above touched only this CTA's own state.  From here on each role waits for the
  // kernels before this one (pdl_wait) right before its first access to memory they may have
  // written: the producer only before its first ACTIVATION tile - the weights are nobody's
  // output, so their first stages are already in flight while the predecessor drains.

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      tc::prefetch_tmap(&tmA);
      tc::prefetch_tmap(&tmB0);
      auto b_tiles = [&](int tile, const CUtensorMap*& m0, const CUtensorMap*& m1, int& row0, int& row1) {
        const int tn = tile / p.tiles_m;
        int seg0, seg1;
        if (EPI == EPI_SWIGLU) {
          seg0 = 0; seg1 = 1; row0 = row1 = tn * BNH;
        } else {
          locate(p, p.nh * tn, seg0, row0);
          locate(p, p.nh * tn + 1, seg1, row1);
        }
        m0 = seg0 == 0 ? &tmB0 : (seg0 == 1 ? &tmB1 : &tmB2);
        m1 = seg1 == 0 ? &tmB0 : (seg1 == 1 ? &tmB1 : &tmB2);
      };
      // weight tiles of the first stages (every stage is free at the start: no wait), then the
      // dependency on the earlier kernels, then the activation tiles of the same stages
      const uint32_t stage_tx = A_BYTES + p.nh * BH_BYTES;
      int tile0 = 0, kbf0 = 0, kbf1 = 0;                  // the CTA's first work item
      if (blockIdx.x < n_items) item_range(p, blockIdx.x, n_tiles, KB, tile0, kbf0, kbf1);
      const int pre = kbf1 - kbf0 < STAGES ? kbf1 - kbf0 : STAGES;
      if (pre > 0) {
        const CUtensorMap *m0, *m1;
        int row0, row1;
        b_tiles(tile0, m0, m1, row0, row1);
        for (int kb = 0; kb < pre; ++kb) {
          uint8_t* st = smem + kb * STAGE_BYTES;
          tc::mbar_expect_tx(&full[kb], stage_tx);
          tc::tma_load_2d(st + A_BYTES, m0, (kbf0 + kb) * BK, row0, &full[kb]);
          if (p.nh == 2) tc::tma_load_2d(st + A_BYTES + BH_BYTES, m1, (kbf0 + kb) * BK, row1, &full[kb]);
        }
      }
      pdl_wait();
      for (int kb = 0; kb < pre; ++kb)
        tc::tma_load_2d(smem + kb * STAGE_BYTES, &tmA, (kbf0 + kb) * BK, (tile0 % p.tiles_m) * BM, &full[kb]);
      int s = pre % STAGES;
      uint32_t ph = pre == STAGES ? 1u : 0u;
      int kb_start = pre;
      bool ok = true;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        int tile, kb0, kb1;
        item_range(p, item, n_tiles, KB, tile, kb0, kb1);
        const int tm = tile % p.tiles_m;
        const CUtensorMap *m0, *m1;
        int row0, row1;
        b_tiles(tile, m0, m1, row0, row1);
        for (int kb = kb0 + kb_start; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* st = smem + s * STAGE_BYTES;
          tc::mbar_expect_tx(&full[s], stage_tx);
          tc::tma_load_2d(st, &tmA, kb * BK, tm * BM, &full[s]);
          tc::tma_load_2d(st + A_BYTES, m0, kb * BK, row0, &full[s]);
          if (p.nh == 2) tc::tma_load_2d(st + A_BYTES + BH_BYTES, m1, kb * BK, row1, &full[s]);
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        kb_start = 0;
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc = p.idesc;
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      int it = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
        int tile, kb0, kb1;
        item_range(p, item, n_tiles, KB, tile, kb0, kb1);
        const int acc = it & 1;
        if (!tc::mbar_wait(&acc_empty[acc], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * (2 * BNH);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t a_addr = tc::smem_u32(smem + s * STAGE_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = tc::smem_desc_k_sw128(a_addr + k * 32);
            const uint64_t db = tc::smem_desc_k_sw128(b_addr + k * 32);
            tc::mma_f16(d_tmem, da, db, idesc, kb > kb0 || k != 0);
          }
          tc::mma_commit(&empty[s]);            // frees the stage once these MMAs retire
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        if (ok) tc::mma_commit(&acc_full[acc]);
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;                 // tensor-memory lane quadrant of this warp
    pdl_wait();                                // outputs, residual and positions are other kernels' memory
    bool ok = true;
    int it = 0;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++it) {
      const int tile = item % n_tiles;
      const int acc = it & 1;
      const int tn = tile / p.tiles_m, tm = tile % p.tiles_m;
      if (!tc::mbar_wait(&acc_full[acc], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      if (EPI == EPI_RESID && p.splits > 1 && !split_turn(p, item, n_tiles, lane, abort_flag)) { ok = false; break; }
      const uint32_t t_addr = tmem_base + acc * (2 * BNH) + ((uint32_t)(quad * 32) << 16);
      if (EPI == EPI_SWIGLU)
        epilogue_swiglu_row<T>(p, t_addr, tm * BM + quad * 32 + lane, tn);
      else
        epilogue_warp<EPI, T>(p, t_addr, tm * BM + quad * 32, lane, tn, p.nh,
                              smem + STAGES * STAGE_BYTES + 256 + (warp - 2) * EPI_STAGE_BYTES);
      if (EPI == EPI_RESID && p.splits > 1) split_done(p, tile, lane);
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&acc_empty[acc]);
    }
    if (!ok && lane == 0) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(200000);       // let loads already in flight land before the CTA exits
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc::fence_after_sync();
    tc::tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------
// The same GEMM on CTA pairs: a cluster of two CTAs (two SMs) works on one 256x256 tile with
// tcgen05.mma.cta_group::2.  Each CTA stages its own 128 rows of x and only ITS 128 of the
// tile's 256 weight rows (the pair's other half is read from the neighbour's shared memory by
// the tensor core), so a k slab costs 32 KB of L2 -> SM traffic per SM instead of 48 KB, and
// the ring is 6 stages deep.  Rank 0 issues the MMAs for both; each CTA holds the accumulator
// of its 128 rows (2 x 256 columns, double-buffered) and runs the same epilogue as above.
//   full[s]      rank 0's only: its producer announces the bytes of BOTH CTAs' slabs, both
//                producers' loads report there
//   empty[s]     one per CTA, signalled by one commit to both (the MMAs that read the stage)
//   acc_full[a]  one per CTA, signalled by one commit to both
//   acc_empty[a] rank 0's only: the 8 epilogue warps of the pair arrive there
// ---------------------------------------------------------------------------------------
constexpr int STAGES2 = 6;
constexpr int STAGE2_BYTES = A_BYTES + BH_BYTES;             // 32768 per CTA
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + 4 * EPI_STAGE_BYTES;
static_assert(SMEM2_BYTES <= 227 * 1024, "shared memory of the paired GEMM");
static_assert((2 * STAGES2 + 4) * 8 + 8 <= 256, "barrier block of the paired GEMM");

template <int EPI, typename T>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmB1, const __grid_constant__ CUtensorMap tmB2,
                    const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // the dynamic shared memory starts at the same offset in both CTAs, so the aligned ring does too
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES2 * STAGE2_BYTES);
  uint64_t* full = bars;                     // [STAGES2]
  uint64_t* empty = bars + STAGES2;          // [STAGES2]
  uint64_t* acc_full = bars + 2 * STAGES2;   // [2]
  uint64_t* acc_empty = acc_full + 2;        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();          // 0 issues the MMAs
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int KB = (p.K + BK - 1) / BK;
  const int n_tiles = p.tiles_m * p.tiles_n;            // tiles_m counts 256-row tiles here
  const int n_items = n_tiles * p.splits;
  pdl_trigger();

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES2; ++i) { tc::mbar_init(&full[i], 1); tc::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], 8); }
    *abort_flag = 0;
    tc::fence_barrier_init();
    tc::fence_proxy_async();
  }
  if (warp == 1) {
    tc::tmem_alloc_pair(tmem_slot, 512);
    tc::tmem_relinquish_pair();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();                    // the neighbour's barriers exist before anything is sent there
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      tc::prefetch_tmap(&tmA);
      tc::prefetch_tmap(&tmB0);
      // this CTA's half of the tile's weight rows: block 2 tn + rank of the concatenated columns
      auto b_half = [&](int tile, const CUtensorMap*& m, int& row) {
        const int tn = tile / p.tiles_m;
        int seg;
        if (EPI == EPI_SWIGLU) {
          seg = (int)rank; row = tn * BNH;
        } else {
          locate(p, 2 * tn + (int)rank, seg, row);
        }
        m = seg == 0 ? &tmB0 : (seg == 1 ? &tmB1 : &tmB2);
      };
      uint32_t full0[STAGES2];                // rank 0's full barriers as shared::cluster addresses
      for (int i = 0; i < STAGES2; ++i) full0[i] = tc::map_to_rank(tc::smem_u32(&full[i]), 0);
      int tile0 = 0, kbf0 = 0, kbf1 = 0;                  // the pair's first work item
      if (pair < n_items) item_range(p, pair, n_tiles, KB, tile0, kbf0, kbf1);
      const int pre = kbf1 - kbf0 < STAGES2 ? kbf1 - kbf0 : STAGES2;
      if (pre > 0) {
        const CUtensorMap* m;
        int row;
        b_half(tile0, m, row);
        for (int kb = 0; kb < pre; ++kb) {
          if (rank == 0) tc::mbar_expect_tx(&full[kb], 2 * STAGE2_BYTES);
          tc::tma_load_2d_pair(smem + kb * STAGE2_BYTES + A_BYTES, m, (kbf0 + kb) * BK, row, full0[kb]);
        }
      }
      pdl_wait();
      for (int kb = 0; kb < pre; ++kb)
        tc::tma_load_2d_pair(smem + kb * STAGE2_BYTES, &tmA, (kbf0 + kb) * BK, ((tile0 % p.tiles_m) * 2 + (int)rank) * BM,
                             full0[kb]);
      int s = pre % STAGES2;
      uint32_t ph = pre == STAGES2 ? 1u : 0u;
      int kb_start = pre;
      bool ok = true;
      for (int item = pair; item < n_items && ok; item += n_pairs) {
        int tile, kb0, kb1;
        item_range(p, item, n_tiles, KB, tile, kb0, kb1);
        const int tm = tile % p.tiles_m;
        const CUtensorMap* m;
        int row;
        b_half(tile, m, row);
        for (int kb = kb0 + kb_start; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* st = smem + s * STAGE2_BYTES;
          if (rank == 0) tc::mbar_expect_tx(&full[s], 2 * STAGE2_BYTES);
          tc::tma_load_2d_pair(st, &tmA, kb * BK, (tm * 2 + (int)rank) * BM, full0[s]);
          tc::tma_load_2d_pair(st + A_BYTES, m, kb * BK, row, full0[s]);
          if (++s == STAGES2) { s = 0; ph ^= 1; }
        }
        kb_start = 0;
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (rank 0 only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = p.idesc;
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      int it = 0;
      for (int item = pair; item < n_items && ok; item += n_pairs, ++it) {
        int tile, kb0, kb1;
        item_range(p, item, n_tiles, KB, tile, kb0, kb1);
        const int acc = it & 1;
        if (!tc::mbar_wait(&acc_empty[acc], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * (2 * BNH);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          const uint32_t a_addr = tc::smem_u32(smem + s * STAGE2_BYTES);
          const uint32_t b_addr = a_addr + A_BYTES;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            const uint64_t da = tc::smem_desc_k_sw128(a_addr + k * 32);
            const uint64_t db = tc::smem_desc_k_sw128(b_addr + k * 32);
            tc::mma_f16_pair(d_tmem, da, db, idesc, kb > kb0 || k != 0);
          }
          tc::mma_commit_pair(&empty[s], 3);            // frees the stage in both CTAs
          if (++s == STAGES2) { s = 0; ph ^= 1; }
        }
        if (ok) tc::mma_commit_pair(&acc_full[acc], 3);
      }
      if (!ok) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs)
    const int quad = warp & 3;
    const uint32_t acc_empty0[2] = {tc::map_to_rank(tc::smem_u32(&acc_empty[0]), 0),
                                    tc::map_to_rank(tc::smem_u32(&acc_empty[1]), 0)};
    pdl_wait();
    bool ok = true;
    int it = 0;
    for (int item = pair; item < n_items && ok; item += n_pairs, ++it) {
      const int tile = item % n_tiles;
      const int acc = it & 1;
      const int tn = tile / p.tiles_m, tm = tile % p.tiles_m;
      if (!tc::mbar_wait(&acc_full[acc], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      if (EPI == EPI_RESID && p.splits > 1 && !split_turn(p, item, n_tiles, lane, abort_flag)) { ok = false; break; }
      const uint32_t t_addr = tmem_base + acc * (2 * BNH) + ((uint32_t)(quad * 32) << 16);
      const int row0 = (tm * 2 + (int)rank) * BM + quad * 32;
      if (EPI == EPI_SWIGLU)
        epilogue_swiglu_row<T>(p, t_addr, row0 + lane, tn);
      else
        epilogue_warp<EPI, T>(p, t_addr, row0, lane, tn, 2,
                              smem + STAGES2 * STAGE2_BYTES + 256 + (warp - 2) * EPI_STAGE_BYTES);
      if (EPI == EPI_RESID && p.splits > 1) split_done(p, tile, lane);
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(acc_empty0[acc]);
    }
    if (!ok && lane == 0) { *abort_flag = 1; set_status(p.status, AKVS_ERR_TIMEOUT); }
  }

  // ---------------------------------------------------------------------- teardown
  if (*abort_flag) __nanosleep(200000);       // let loads already in flight land before the CTA exits
  tc::fence_before_sync();
  __syncthreads();
  tc::cluster_sync_all();                     // neither CTA's shared or tensor memory goes while the other may use it
  if (warp == 1) {
    tc::fence_after_sync();
    tc::tmem_dealloc_pair(tmem_base, 512);
  }
}

typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                             const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn get_encoder() {
  static EncodeFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeFn>(p);
  }
  return fn;
}

int g_sm_count = 0;
int sm_count() {
  if (!g_sm_count) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&g_sm_count, cudaDevAttrMultiProcessorCount, dev);
    if (g_sm_count <= 0) g_sm_count = 148;
  }
  return g_sm_count;
}

// Launch with clusters of two CTAs, as a programmatic dependent of the kernel before it.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_pair(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = 2;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// How many CTA pairs of the paired GEMM the device runs at once (0: none, use single CTAs).
int g_pair_count = -1;
int pair_count() {
  if (g_pair_count < 0) {
    g_pair_count = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * sm_count());
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = SMEM2_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_pair_kernel<EPI_STORE, f16>, &cfg) == cudaSuccess && n > 0)
      g_pair_count = n;
    else
      cudaGetLastError();
  }
  return g_pair_count;
}

}  // namespace

// A tensor map is a pure function of (base, rows, cols, ld, box): the maps of the weights and of
// the workspace's activation buffers recur on every layer call of every step, so they are
// encoded once per process and looked up afterwards (a few hundred driver calls per step
// otherwise).  Process-wide and, like the rest of the library's host state, not thread-safe.
namespace {
struct TmapKey {
  const void* base; uint64_t rows, cols, ld; uint32_t box;
  bool operator==(const TmapKey& o) const { return base == o.base && rows == o.rows && cols == o.cols && ld == o.ld && box == o.box; }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey& k) const {
    uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
    h ^= (k.rows + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2));
    h ^= (k.cols * 0xC2B2AE3D27D4EB4Full + (h << 6) + (h >> 2));
    h ^= (k.ld * 31 + k.box + (h << 6) + (h >> 2));
    return (size_t)h;
  }
};
std::unordered_map<TmapKey, CUtensorMap, TmapKeyHash> g_tmap_cache;
constexpr size_t kTmapCacheMax = 16384;
}  // namespace

int32_t encode_tmap_2d_16bit(CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t ld,
                            uint32_t box_rows) {
  EncodeFn enc = get_encoder();
  if (!enc) return AKVS_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld * 2) % 16 != 0) return AKVS_ERR_SHAPE;
  const TmapKey key{base, rows, cols, ld, box_rows};
  auto it = g_tmap_cache.find(key);
  if (it != g_tmap_cache.end()) {
    *map = it->second;
    return AKVS_OK;
  }
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld * 2};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return AKVS_ERR_CUDA;
  if (g_tmap_cache.size() >= kTmapCacheMax) g_tmap_cache.clear();
  g_tmap_cache.emplace(key, *map);
  return AKVS_OK;
}

int32_t encode_tmap_3d_16bit(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2, uint64_t ld1,
                            uint64_t ld2, uint32_t b1, uint32_t b2) {
  EncodeFn enc = get_encoder();
  if (!enc) return AKVS_ERR_CUDA;
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (ld1 * 2) % 16 != 0 || (ld2 * 2) % 16 != 0) return AKVS_ERR_SHAPE;
  const cuuint64_t dims[3] = {d0, d1, d2};
  const cuuint64_t strides[2] = {ld1 * 2, ld2 * 2};
  const cuuint32_t box[3] = {64, b1, b2};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AKVS_OK : AKVS_ERR_CUDA;
}

// x [M][K]; up to three weight matrices w[i] [n[i]][K] of the same 16-bit type (n[i] a multiple of 128) whose
// outputs go to out[i] with row stride ldc[i].
//   epi 0: out[i] = x w[i]^T (16-bit);   epi 1: out[0] (float) += x w[0]^T;
//   epi 2: out[0] = silu(x w[0]^T) * (x w[1]^T) (16-bit), n[0] == n[1].
// splits_force (epi 1 only): 0 = the k range is split by the cost model; 1..4 = that many splits.
int32_t launch_linear_tc(int dtype, int epi, const void* x, int M, int K, int n_seg, const void* const* w, const int* n,
                         void* const* out, const int* ldc, int32_t* status, cudaStream_t st, const float2* rope,
                         const int32_t* pos, int rope_mask, int tiling, int n_pos, int splits_force) {
  if (M == 0) return AKVS_OK;
  if (K % 8 != 0 || n_seg < 1 || n_seg > 3) return AKVS_ERR_SHAPE;
  if (dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  static bool attr_set = false;
  if (!attr_set) {
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_STORE, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_STORE, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_RESID, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_kernel<EPI_SWIGLU, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_STORE, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_RESID, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_SWIGLU, bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_STORE, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_RESID, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    AKVS_CUDA(cudaFuncSetAttribute(gemm_tc_pair_kernel<EPI_SWIGLU, f16>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES));
    attr_set = true;
  }
  GemmParams p;
  p.M = M;
  p.K = K;
  p.n_seg = n_seg;
  p.status = status;
  p.rope = rope;
  p.pos = pos;
  p.rope_mask = (epi == EPI_STORE && rope && pos && n_pos > 0) ? rope_mask : 0;
  p.n_pos = n_pos;
  const uint32_t fmt = dtype == AKVS_F16 ? tc::kF16 : tc::kBF16;
  CUtensorMap tmA, tmB[3];
  AKVS_TRY(encode_tmap_2d_16bit(&tmA, x, M, K, K, BM));
  int blocks = 0;
  for (int i = 0; i < 3; ++i) {
    const int s = i < n_seg ? i : 0;
    if (n[s] % BNH != 0) return AKVS_ERR_SHAPE;
    AKVS_TRY(encode_tmap_2d_16bit(&tmB[i], w[s], n[s], K, K, BNH));
    p.seg_blocks[i] = n[s] / BNH;
    p.seg_out[i] = out[i < n_seg && (epi != EPI_SWIGLU || i == 0) ? i : 0];
    p.seg_ldc[i] = ldc[i < n_seg && (epi != EPI_SWIGLU || i == 0) ? i : 0];
    if (i < n_seg) blocks += n[s] / BNH;
  }
  p.tiles_m = (M + BM - 1) / BM;
  p.nh = 2;
  p.splits = 1;
  p.split_count = nullptr;
  p.split_warps = 4;
  const int KB = (K + BK - 1) / BK;
  p.kb_split = KB;
  const int sms = sm_count();
  // CTA pairs on 256x256 tiles: a tile takes the same number of MMA cycles as two 128x256 tiles
  // of single CTAs, and the pair moves a third less operand data per SM (measured on the 8B
  // shapes: main loop ~8 % faster under the power cap).  tiling 1 / 2 force single CTAs / pairs
  // (tests, comparisons).
  const int pairs = (tiling == 1 || M <= BM) ? 0 : pair_count();
  bool use_pair = false;
  if (epi == EPI_SWIGLU) {
    if (n_seg != 2 || n[0] != n[1]) return AKVS_ERR_SHAPE;
    p.tiles_n = n[0] / BNH;
  } else if (epi == EPI_RESID) {
    // The residual epilogue adds into h at the L2, so the k range may be split over several work
    // items at no extra pass.  Cost model in units of one 128x256x64 slab on one SM: rounds x
    // (slabs per item x cost of a slab on that tiling + a per-item constant); a 128x128 tile's slab
    // costs 0.62 (it reads as many shared-memory bytes per flop again), a pair's 0.92 per SM.
    // A split keeps at least 32 slabs per item, so that an item's epilogue still fits under the
    // next item's main loop; more splits must win by 3 % each.
    double best = 1e30;
    for (int pr = 0; pr < 2; ++pr) {
      if (pr == 1 && pairs == 0) continue;
      if (pr == 0 && tiling == 2 && pairs > 0) continue;
      for (int nh = 1; nh <= 2; ++nh) {
        if (pr == 1 && nh == 1) continue;
        const int tiles = (pr ? (M + 2 * BM - 1) / (2 * BM) : p.tiles_m) * ((blocks + nh - 1) / nh);
        const int cap = pr ? pairs : sms;
        const double slab = pr ? 0.92 : (nh == 2 ? 1.0 : 0.62);
        for (int sp = 1; sp <= 4; ++sp) {
          if (splits_force > 0 && sp != splits_force) continue;
          const int kbs = (KB + sp - 1) / sp;
          if ((kbs + 0) * (sp - 1) >= KB && sp > 1) continue;      // the last split would be empty
          if (splits_force == 0 && sp > 1 && kbs < AKVS_SPLIT_MIN_KB) continue;
          const int rounds = (tiles * sp + cap - 1) / cap;
          const double cost = rounds * (kbs * slab + 4.0) * (1.0 + 0.03 * (sp - 1));
          if (cost < best) {
            best = cost;
            use_pair = pr == 1;
            p.nh = nh;
            p.splits = sp;
            p.kb_split = kbs;
          }
        }
      }
    }
    if (best >= 1e30) return AKVS_ERR_SHAPE;                     // a forced split count the k range cannot carry
    p.tiles_n = (blocks + p.nh - 1) / p.nh;
    if (p.splits > 1) {
      const int tiles = (use_pair ? (M + 2 * BM - 1) / (2 * BM) : p.tiles_m) * p.tiles_n;
      static unsigned int* counters[64] = {};
      int dev = 0;
      AKVS_CUDA(cudaGetDevice(&dev));
      if (tiles > SPLITK_MAX_TILES || dev < 0 || dev >= 64) {
        if (splits_force > 1) return AKVS_ERR_TOO_LARGE;
        p.splits = 1;                                           // (only reachable with the tiling the model chose for 1 split
        p.kb_split = KB;                                        //  being worse than another: correct, just not the fastest)
      } else {
        if (!counters[dev]) AKVS_CUDA(cudaGetSymbolAddress(reinterpret_cast<void**>(&counters[dev]), g_splitk_count));
        p.split_count = counters[dev];
        p.split_warps = use_pair ? 8 : 4;
      }
    }
  } else {
    // 128x128 tiles when that shortens the launch: a tile of half the width takes ~0.62 of the
    // time, rounds = tiles / SMs
    const int t2 = p.tiles_m * ((blocks + 1) / 2), t1 = p.tiles_m * blocks;
    const double cost2 = (double)((t2 + sms - 1) / sms), cost1 = 0.62 * ((t1 + sms - 1) / sms);
    if (cost1 < 0.9 * cost2) p.nh = 1;
    p.tiles_n = (blocks + p.nh - 1) / p.nh;
  }
  if (epi != EPI_RESID && (p.nh == 2 || tiling == 2) && pairs > 0) {
    // pairs when that takes no more rounds than single CTAs on 128x256 tiles
    const int tiles_n2 = (blocks + 1) / 2;
    const int tn = epi == EPI_SWIGLU ? p.tiles_n : tiles_n2;
    const int t_pair = ((M + 2 * BM - 1) / (2 * BM)) * tn, t_single = p.tiles_m * tn;
    const int r_pair = (t_pair + pairs - 1) / pairs, r_single = (t_single + sms - 1) / sms;
    if (tiling == 2 || r_pair <= r_single) {
      use_pair = true;
      if (p.nh == 1) { p.nh = 2; p.tiles_n = tiles_n2; }
    }
  }
  double flops = 0;
  for (int i = 0; i < n_seg; ++i) flops += 2.0 * M * (double)n[i] * K;
  ProfScope prof(1, epi, flops, st);
  if (epi < 0 || epi > 2) return AKVS_ERR_INVALID_ARG;
  if (use_pair) {
    p.tiles_m = (M + 2 * BM - 1) / (2 * BM);
    p.idesc = tc::idesc_f16(fmt, 2 * BM, 2 * BNH, 0);
    const int items = p.tiles_m * p.tiles_n * p.splits;
    const int n_pairs = items < pairs ? items : pairs;
#define AKVS_GEMM_LAUNCH(E, T) \
  AKVS_CUDA(launch_pdl_pair(gemm_tc_pair_kernel<E, T>, dim3(2 * n_pairs), dim3(THREADS), SMEM2_BYTES, st, tmA, tmB[0], tmB[1], tmB[2], p))
    if (dtype == AKVS_BF16) {
      if (epi == EPI_STORE) AKVS_GEMM_LAUNCH(EPI_STORE, bf16);
      else if (epi == EPI_RESID) AKVS_GEMM_LAUNCH(EPI_RESID, bf16);
      else AKVS_GEMM_LAUNCH(EPI_SWIGLU, bf16);
    } else {
      if (epi == EPI_STORE) AKVS_GEMM_LAUNCH(EPI_STORE, f16);
      else if (epi == EPI_RESID) AKVS_GEMM_LAUNCH(EPI_RESID, f16);
      else AKVS_GEMM_LAUNCH(EPI_SWIGLU, f16);
    }
#undef AKVS_GEMM_LAUNCH
    AKVS_LAUNCHED();
    return AKVS_OK;
  }
  p.idesc = tc::idesc_f16(fmt, BM, p.nh * BNH, 0);
  const int n_items = p.tiles_m * p.tiles_n * p.splits;
  const int grid = n_items < sm_count() ? n_items : sm_count();
#define AKVS_GEMM_LAUNCH(E, T) \
  AKVS_CUDA(launch_pdl(gemm_tc_kernel<E, T>, dim3(grid), dim3(THREADS), SMEM_BYTES, st, tmA, tmB[0], tmB[1], tmB[2], p))
  if (dtype == AKVS_BF16) {
    if (epi == EPI_STORE) AKVS_GEMM_LAUNCH(EPI_STORE, bf16);
    else if (epi == EPI_RESID) AKVS_GEMM_LAUNCH(EPI_RESID, bf16);
    else AKVS_GEMM_LAUNCH(EPI_SWIGLU, bf16);
  } else {
    if (epi == EPI_STORE) AKVS_GEMM_LAUNCH(EPI_STORE, f16);
    else if (epi == EPI_RESID) AKVS_GEMM_LAUNCH(EPI_RESID, f16);
    else AKVS_GEMM_LAUNCH(EPI_SWIGLU, f16);
  }
#undef AKVS_GEMM_LAUNCH
  AKVS_LAUNCHED();
  return AKVS_OK;
}
