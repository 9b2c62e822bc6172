// Shared device/host helpers for the akvs kernels (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "akvs.h"

typedef __nv_bfloat16 bf16;
typedef __half f16;

// Model dtypes: AKVS_F32 (everything float), AKVS_BF16 and AKVS_F16 (weights, unit cache,
// activations and K/V outputs in that 16-bit type).  Accumulation, the residual stream,
// softmax, norms, offsets and scores are float in every mode.  The tensor cores take either
// 16-bit type at the same rate, but both operands of one MMA must have the same type.
#define AKVS_TRY(expr)                              \
  do {                                              \
    int32_t rc_ = (expr);                           \
    if (rc_ != AKVS_OK) return rc_;                 \
  } while (0)

#define AKVS_CUDA(expr)                             \
  do {                                              \
    if ((expr) != cudaSuccess) return AKVS_ERR_CUDA; \
  } while (0)

// Every kernel launch of the library goes through this: it counts the launch (the count is
// what akvs_launch_count reports) and turns a launch failure into an error code.
extern unsigned long long g_akvs_launches;
#define AKVS_LAUNCHED()                             \
  do {                                              \
    ++g_akvs_launches;                              \
    if (cudaPeekAtLastError() != cudaSuccess) return AKVS_ERR_CUDA; \
  } while (0)

// Optional per-launch timing of one kernel class with CUDA events on the launching stream
// (akvs_prof_*).  kind: 1 = tensor-core linear layers, 2 = correction pass, 3 = attention.
void akvs_prof_mark(int kind, int sub, double work, bool begin, cudaStream_t st);
struct ProfScope {
  int kind, sub; double work; cudaStream_t st;
  ProfScope(int k, int s, double w, cudaStream_t t) : kind(k), sub(s), work(w), st(t) { akvs_prof_mark(k, s, w, true, t); }
  ~ProfScope() { akvs_prof_mark(kind, sub, work, false, st); }
};

#include <type_traits>
// Calls f(T{}) with T = float | bf16 | f16 for the model dtype.
template <typename F>
static inline int32_t dispatch_dtype(int dtype, F&& f) {
  switch (dtype) {
    case AKVS_F32: return f(float{});
    case AKVS_BF16: return f(bf16{});
    case AKVS_F16: return f(f16{});
    default: return AKVS_ERR_UNSUPPORTED;
  }
}
// Calls f(std::integral_constant<int, FMT>{}) for the cache format.
template <typename F>
static inline int32_t dispatch_fmt(int fmt, F&& f) {
  switch (fmt) {
    case AKVS_KV_NATIVE: return f(std::integral_constant<int, AKVS_KV_NATIVE>{});
    case AKVS_KV_Q4: return f(std::integral_constant<int, AKVS_KV_Q4>{});
    case AKVS_KV_Q2: return f(std::integral_constant<int, AKVS_KV_Q2>{});
    case AKVS_KV_FP8: return f(std::integral_constant<int, AKVS_KV_FP8>{});
    default: return AKVS_ERR_UNSUPPORTED;
  }
}
static inline size_t dtype_size(int dtype) { return dtype == AKVS_F32 ? 4 : 2; }

static inline int64_t akvs_align_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }
static inline int akvs_cdiv(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

// ---------------------------------------------------------------------------------------
// 16-byte vector access: VEC elements of T <-> float registers.
// ---------------------------------------------------------------------------------------
template <typename T> struct VecOf;
template <> struct VecOf<float> { static constexpr int N = 4; };
template <> struct VecOf<bf16> { static constexpr int N = 8; };
template <> struct VecOf<f16> { static constexpr int N = 8; };

__device__ __forceinline__ void ld16(const float* p, float (&o)[4]) {
  float4 v = *reinterpret_cast<const float4*>(p);
  o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
}
__device__ __forceinline__ void st16(float* p, const float (&o)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ void ld16(const bf16* p, float (&o)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o[2 * i] = __uint_as_float(w[i] << 16);
    o[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);   // .x = a (low half), .y = b
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void st16(bf16* p, const float (&o)[8]) {
  uint4 v;
  v.x = pack_bf16x2(o[0], o[1]);
  v.y = pack_bf16x2(o[2], o[3]);
  v.z = pack_bf16x2(o[4], o[5]);
  v.w = pack_bf16x2(o[6], o[7]);
  *reinterpret_cast<uint4*>(p) = v;
}

__device__ __forceinline__ void ld16(const f16* p, float (&o)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
    o[2 * i] = f.x;
    o[2 * i + 1] = f.y;
  }
}
// float -> half with saturation to the largest finite value (no infinities are produced):
// one cvt for two values; the first operand of the instruction lands in the upper half
__device__ __forceinline__ uint32_t pack_f16x2(float a, float b) {
  uint32_t r;
  asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
  return r;
}
__device__ __forceinline__ void st16(f16* p, const float (&o)[8]) {
  uint4 v;
  v.x = pack_f16x2(o[0], o[1]);
  v.y = pack_f16x2(o[2], o[3]);
  v.z = pack_f16x2(o[4], o[5]);
  v.w = pack_f16x2(o[6], o[7]);
  *reinterpret_cast<uint4*>(p) = v;
}

template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<bf16>(float a, float b) { return pack_bf16x2(a, b); }
template <> __device__ __forceinline__ uint32_t pack2<f16>(float a, float b) { return pack_f16x2(a, b); }

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(f16 x) { return __half2float(x); }
__device__ __forceinline__ float to_f(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float x) { return __float2bfloat16_rn(x); }
template <> __device__ __forceinline__ f16 from_f<f16>(float x) {
  const uint32_t r = pack_f16x2(x, 0.f);
  return __ushort_as_half((unsigned short)(r & 0xFFFFu));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
  return v;
}

// Programmatic dependent launch: a kernel launched with launch_pdl() may be scheduled while
// the kernel before it in the stream is still draining, so that its launch latency and its
// local prologue (barrier set-up, tensor-memory allocation, descriptor prefetch) overlap the
// predecessor's tail.  Such a kernel calls pdl_trigger() first thing (its own successor may be
// scheduled as soon as SM resources free up) and pdl_wait() before its first access to global
// memory that an earlier kernel may have written or may still read: the wait returns when every
// earlier kernel has completed and its writes are visible.  Both are no-ops under a plain launch.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Device status word: first error wins.
__device__ __forceinline__ void set_status(int32_t* status, int32_t code) {
  if (status) atomicCAS(status, 0, code);
}

// ---------------------------------------------------------------------------------------
// Internal launchers (host).  All take the model dtype as a runtime value.
// ---------------------------------------------------------------------------------------
struct KvLayer {            // one layer of a unit store, as the correction kernels read it
  const void* k;
  const void* v;
  const void* k_meta;       // half2 (scale, min) per 64-group, or null
  const void* v_meta;
  int fmt;                  // AKVS_KV_NATIVE | AKVS_KV_Q2 | AKVS_KV_Q4
};

struct ReqMaps {            // per-request index maps (device)
  const int32_t* ctx_off;   // [M+1]
  const int32_t* unit_pos;  // [M] position of a unit's first token within its own request (= ctx_off for one request)
  const int32_t* tok_unit;  // [N] unit slot of context token j
  const int32_t* tok_src;   // [N] row of token j in the unit store
  const int32_t* row_of_pos;// [T] index into the recomputed rows, or -1
  const uint8_t* kflag;     // [N] 1 if j in S^K
  const uint8_t* vflag;     // [N]
  const int4* tok_meta;     // [2][T] K records, then V records: (store row, fresh row or -1, unit slot, weight bits)
};

int32_t launch_embed(int dtype, const void* tok_emb, const int32_t* ids, const int32_t* gather, int n, int d,
                     int vocab, int32_t* status, float* h, cudaStream_t st);
int32_t launch_gather_rows(const float* src, const int32_t* rows, int n, int d, int n_src, int32_t* status, float* dst,
                           cudaStream_t st);
int32_t launch_rmsnorm(int out_dtype, const float* h, const float* gain, float eps, int n, int d, void* x,
                       cudaStream_t st);
int32_t launch_rope_table(float base, int hd, int n_pos, float2* table, cudaStream_t st);
int32_t launch_rope(int dtype, void* x, const int32_t* pos, int n, int n_heads, int hd, int ld,
                    const float2* table, int n_pos, int32_t* status, float base, cudaStream_t st);
int32_t launch_iota(int32_t* p, int n, int start, cudaStream_t st);
int32_t launch_quantize(int dtype, const void* x, int n, int n_kv, int hd, int bits, void* codes, void* meta,
                        cudaStream_t st);

int32_t launch_linear_simt(int dtype, const void* x, const void* w, const void* w2, void* y, float* resid,
                           int M, int N, int K, int ldy, cudaStream_t st);

// 16-bit tensor-core linear layers (gemm_tc.cu), dtype AKVS_BF16 or AKVS_F16.  epi 0: out[i] = x w[i]^T; 1: out[0] (float) += x w[0]^T;
// 2: out[0] = silu(x w[0]^T) * (x w[1]^T).
// With epi 0, segments whose bit is set in rope_mask (heads of 128 columns) are rotated through
// rope[pos[row]] in the epilogue (rope: [n_pos][64] (cos, sin); null = no rotation; a position
// outside [0, n_pos) raises AKVS_ERR_INVALID_ARG in the status word and rotates by position 0).
// tiling 0: single CTAs or CTA pairs, whichever the shape favours; 1: single CTAs; 2: pairs (M > 128).
// splits_force (epi 1): 0 = the k range is split over work items where a cost model favours it
// (launches that would leave SMs idle); 1..4 = exactly that many splits.
int32_t launch_linear_tc(int dtype, int epi, const void* x, int M, int K, int n_seg, const void* const* w, const int* n,
                         void* const* out, const int* ldc, int32_t* status, cudaStream_t st,
                         const float2* rope = nullptr, const int32_t* pos = nullptr, int rope_mask = 0, int tiling = 0,
                         int n_pos = 0, int splits_force = 0);

// tcgen05 attention (attn_tc.cu): 16-bit types, head_dim 128.
int32_t launch_attention_tc(int dtype, const void* q, const void* k, const void* v, void* out, const int32_t* k_lo,
                            const int32_t* k_hi, const int32_t* k_lo2, const int32_t* k_hi2, int R, int T, int n_q,
                            int n_kv, int32_t* status, cudaStream_t st);
int32_t launch_attention_simt(int dtype, const void* q, const void* k, const void* v, void* out,
                              const int32_t* k_lo, const int32_t* k_hi, const int32_t* k_lo2, const int32_t* k_hi2,
                              int R, int n_q, int n_kv, int hd, cudaStream_t st);

int32_t launch_tok_maps(const int32_t* ctx_off, const int32_t* slot_src_off, int M, int N, int32_t* tok_unit,
                        int32_t* tok_src, cudaStream_t st);
int32_t launch_row_maps(const int32_t* rows, int n_rows, const int32_t* sk_idx, const int32_t* sv_idx, int n_probe,
                        int N, int T, int32_t* row_of_pos, uint8_t* kflag, uint8_t* vflag, cudaStream_t st);
int32_t launch_tok_meta(const int32_t* tok_unit, const int32_t* tok_src, const int32_t* row_of_pos,
                        const uint8_t* kflag, const uint8_t* vflag, const float* w_k, const float* w_v, int N, int T,
                        int n_probe_rows, int4* tok_meta /*[2][T]*/, cudaStream_t st);
int32_t launch_scores(int dtype, const KvLayer& kv, const ReqMaps& maps, const void* k_fresh, const void* v_fresh,
                      int N, int n_kv, int hd, const float2* table, float* d_k, float* d_v, cudaStream_t st);
int32_t launch_select(const float* d_k, const float* d_v, const int32_t* ctx_off, const int32_t* probe_off, int M,
                      int N, int n_query, int32_t* sk_idx, int32_t* sv_idx, float* w_k, float* w_v, int32_t* rows,
                      uint64_t* keys /*[2N]*/, uint8_t* flags /*[2N]*/, int32_t* counts /*[2]*/, int32_t* status,
                      cudaStream_t st);
int32_t launch_offsets(int dtype, const KvLayer& kv, const ReqMaps& maps, const int32_t* probe_off,
                       const int32_t* sk_idx, const int32_t* sv_idx, const void* k_fresh, const void* v_fresh, int M,
                       int N, int n_probe_cap, int n_kv, int hd, const float2* table, float* mu_k, float* mu_v,
                       int32_t* status, cudaStream_t st);
int32_t launch_residual_stats(int dtype, const KvLayer& kv, const int32_t* ctx_off, const int32_t* tok_src,
                              const void* k_fresh, const void* v_fresh, int M, int n_kv, int hd, const float2* table,
                              const float* sel_k, const float* sel_v, const float* mu_k, const float* mu_v,
                              const float* w_k, const float* w_v, float* mean_k, float* mean_v, float* energy,
                              cudaStream_t st);
// weighted = false: no offsets are added (direct reuse); the weights themselves ride in tok_meta
int32_t launch_correct(int dtype, const KvLayer& kv, const ReqMaps& maps, const void* k_fresh, const void* v_fresh,
                       bool weighted, const float* mu_k, const float* mu_v, int N, int n_query, int n_kv, int hd,
                       const float2* table, void* out_k, void* out_v, cudaStream_t st);
