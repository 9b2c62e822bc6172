// Probe selection, per-unit offset estimation and the correction pass
// (paper Section 3.3 and Algorithm 1 lines 2, 5-8).
//
// Layouts: fresh rows [n_rows][n_kv][hd] (type T); one layer of the unit store
// [store_tok][n_kv][hd] (type TW, equal to T in every shipped configuration) or packed 2/4-bit codes with half2 (scale, min) per 64-dim group;
// outputs [T][n_kv][hd].  A "pair chunk" is a 16-byte vector of the lower half of a head
// together with its RoPE partner 16 bytes in the upper half; one thread owns one pair chunk
// so that the re-alignment rotation needs no exchange between threads and every global
// access is a full 16-byte vector.
#include "common.cuh"
#include <cuda_fp8.h>

// ---------------------------------------------------------------------------------------
// Reading one pair chunk of the reused K or V of store row `src`, head `h`, chunk `c`.
// ---------------------------------------------------------------------------------------
// Eight (or four) FP8 E4M3 bytes -> floats (E4M3 values are exact in float16).
template <int V>
__device__ __forceinline__ void ld_fp8(const uint8_t* p, float (&out)[V]) {
  uint32_t w[V / 4];
  if constexpr (V == 8) {
    const uint2 t = *reinterpret_cast<const uint2*>(p);
    w[0] = t.x; w[1] = t.y;
  } else {
    w[0] = *reinterpret_cast<const uint32_t*>(p);
  }
#pragma unroll
  for (int i = 0; i < V / 2; ++i) {
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)((w[i >> 1] >> (16 * (i & 1))) & 0xFFFFu), __NV_E4M3);
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&h));
    out[2 * i] = f.x; out[2 * i + 1] = f.y;
  }
}

template <int BYTES>
__device__ __forceinline__ uint32_t ld_codes(const uint8_t* p) {
  if constexpr (BYTES == 4) return *reinterpret_cast<const uint32_t*>(p);
  else if constexpr (BYTES == 2) return *reinterpret_cast<const uint16_t*>(p);
  else return *p;
}

template <typename T, int FMT>
__device__ __forceinline__ void load_cached_chunk(const void* base, const void* meta, int64_t src, int n_kv, int hd,
                                                  int h, int dim0, float (&out)[VecOf<T>::N]) {
  constexpr int V = VecOf<T>::N;
  if constexpr (FMT == AKVS_KV_NATIVE) {
    ld16(reinterpret_cast<const T*>(base) + ((size_t)src * n_kv + h) * hd + dim0, out);
  } else if constexpr (FMT == AKVS_KV_FP8) {
    ld_fp8<V>(reinterpret_cast<const uint8_t*>(base) + ((size_t)src * n_kv + h) * hd + dim0, out);
  } else {
    constexpr int BITS = FMT;
    constexpr int BYTES = V * BITS / 8;
    const uint8_t* cp = reinterpret_cast<const uint8_t*>(base) + (((size_t)src * n_kv + h) * hd + dim0) * BITS / 8;
    const uint32_t packed = ld_codes<BYTES>(cp);
    const __half2 sm = reinterpret_cast<const __half2*>(meta)[((size_t)src * n_kv + h) * (hd / 64) + dim0 / 64];
    const float s = __low2float(sm), m = __high2float(sm);
#pragma unroll
    for (int i = 0; i < V; ++i)
      out[i] = __fmaf_rn((float)((packed >> (BITS * i)) & ((1u << BITS) - 1u)), s, m);
  }
}

// V consecutive floats / float2 as 16-byte loads (the addresses are 16-byte aligned by layout)
template <int V>
__device__ __forceinline__ void ld_f(const float* p, float (&o)[V]) {
#pragma unroll
  for (int i = 0; i < V; i += 4) {
    const float4 t = *reinterpret_cast<const float4*>(p + i);
    o[i] = t.x; o[i + 1] = t.y; o[i + 2] = t.z; o[i + 3] = t.w;
  }
}
template <int V>
__device__ __forceinline__ void ld_f2(const float2* p, float2 (&o)[V]) {
#pragma unroll
  for (int i = 0; i < V; i += 2) {
    const float4 t = *reinterpret_cast<const float4*>(p + i);
    o[i] = make_float2(t.x, t.y); o[i + 1] = make_float2(t.z, t.w);
  }
}

// ---------------------------------------------------------------------------------------
// Index maps of a request.
// ---------------------------------------------------------------------------------------
__global__ void tok_maps_kernel(const int32_t* __restrict__ ctx_off, const int32_t* __restrict__ slot_src_off, int M,
                                int N, int32_t* __restrict__ tok_unit, int32_t* __restrict__ tok_src) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= N) return;
  int lo = 0, hi = M;                 // largest u with ctx_off[u] <= j (empty units skipped)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (ctx_off[mid] <= j) lo = mid; else hi = mid;
  }
  tok_unit[j] = lo;
  tok_src[j] = slot_src_off[lo] + (j - ctx_off[lo]);
}

int32_t launch_tok_maps(const int32_t* ctx_off, const int32_t* slot_src_off, int M, int N, int32_t* tok_unit,
                        int32_t* tok_src, cudaStream_t st) {
  if (N == 0) return AKVS_OK;
  tok_maps_kernel<<<akvs_cdiv(N, 256), 256, 0, st>>>(ctx_off, slot_src_off, M, N, tok_unit, tok_src);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

__global__ void row_maps_clear_kernel(int N, int T, int32_t* __restrict__ row_of_pos, uint8_t* __restrict__ kflag,
                                      uint8_t* __restrict__ vflag) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < T) row_of_pos[j] = -1;
  if (j < N) { kflag[j] = 0; vflag[j] = 0; }
}
__global__ void row_maps_fill_kernel(const int32_t* __restrict__ rows, int n_rows, const int32_t* __restrict__ sk_idx,
                                     const int32_t* __restrict__ sv_idx, int n_probe, int N, int T,
                                     int32_t* __restrict__ row_of_pos, uint8_t* __restrict__ kflag,
                                     uint8_t* __restrict__ vflag) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_rows) { const int p = rows[i]; if (p >= 0 && p < T) row_of_pos[p] = i; }
  if (i < n_probe) {
    const int a = sk_idx[i], b = sv_idx[i];
    if (a >= 0 && a < N) kflag[a] = 1;
    if (b >= 0 && b < N) vflag[b] = 1;
  }
}

// Per-token records of the correction pass, one array for K and one for V ([2][T]):
//   (store row, fresh row or -1, unit slot, bits of the weight w)
// A token in S^K (S^V) takes its fresh K (V) row; query tokens take both from the fresh rows
// that follow the probes.  The weights are fixed after selection, so they ride in the record
// and the correction pass makes one 16-byte load per token and role.
__global__ void tok_meta_kernel(const int32_t* __restrict__ tok_unit, const int32_t* __restrict__ tok_src,
                                const int32_t* __restrict__ row_of_pos, const uint8_t* __restrict__ kflag,
                                const uint8_t* __restrict__ vflag, const float* __restrict__ w_k,
                                const float* __restrict__ w_v, int N, int T, int n_probe_rows,
                                int4* __restrict__ tok_meta) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= T) return;
  if (j >= N) {
    const int r = n_probe_rows + (j - N);
    tok_meta[j] = make_int4(-1, r, 0, 0);
    tok_meta[(size_t)T + j] = make_int4(-1, r, 0, 0);
  } else {
    const int r = row_of_pos[j];
    tok_meta[j] = make_int4(tok_src[j], kflag[j] ? r : -1, tok_unit[j], __float_as_int(w_k ? w_k[j] : 0.f));
    tok_meta[(size_t)T + j] = make_int4(tok_src[j], vflag[j] ? r : -1, tok_unit[j], __float_as_int(w_v ? w_v[j] : 0.f));
  }
}

int32_t launch_tok_meta(const int32_t* tok_unit, const int32_t* tok_src, const int32_t* row_of_pos,
                        const uint8_t* kflag, const uint8_t* vflag, const float* w_k, const float* w_v, int N, int T,
                        int n_probe_rows, int4* tok_meta, cudaStream_t st) {
  if (T == 0) return AKVS_OK;
  tok_meta_kernel<<<akvs_cdiv(T, 256), 256, 0, st>>>(tok_unit, tok_src, row_of_pos, kflag, vflag, w_k, w_v, N, T,
                                                    n_probe_rows, tok_meta);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

int32_t launch_row_maps(const int32_t* rows, int n_rows, const int32_t* sk_idx, const int32_t* sv_idx, int n_probe,
                        int N, int T, int32_t* row_of_pos, uint8_t* kflag, uint8_t* vflag, cudaStream_t st) {
  if (T == 0) return AKVS_OK;
  row_maps_clear_kernel<<<akvs_cdiv(T, 256), 256, 0, st>>>(N, T, row_of_pos, kflag, vflag);
  AKVS_LAUNCHED();
  const int m = n_rows > n_probe ? n_rows : n_probe;
  if (m > 0) {
    row_maps_fill_kernel<<<akvs_cdiv(m, 256), 256, 0, st>>>(rows, n_rows, sk_idx, sv_idx, n_probe, N, T, row_of_pos,
                                                            kflag, vflag);
    AKVS_LAUNCHED();
  }
  return AKVS_OK;
}

// ---------------------------------------------------------------------------------------
// Divergence scores at the check layer (Section 3.3): one warp per context token,
// d_K = || k_fresh - Rot(off_u) k_cached ||_2 over all kv heads, d_V likewise.
// ---------------------------------------------------------------------------------------
template <typename T, typename TW, int FMT>
__global__ void scores_kernel(KvLayer kv, ReqMaps maps, const T* __restrict__ k_fresh, const T* __restrict__ v_fresh,
                              int N, int n_kv, int hd, const float2* __restrict__ table, float* __restrict__ d_k,
                              float* __restrict__ d_v) {
  constexpr int V = VecOf<T>::N;
  const int j = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (j >= N) return;
  const int lane = threadIdx.x & 31;
  const int half = hd / 2, ch = half / V;
  const int u = maps.tok_unit[j];
  const int64_t src = maps.tok_src[j];
  const float2* rot = table + (size_t)maps.unit_pos[u] * half;
  float sk = 0.f, sv = 0.f;
  for (int pc = lane; pc < n_kv * ch; pc += 32) {
    const int h = pc / ch, c = pc % ch;
    float lo[V], hi[V], flo[V], fhi[V];
    load_cached_chunk<TW, FMT>(kv.k, kv.k_meta, src, n_kv, hd, h, c * V, lo);
    load_cached_chunk<TW, FMT>(kv.k, kv.k_meta, src, n_kv, hd, h, half + c * V, hi);
    const T* fp = k_fresh + ((size_t)j * n_kv + h) * hd + c * V;
    ld16(fp, flo);
    ld16(fp + half, fhi);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const float2 t = rot[c * V + i];
      const float a = flo[i] - (lo[i] * t.x - hi[i] * t.y);
      const float b = fhi[i] - (hi[i] * t.x + lo[i] * t.y);
      sk += a * a + b * b;
    }
    load_cached_chunk<TW, FMT>(kv.v, kv.v_meta, src, n_kv, hd, h, c * V, lo);
    load_cached_chunk<TW, FMT>(kv.v, kv.v_meta, src, n_kv, hd, h, half + c * V, hi);
    const T* vp = v_fresh + ((size_t)j * n_kv + h) * hd + c * V;
    ld16(vp, flo);
    ld16(vp + half, fhi);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      const float a = flo[i] - lo[i], b = fhi[i] - hi[i];
      sv += a * a + b * b;
    }
  }
  sk = warp_sum(sk);
  sv = warp_sum(sv);
  if (lane == 0) { d_k[j] = sqrtf(sk); d_v[j] = sqrtf(sv); }
}

static int32_t check_kv_shape(int dtype, const KvLayer& kv, int hd) {
  const int V = dtype == AKVS_F32 ? 4 : 8;
  if (hd % (2 * V) != 0) return AKVS_ERR_UNSUPPORTED;
  if (kv.fmt != AKVS_KV_NATIVE && kv.fmt != AKVS_KV_Q4 && kv.fmt != AKVS_KV_Q2 && kv.fmt != AKVS_KV_FP8)
    return AKVS_ERR_UNSUPPORTED;
  if ((kv.fmt == AKVS_KV_Q4 || kv.fmt == AKVS_KV_Q2) && (hd % 64 != 0 || !kv.k_meta || !kv.v_meta))
    return AKVS_ERR_UNSUPPORTED;
  return AKVS_OK;
}

int32_t launch_scores(int dtype, const KvLayer& kv, const ReqMaps& maps, const void* k_fresh, const void* v_fresh,
                      int N, int n_kv, int hd, const float2* table, float* d_k, float* d_v, cudaStream_t st) {
  if (N == 0) return AKVS_OK;
  AKVS_TRY(check_kv_shape(dtype, kv, hd));
  const int grid = akvs_cdiv(N, 8);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    return dispatch_fmt(kv.fmt, [&](auto f) -> int32_t {
      scores_kernel<T, T, decltype(f)::value><<<grid, 256, 0, st>>>(kv, maps, (const T*)k_fresh, (const T*)v_fresh, N,
                                                                   n_kv, hd, table, d_k, d_v);
      AKVS_LAUNCHED();
      return AKVS_OK;
    });
  });
}

// ---------------------------------------------------------------------------------------
// Top-b selection (Section 3.3).  Order: larger score first, equal scores by smaller token
// index; -0.0 counts as +0.0; NaN raises the status word.  Scores are non-negative, so the
// float bit pattern orders them; key = (~bits << 32) | local index sorts ascending into the
// wanted order and is unique, hence rank = #{keys smaller} and "rank < b" is the set.
// ---------------------------------------------------------------------------------------
__global__ void select_keys_kernel(const float* __restrict__ d_k, const float* __restrict__ d_v,
                                   const int32_t* __restrict__ ctx_off, int M, int N, uint64_t* __restrict__ keys,
                                   float* __restrict__ w_k, float* __restrict__ w_v, int32_t* status) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= N) return;
  int lo = 0, hi = M;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (ctx_off[mid] <= j) lo = mid; else hi = mid;
  }
  const uint32_t local = (uint32_t)(j - ctx_off[lo]);
  const float a = d_k[j] + 0.0f, b = d_v[j] + 0.0f;
  if (a != a || b != b) set_status(status, AKVS_ERR_NAN_SCORE);
  keys[j] = ((uint64_t)(~__float_as_uint(a)) << 32) | local;
  keys[N + j] = ((uint64_t)(~__float_as_uint(b)) << 32) | local;
  w_k[j] = fminf(a, 1.0f);
  w_v[j] = fminf(b, 1.0f);
}

constexpr int SEL_THREADS = 256;
constexpr int SEL_TILE = 1024;

// grid (M, 2): unit u, set s (0 = K, 1 = V).
__global__ void __launch_bounds__(SEL_THREADS)
select_rank_kernel(const uint64_t* __restrict__ keys, const int32_t* __restrict__ ctx_off,
                   const int32_t* __restrict__ probe_off, int N, uint8_t* __restrict__ flags,
                   int32_t* __restrict__ sk_idx, int32_t* __restrict__ sv_idx) {
  __shared__ uint64_t tile[SEL_TILE];
  __shared__ int warp_tot[SEL_THREADS / 32];
  __shared__ int carry;
  const int u = blockIdx.x, s = blockIdx.y;
  const int a = ctx_off[u], n = ctx_off[u + 1] - a;
  const int b = probe_off[u + 1] - probe_off[u];
  const uint64_t* key = keys + (size_t)s * N + a;
  uint8_t* flag = flags + (size_t)s * N + a;
  int32_t* out = (s == 0 ? sk_idx : sv_idx) + probe_off[u];

  // ranks, SEL_THREADS tokens at a time against key tiles staged in shared memory
  for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
    const int j = j0 + threadIdx.x;
    const uint64_t mine = j < n ? key[j] : 0;
    int rank = 0;
    for (int t0 = 0; t0 < n; t0 += SEL_TILE) {
      const int tn = min(SEL_TILE, n - t0);
      __syncthreads();
      for (int i = threadIdx.x; i < tn; i += SEL_THREADS) tile[i] = key[t0 + i];
      __syncthreads();
      if (j < n)
        for (int i = 0; i < tn; ++i) rank += tile[i] < mine;
    }
    if (j < n) flag[j] = rank < b;
  }
  __syncthreads();
  // compaction in ascending token order: block scan over the flags
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int j0 = 0; j0 < n; j0 += SEL_THREADS) {
    const int j = j0 + threadIdx.x;
    const int f = j < n ? flag[j] : 0;
    int incl = f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < wid; ++w) before += warp_tot[w];
    if (f) out[before + incl - 1] = a + j;
    __syncthreads();
    if (threadIdx.x == SEL_THREADS - 1) carry = before + incl;
    __syncthreads();
  }
}

// One CTA: rows = sorted union of both flag sets, then the query positions.
__global__ void __launch_bounds__(1024)
select_rows_kernel(const uint8_t* __restrict__ flags, int N, int n_query, int32_t* __restrict__ rows,
                   int32_t* __restrict__ counts) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  for (int j0 = 0; j0 < N; j0 += 1024) {
    const int j = j0 + threadIdx.x;
    const int f = j < N ? (flags[j] | flags[N + j]) : 0;
    int incl = f;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < wid; ++w) before += warp_tot[w];
    if (f) rows[before + incl - 1] = j;
    __syncthreads();
    if (threadIdx.x == 1023) carry = before + incl;
    __syncthreads();
  }
  const int P = carry;
  for (int i = threadIdx.x; i < n_query; i += 1024) rows[P + i] = N + i;
  if (threadIdx.x == 0) { counts[0] = P; counts[1] = P + n_query; }
}

int32_t launch_select(const float* d_k, const float* d_v, const int32_t* ctx_off, const int32_t* probe_off, int M,
                      int N, int n_query, int32_t* sk_idx, int32_t* sv_idx, float* w_k, float* w_v, int32_t* rows,
                      uint64_t* keys, uint8_t* flags, int32_t* counts, int32_t* status, cudaStream_t st) {
  if (N > 0) {
    select_keys_kernel<<<akvs_cdiv(N, 256), 256, 0, st>>>(d_k, d_v, ctx_off, M, N, keys, w_k, w_v, status);
    AKVS_LAUNCHED();
    select_rank_kernel<<<dim3(M, 2), SEL_THREADS, 0, st>>>(keys, ctx_off, probe_off, N, flags, sk_idx, sv_idx);
    AKVS_LAUNCHED();
  }
  select_rows_kernel<<<1, 1024, 0, st>>>(flags, N, n_query, rows, counts);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

// ---------------------------------------------------------------------------------------
// Mean estimation (Section 3.3; Algorithm 1 line 5): mu_u = (1/b_u) sum_{j in S_u} (fresh_j -
// reuse_j).  One CTA per (unit, kv head, K|V).  A thread owns one pair chunk (16 bytes of the
// lower half of the head and the RoPE partner 16 bytes in the upper half) of one probe slot:
// every global access is a 16-byte vector, a head's row is read as two whole 128-byte lines
// by neighbouring threads, and the 256 / (chunks per head) slots take the unit's probes side
// by side (all of them at once for b_u up to the slot count), so the dependent index loads
// (probe -> recomputed row, store row) are paid once.  Slots are summed in a fixed order.
// The probe arrays may have been written by the caller: an index outside the context or a
// probe range outside the arrays raises AKVS_ERR_INVALID_ARG and is skipped, never read.
// ---------------------------------------------------------------------------------------
constexpr int OFF_THREADS = 256;

template <typename T, typename TW, int FMT>
__global__ void __launch_bounds__(OFF_THREADS)
offsets_kernel(KvLayer kv, ReqMaps maps, const int32_t* __restrict__ probe_off, const int32_t* __restrict__ sk_idx,
               const int32_t* __restrict__ sv_idx, const T* __restrict__ k_fresh, const T* __restrict__ v_fresh,
               int N, int n_probe_cap, int n_kv, int hd, const float2* __restrict__ table, float* __restrict__ mu_k,
               float* __restrict__ mu_v, int32_t* status) {
  constexpr int V = VecOf<T>::N;
  extern __shared__ float part[];                 // [slots][hd]
  pdl_trigger();
  const int u = blockIdx.x, h = blockIdx.y, is_v = blockIdx.z;
  const int half = hd / 2, ch = half / V;
  const int slots = OFF_THREADS / ch;
  const int slot = threadIdx.x / ch, c = threadIdx.x - slot * ch;
  int p0 = probe_off[u], b = probe_off[u + 1] - p0;
  if (p0 < 0 || b < 0 || (int64_t)p0 + b > n_probe_cap) {
    if (threadIdx.x == 0) set_status(status, AKVS_ERR_INVALID_ARG);
    p0 = 0;
    b = 0;
  }
  const int32_t* S = (is_v ? sv_idx : sk_idx) + p0;
  const T* fresh = is_v ? v_fresh : k_fresh;
  const void* cbase = is_v ? kv.v : kv.k;
  const void* cmeta = is_v ? kv.v_meta : kv.k_meta;
  float acc_lo[V], acc_hi[V];
#pragma unroll
  for (int i = 0; i < V; ++i) acc_lo[i] = acc_hi[i] = 0.f;
  // First the reused half, -sum Rot(off_u) K_cached: the probe lists, the index maps, the
  // rotation table and the unit cache are inputs no kernel of the layer writes, so this part
  // runs while the projection GEMM before this kernel is still busy.  Then, once that GEMM has
  // completed (griddepcontrol.wait), + sum of the fresh rows.
  if (slot < slots) {
    float2 rot[V];
    if (!is_v) ld_f2<V>(table + (size_t)maps.unit_pos[u] * half + c * V, rot);
    for (int i = slot; i < b; i += slots) {
      const int j = S[i];
      if (j < 0 || j >= N) { set_status(status, AKVS_ERR_INVALID_ARG); continue; }
      if (maps.row_of_pos[j] < 0) continue;         // inconsistent caller-supplied sets: skip
      const int64_t src = maps.tok_src[j];
      float lo[V], hi[V];
      load_cached_chunk<TW, FMT>(cbase, cmeta, src, n_kv, hd, h, c * V, lo);
      load_cached_chunk<TW, FMT>(cbase, cmeta, src, n_kv, hd, h, half + c * V, hi);
#pragma unroll
      for (int e = 0; e < V; ++e) {
        float rl = lo[e], rh = hi[e];
        if (!is_v) {
          rl = lo[e] * rot[e].x - hi[e] * rot[e].y;
          rh = hi[e] * rot[e].x + lo[e] * rot[e].y;
        }
        acc_lo[e] -= rl;
        acc_hi[e] -= rh;
      }
    }
  }
  pdl_wait();
  if (slot < slots) {
    for (int i = slot; i < b; i += slots) {
      const int j = S[i];
      if (j < 0 || j >= N) continue;
      const int row = maps.row_of_pos[j];
      if (row < 0) continue;
      float flo[V], fhi[V];
      const T* fp = fresh + ((size_t)row * n_kv + h) * hd + c * V;
      ld16(fp, flo);
      ld16(fp + half, fhi);
#pragma unroll
      for (int e = 0; e < V; ++e) {
        acc_lo[e] += flo[e];
        acc_hi[e] += fhi[e];
      }
    }
#pragma unroll
    for (int e = 0; e < V; ++e) {
      part[slot * hd + c * V + e] = acc_lo[e];
      part[slot * hd + half + c * V + e] = acc_hi[e];
    }
  }
  __syncthreads();
  float* mu = (is_v ? mu_v : mu_k) + ((size_t)u * n_kv + h) * hd;
  for (int e = threadIdx.x; e < hd; e += OFF_THREADS) {
    float s = 0.f;
    for (int w = 0; w < slots; ++w) s += part[w * hd + e];
    mu[e] = b > 0 ? s / (float)b : 0.f;
  }
}

int32_t launch_offsets(int dtype, const KvLayer& kv, const ReqMaps& maps, const int32_t* probe_off,
                       const int32_t* sk_idx, const int32_t* sv_idx, const void* k_fresh, const void* v_fresh, int M,
                       int N, int n_probe_cap, int n_kv, int hd, const float2* table, float* mu_k, float* mu_v,
                       int32_t* status, cudaStream_t st) {
  if (M == 0) return AKVS_OK;
  AKVS_TRY(check_kv_shape(dtype, kv, hd));
  const int V = dtype == AKVS_F32 ? 4 : 8;
  const int ch = hd / 2 / V;
  if (ch > OFF_THREADS) return AKVS_ERR_UNSUPPORTED;
  const dim3 grid(M, n_kv, 2);
  const size_t smem = (size_t)(OFF_THREADS / ch) * hd * sizeof(float);
  if (smem > 48 * 1024) return AKVS_ERR_UNSUPPORTED;
  ProfScope prof(5, kv.fmt, 0.0, st);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    return dispatch_fmt(kv.fmt, [&](auto f) -> int32_t {
      AKVS_CUDA(launch_pdl(offsets_kernel<T, T, decltype(f)::value>, grid, dim3(OFF_THREADS), smem, st, kv, maps,
                           probe_off, sk_idx, sv_idx, (const T*)k_fresh, (const T*)v_fresh, N, n_probe_cap, n_kv, hd,
                           table, mu_k, mu_v, status));
      AKVS_LAUNCHED();
      return AKVS_OK;
    });
  });
}

// ---------------------------------------------------------------------------------------
// Correction pass (Algorithm 1 lines 6-8) fused with dequantisation and re-alignment:
//   context token j of unit u, not in S^K:  K_out = Rot(off_u) deq(K_cached) + w_K[j] mu_K[u]
//                              in S^K:      K_out = fresh K of its recomputed row
//   V likewise with S^V (no rotation);  query token i: fresh K/V of row P + i.
//
// Work split.  A token's K row and V row are two "role rows".  A thread owns ONE pair chunk (16
// bytes of the lower half of a head + its RoPE partner 16 bytes in the upper half) of one role
// for the whole launch, so its rotation entries and the unit's offsets sit in registers and are
// refetched only when the token's unit changes (units are runs of a hundred tokens and more).
// A CTA takes a contiguous slice of tokens, `tl` of them side by side; the grid is one wave of
// equal slices.
//
// Data movement.  The input is streamed through shared memory with per-thread asynchronous
// copies (cp.async), COR_DEPTH tokens ahead, so the bytes in flight do not cost registers: the
// `ch` threads that own a head's chunks (always lanes of one warp) copy that head's bytes of the
// token's row - cached codes (+ the group records) or a fresh row - 16 bytes per thread and
// copy, into their slot of the ring; cp.async.wait_group + __syncwarp hands the slot to its
// owners, who decode, rotate and add w mu on packed float pairs (fma.rn.f32x2) and store 16-byte
// vectors that neighbouring threads complete to whole 128-byte lines.  Fresh rows are copied as
// the bytes they are.
//
// Overlap with the kernel before it.  The per-token records, the rotation table and the unit
// cache are inputs that no kernel of the layer writes, so the slice's records and the first
// COR_DEPTH tokens' CACHE bytes are requested BEFORE griddepcontrol.wait, while the offset kernel
// (and the projection GEMM before it) still run; only the fresh rows and the offsets wait.
// ---------------------------------------------------------------------------------------
#ifndef AKVS_COR_DEPTH
#define AKVS_COR_DEPTH 4
#endif
#ifndef AKVS_COR_CTAS
#define AKVS_COR_CTAS 3
#endif
constexpr int COR_THREADS = 256, COR_DEPTH = AKVS_COR_DEPTH, COR_CTAS_PER_SM = AKVS_COR_CTAS;

// Packed float pairs: the sm_100 float2 builtins (one FFMA2 / FMUL2 / FADD2 per two lanes of
// arithmetic) keep a pair in an aligned register pair from the conversion to the pack, with no
// moves in between.
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void unpack16(const uint4& r, float2 (&o)[2], const float*) {
  o[0] = make_float2(__uint_as_float(r.x), __uint_as_float(r.y));
  o[1] = make_float2(__uint_as_float(r.z), __uint_as_float(r.w));
}
__device__ __forceinline__ void unpack16(const uint4& r, float2 (&o)[4], const bf16*) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
}
__device__ __forceinline__ void unpack16(const uint4& r, float2 (&o)[4], const f16*) {
  const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
}
__device__ __forceinline__ uint4 pack16(const float2 (&o)[2], const float*) {
  return make_uint4(__float_as_uint(o[0].x), __float_as_uint(o[0].y), __float_as_uint(o[1].x), __float_as_uint(o[1].y));
}
__device__ __forceinline__ uint4 pack16(const float2 (&o)[4], const bf16*) {
  return make_uint4(pack_bf16x2(o[0].x, o[0].y), pack_bf16x2(o[1].x, o[1].y), pack_bf16x2(o[2].x, o[2].y),
                    pack_bf16x2(o[3].x, o[3].y));
}
__device__ __forceinline__ uint4 pack16(const float2 (&o)[4], const f16*) {
  return make_uint4(pack_f16x2(o[0].x, o[0].y), pack_f16x2(o[1].x, o[1].y), pack_f16x2(o[2].x, o[2].y),
                    pack_f16x2(o[3].x, o[3].y));
}

__device__ __forceinline__ uint4 lds128(uint32_t a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
  return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
  return v;
}
__device__ __forceinline__ void cp_async16s(uint32_t dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async4s(uint32_t dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(gsrc) : "memory");
}

// V cached elements starting at element `e` of one head, from that head's bytes in shared memory
// (shared-memory addresses; `codes`: the head's values or codes as they lie in the store; `recs`:
// its (scale, min) records).
template <typename T, int FMT>
__device__ __forceinline__ void decode_head_chunk(uint32_t codes, uint32_t recs, int e, float2 (&out)[VecOf<T>::N / 2]) {
  constexpr int V = VecOf<T>::N;
  if constexpr (FMT == AKVS_KV_NATIVE) {
    unpack16(lds128(codes + e * (int)sizeof(T)), out, (const T*)nullptr);
  } else if constexpr (FMT == AKVS_KV_FP8) {
    uint32_t w[2];
    if constexpr (V == 8) {
      const uint2 t = lds64(codes + e);
      w[0] = t.x; w[1] = t.y;
    } else {
      w[0] = lds32(codes + e);
    }
#pragma unroll
    for (int i = 0; i < V / 2; ++i) {
      const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)((w[i >> 1] >> (16 * (i & 1))) & 0xFFFFu), __NV_E4M3);
      out[i] = __half22float2(*reinterpret_cast<const __half2*>(&h));
    }
  } else {
    constexpr int BYTES = V * FMT / 8;                   // 4, 2 or 1 bytes of codes
    const int byte0 = e * FMT / 8;
    const uint32_t word = lds32(codes + (byte0 & ~3));
    const uint32_t packed = BYTES == 4 ? word : (word >> (8 * (byte0 & 3))) & ((1u << (8 * BYTES)) - 1u);
    const uint32_t rec = lds32(recs + (e / 64) * 4);
    const __half2 sm = *reinterpret_cast<const __half2*>(&rec);
    const float s = __low2float(sm), mn = __high2float(sm);
    const float2 s2 = make_float2(s, s), mn2 = make_float2(mn, mn), bias2 = make_float2(-8388608.f, -8388608.f);
    // code -> float without the integer-to-float unit: 2^23 + code as a bit pattern, minus 2^23
    // (exact), then the same single-rounding fma(code, scale, min) as everywhere else
#pragma unroll
    for (int i = 0; i < V / 2; ++i) {
      const uint32_t u0 = ((packed >> (FMT * 2 * i)) & ((1u << FMT) - 1u)) | 0x4B000000u;
      const uint32_t u1 = ((packed >> (FMT * (2 * i + 1))) & ((1u << FMT) - 1u)) | 0x4B000000u;
      out[i] = __ffma2_rn(__fadd2_rn(make_float2(__uint_as_float(u0), __uint_as_float(u1)), bias2), s2, mn2);
    }
  }
}

template <typename T, int FMT>
__global__ void __launch_bounds__(COR_THREADS, COR_CTAS_PER_SM)
correct_kernel(KvLayer kv, const int4* __restrict__ tok_meta, const int32_t* __restrict__ unit_pos,
               const T* __restrict__ k_fresh, const T* __restrict__ v_fresh, const float* __restrict__ mu_k,
               const float* __restrict__ mu_v, int T_tok, int n_kv, int hd, int ipt, int tl, int slice, int slot_bytes,
               int weighted, const float2* __restrict__ table, T* __restrict__ out_k, T* __restrict__ out_v) {
  // ipt = pair chunks of the kv heads this CTA column (blockIdx.y) covers: heads per CTA x chunks per head
  constexpr int V = VecOf<T>::N;
  constexpr int ES = (int)sizeof(T);
  constexpr int CODE_BITS = FMT == AKVS_KV_NATIVE ? 8 * ES : FMT;      // bits per cached element
  extern __shared__ __align__(16) uint8_t cor_smem[];
  int4* meta_s = reinterpret_cast<int4*>(cor_smem);                    // [2][slice] the slice's records
  pdl_trigger();
  const int t0 = blockIdx.x * slice;
  const int n_slice = min(T_tok, t0 + slice) - t0;
  for (int i = threadIdx.x; i < 2 * n_slice; i += COR_THREADS) {
    const int r = i >= n_slice, jl = i - r * n_slice;
    meta_s[r * slice + jl] = tok_meta[(size_t)r * T_tok + t0 + jl];
  }
  __syncthreads();

  const int half = hd / 2, ch = half / V;
  const int tpt = 2 * ipt;                              // threads per token: K items, then V items
  const int lane_tok = threadIdx.x / tpt;
  const int rem = threadIdx.x - lane_tok * tpt;
  const int role = rem / ipt;                           // 0: K, 1: V
  const int item = rem - role * ipt;
  const int h = blockIdx.y * (ipt / ch) + item / ch, c = item % ch;
  const bool active = lane_tok < tl && h < n_kv;        // idle lanes still take part in the warp syncs
  const int n_q = (n_slice + tl - 1) / tl;              // steps of the CTA (the same for every thread)
  const int n_mine = active ? (n_slice - lane_tok + tl - 1) / tl : 0;   // tokens of this thread
  // shared-memory addresses: this role's records; the slot of this thread's head in ring stage 0
  const uint32_t meta_a = tc_smem_u32(meta_s) + (uint32_t)(role * slice + lane_tok) * 16u;
  const uint32_t meta_step = (uint32_t)tl * 16u;
  const uint32_t ring0 = tc_smem_u32(cor_smem) + (uint32_t)(2 * slice) * 16u + (uint32_t)(threadIdx.x / ch) * slot_bytes;
  const uint32_t ring_stride = (uint32_t)(COR_THREADS / ch) * slot_bytes;
  const uint32_t ring_end = ring0 + COR_DEPTH * ring_stride;
  // global bases of this thread's pieces
  const int head_code_bytes = hd * CODE_BITS / 8;
  const uint32_t cache_row_bytes = (uint32_t)(n_kv * head_code_bytes);   // 32-bit sizes: one widening multiply per address
  const uint32_t fresh_row_bytes = (uint32_t)(n_kv * hd * ES);
  const uint8_t* cache_p = reinterpret_cast<const uint8_t*>(role ? kv.v : kv.k) + (size_t)h * head_code_bytes + c * 16;
  const uint8_t* rec_p = reinterpret_cast<const uint8_t*>(role ? kv.v_meta : kv.k_meta) + (size_t)h * (hd / 64) * 4 + c * 4;
  const uint32_t rec_row_bytes = (uint32_t)(n_kv * (hd / 64) * 4);
  const uint8_t* fresh_p = reinterpret_cast<const uint8_t*>(role ? v_fresh : k_fresh) + (size_t)h * hd * ES + c * 16;
  uint8_t* out_p = reinterpret_cast<uint8_t*>(role ? out_v : out_k) + ((size_t)(t0 + lane_tok) * n_kv + h) * hd * ES + c * 16;
  const uint32_t out_step = (uint32_t)tl * fresh_row_bytes;
  const float* __restrict__ mu = (role ? mu_v : mu_k) + (size_t)h * hd + c * V;
  const uint32_t hi_off = (uint32_t)ch * 16u;           // byte distance of the upper chunk (fresh rows, native cache)
  const bool copy_codes = c * 16 < head_code_bytes;      // quantised formats: fewer 16-byte pieces than lanes
  const bool copy_rec = c < hd / 64;

  // Requests the bytes of local token q into ring stage `dst` (WHICH: 1 = cached rows only,
  // 2 = fresh rows only, 3 = either).  No-op past the slice.
  auto issue = [&](int q, uint32_t dst, auto which) {
    constexpr int WHICH = decltype(which)::value;
    if (q >= n_mine) return;
    const uint4 m = lds128(meta_a + (uint32_t)q * meta_step);
    if ((int)m.y >= 0) {
      if (WHICH & 2) {
        const uint8_t* src = fresh_p + (uint64_t)m.y * fresh_row_bytes;
        cp_async16s(dst + c * 16, src);
        cp_async16s(dst + c * 16 + hi_off, src + hi_off);
      }
    } else if (WHICH & 1) {
      if constexpr (FMT == AKVS_KV_NATIVE) {
        const uint8_t* src = cache_p + (uint64_t)m.x * cache_row_bytes;
        cp_async16s(dst + c * 16, src);
        cp_async16s(dst + c * 16 + hi_off, src + hi_off);
      } else {
        if (copy_codes) cp_async16s(dst + c * 16, cache_p + (uint64_t)m.x * cache_row_bytes);
        if constexpr (FMT == AKVS_KV_Q4 || FMT == AKVS_KV_Q2)
          if (copy_rec) cp_async4s(dst + head_code_bytes + c * 4, rec_p + (uint64_t)m.x * rec_row_bytes);
      }
    }
  };
  using W1 = std::integral_constant<int, 1>;
  using W2_ = std::integral_constant<int, 2>;
  using W3 = std::integral_constant<int, 3>;

#pragma unroll
  for (int q = 0; q < COR_DEPTH; ++q) {
    issue(q, ring0 + q * ring_stride, W1{});
    cp_async_commit();
  }
  pdl_wait();                                           // fresh rows and offsets are other kernels' outputs
#pragma unroll
  for (int q = 0; q < COR_DEPTH; ++q) {
    issue(q, ring0 + q * ring_stride, W2_{});
    cp_async_commit();
  }

  float2 C2[V / 2], S2[V / 2], NS2[V / 2], ML2[V / 2], MH2[V / 2];   // (cos, cos), (sin, sin), (-sin, -sin), offsets of the lower / upper chunk
  int cur_unit = -1;
  uint32_t slot = ring0, meta_q = meta_a;
  for (int q = 0; q < n_q; ++q, meta_q += meta_step) {
    cp_async_wait<COR_DEPTH - 1>();                     // everything up to this token's copies has landed
    __syncwarp();                                       // ... for every lane of the head's group
    if (q < n_mine) {
      const uint4 m = lds128(meta_q);
      if ((int)m.y >= 0) {                              // a fresh row: the bytes as they are
        *reinterpret_cast<uint4*>(out_p) = lds128(slot + c * 16);
        *reinterpret_cast<uint4*>(out_p + hi_off) = lds128(slot + c * 16 + hi_off);
      } else {
        if ((int)m.z != cur_unit) {
          cur_unit = (int)m.z;
          if (role == 0) {
            float2 rot[V];
            ld_f2<V>(table + (size_t)unit_pos[cur_unit] * half + c * V, rot);
#pragma unroll
            for (int i = 0; i < V / 2; ++i) {
              C2[i] = make_float2(rot[2 * i].x, rot[2 * i + 1].x);
              S2[i] = make_float2(rot[2 * i].y, rot[2 * i + 1].y);
              NS2[i] = make_float2(-rot[2 * i].y, -rot[2 * i + 1].y);
            }
          }
          if (weighted) {
            float ml[V], mh[V];
            const float* mp = mu + (size_t)cur_unit * n_kv * hd;
            ld_f<V>(mp, ml);
            ld_f<V>(mp + half, mh);
#pragma unroll
            for (int i = 0; i < V / 2; ++i) {
              ML2[i] = make_float2(ml[2 * i], ml[2 * i + 1]);
              MH2[i] = make_float2(mh[2 * i], mh[2 * i + 1]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < V / 2; ++i) ML2[i] = MH2[i] = make_float2(0.f, 0.f);
          }
        }
        float2 lo[V / 2], hi[V / 2];
        decode_head_chunk<T, FMT>(slot, slot + head_code_bytes, c * V, lo);
        decode_head_chunk<T, FMT>(slot, slot + head_code_bytes, half + c * V, hi);
        const float w = __uint_as_float(m.w);
        const float2 W2 = make_float2(w, w);
        if (role == 0) {
          // lo' = a cos - b sin + w mu_lo,  hi' = b cos + a sin + w mu_hi
#pragma unroll
          for (int i = 0; i < V / 2; ++i) {
            const float2 a2 = lo[i], b2 = hi[i];
            lo[i] = fma2(b2, NS2[i], fma2(W2, ML2[i], mul2(a2, C2[i])));
            hi[i] = fma2(a2, S2[i], fma2(W2, MH2[i], mul2(b2, C2[i])));
          }
        } else {
#pragma unroll
          for (int i = 0; i < V / 2; ++i) {
            lo[i] = fma2(W2, ML2[i], lo[i]);
            hi[i] = fma2(W2, MH2[i], hi[i]);
          }
        }
        *reinterpret_cast<uint4*>(out_p) = pack16(lo, (const T*)nullptr);
        *reinterpret_cast<uint4*>(out_p + hi_off) = pack16(hi, (const T*)nullptr);
      }
    }
    out_p += out_step;
    __syncwarp();                                       // the group is done with the stage before it is refilled
    if (q + COR_DEPTH < n_mine) issue(q + COR_DEPTH, slot, W3{});
    cp_async_commit();                                  // one group per step keeps the wait count constant
    slot += ring_stride;
    if (slot == ring_end) slot = ring0;
  }
}

int g_cor_slots = 0;                 // CTA slots of the device for the correction kernel (SMs x CTAs per SM)

int32_t launch_correct(int dtype, const KvLayer& kv, const ReqMaps& maps, const void* k_fresh, const void* v_fresh,
                       bool weighted, const float* mu_k, const float* mu_v, int N, int n_query, int n_kv, int hd,
                       const float2* table, void* out_k, void* out_v, cudaStream_t st) {
  const int T_tok = N + n_query;
  if (T_tok == 0) return AKVS_OK;
  AKVS_TRY(check_kv_shape(dtype, kv, hd));
  const int V = dtype == AKVS_F32 ? 4 : 8;
  const int es = (int)dtype_size(dtype);
  const int ch = hd / 2 / V;                            // pair chunks of one head
  if (ch > 32 || (ch & (ch - 1)) != 0) return AKVS_ERR_UNSUPPORTED;   // a head's chunk owners are lanes of one warp
  const int heads_per_cta = n_kv < COR_THREADS / (2 * ch) ? n_kv : COR_THREADS / (2 * ch);
  const int head_groups = (n_kv + heads_per_cta - 1) / heads_per_cta;
  const int ipt = heads_per_cta * ch;                   // pair chunks of one role row within a head group
  if ((int64_t)T_tok * n_kv * hd >= (1ll << 31)) return AKVS_ERR_SHAPE;
  if (!g_cor_slots) {
    int dev = 0, sms = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    g_cor_slots = (sms > 0 ? sms : 148) * COR_CTAS_PER_SM;
  }
  const int tl = COR_THREADS / (2 * ipt);               // tokens side by side in a CTA
  const int slots = g_cor_slots / head_groups > 0 ? g_cor_slots / head_groups : 1;
  int slice = (T_tok + slots - 1) / slots;              // one wave of equal slices
  slice = (slice + tl - 1) / tl * tl;
  const int grid = (T_tok + slice - 1) / slice;
  // bytes of one head in the ring: a fresh row's head, or the cached head and its records
  const int code_bits = kv.fmt == AKVS_KV_NATIVE ? 8 * es : kv.fmt;
  int slot_bytes = hd * code_bits / 8 + ((kv.fmt == AKVS_KV_Q4 || kv.fmt == AKVS_KV_Q2) ? (hd / 64) * 4 : 0);
  if (slot_bytes < hd * es) slot_bytes = hd * es;
  slot_bytes = (slot_bytes + 15) / 16 * 16;
  const size_t smem = (size_t)2 * slice * sizeof(int4) + (size_t)COR_DEPTH * (COR_THREADS / ch) * slot_bytes;
  if (smem > 200 * 1024) return AKVS_ERR_TOO_LARGE;
  // algorithmic bytes: every context K and V element read once in its cache format and
  // written once; fresh rows and query rows copied; 8 bytes of weights per context token
  const double in_b = kv.fmt == AKVS_KV_NATIVE ? (double)es : kv.fmt == AKVS_KV_FP8 ? 1.0 : kv.fmt / 8.0 + 4.0 / 64.0;
  const double out_b = (double)es;
  const double bytes = 2.0 * n_kv * hd * ((double)N * (in_b + out_b) + (double)n_query * 2 * out_b) + 8.0 * N;
  ProfScope prof(2, kv.fmt, bytes, st);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    return dispatch_fmt(kv.fmt, [&](auto f) -> int32_t {
      auto kern = correct_kernel<T, decltype(f)::value>;
      static size_t smem_allowed = 48 * 1024;          // per instantiation: raised when a launch needs more
      if (smem > smem_allowed) {
        AKVS_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        smem_allowed = smem;
      }
      AKVS_CUDA(launch_pdl(kern, dim3(grid, head_groups), dim3(COR_THREADS), smem, st, kv, maps.tok_meta, maps.unit_pos,
                           (const T*)k_fresh, (const T*)v_fresh, mu_k, mu_v, T_tok, n_kv, hd, ipt, tl, slice, slot_bytes,
                           weighted ? 1 : 0, table, (T*)out_k, (T*)out_v));
      AKVS_LAUNCHED();
      return AKVS_OK;
    });
  });
}

// ---------------------------------------------------------------------------------------
// Diagnostics of the residual model r_i = mu + xi_i (Section 3.4; the appendix's mean-explained
// energy): per unit and per K | V, over ALL tokens of the unit (fresh K/V of every context row
// come from a full recompute),
//   mean      = sum_i sel_i r_i / sum_i sel_i
//   total     = sum_i |r_i|^2,   remaining = sum_i |r_i - w_i mu|^2
// One CTA per (unit, K | V); a thread owns RS_PAIRS rotation pairs of the row and walks the
// unit's tokens in order (fixed summation order), so the per-dimension sums stay in registers.
// ---------------------------------------------------------------------------------------
constexpr int RS_THREADS = 256, RS_PAIRS = 8;

template <typename T, int FMT>
__global__ void __launch_bounds__(RS_THREADS)
residual_stats_kernel(KvLayer kv, const int32_t* __restrict__ ctx_off, const int32_t* __restrict__ tok_src,
                      const T* __restrict__ k_fresh, const T* __restrict__ v_fresh, int n_kv, int hd,
                      const float2* __restrict__ table, const float* __restrict__ sel_k,
                      const float* __restrict__ sel_v, const float* __restrict__ mu_k, const float* __restrict__ mu_v,
                      const float* __restrict__ w_k, const float* __restrict__ w_v, float* __restrict__ mean_k,
                      float* __restrict__ mean_v, float* __restrict__ energy) {
  __shared__ double red[2][RS_THREADS / 32];
  const int u = blockIdx.x, is_v = blockIdx.y;
  const int half = hd / 2, P = n_kv * half;
  const int a = ctx_off[u], e = ctx_off[u + 1];
  const T* fresh = is_v ? v_fresh : k_fresh;
  const void* cbase = is_v ? kv.v : kv.k;
  const void* cmeta = is_v ? kv.v_meta : kv.k_meta;
  const float* sel = is_v ? sel_v : sel_k;
  const float* mu = is_v ? mu_v : mu_k;
  const float* w = is_v ? w_v : w_k;
  const float2* rot = table + (size_t)a * half;           // a single request: the unit starts at position a
  float s_lo[RS_PAIRS], s_hi[RS_PAIRS], m_lo[RS_PAIRS], m_hi[RS_PAIRS];
#pragma unroll
  for (int i = 0; i < RS_PAIRS; ++i) {
    s_lo[i] = s_hi[i] = 0.f;
    const int p = threadIdx.x + i * RS_THREADS;
    const int h = p / half, d = p - h * half;
    m_lo[i] = mu && p < P ? mu[((size_t)u * n_kv + h) * hd + d] : 0.f;
    m_hi[i] = mu && p < P ? mu[((size_t)u * n_kv + h) * hd + half + d] : 0.f;
  }
  double tot = 0.0, rem = 0.0;
  float ssum = 0.f;
  for (int j = a; j < e; ++j) {
    const int64_t src = tok_src[j];
    const float sj = sel ? sel[j] : 1.f, wj = w ? w[j] : 1.f;
    ssum += sj;
    float t_acc = 0.f, r_acc = 0.f;
#pragma unroll
    for (int i = 0; i < RS_PAIRS; ++i) {
      const int p = threadIdx.x + i * RS_THREADS;
      if (p >= P) break;
      const int h = p / half, d = p - h * half;
      float lo[1], hi[1];
      {
        // scalar decode of elements d and half + d of head h (every cache format)
        if constexpr (FMT == AKVS_KV_NATIVE) {
          const T* cp = reinterpret_cast<const T*>(cbase) + ((size_t)src * n_kv + h) * hd;
          lo[0] = to_f(cp[d]);
          hi[0] = to_f(cp[half + d]);
        } else if constexpr (FMT == AKVS_KV_FP8) {
          const uint8_t* cp = reinterpret_cast<const uint8_t*>(cbase) + ((size_t)src * n_kv + h) * hd;
          const __half_raw ra = __nv_cvt_fp8_to_halfraw(cp[d], __NV_E4M3), rb = __nv_cvt_fp8_to_halfraw(cp[half + d], __NV_E4M3);
          lo[0] = __half2float(*reinterpret_cast<const __half*>(&ra));
          hi[0] = __half2float(*reinterpret_cast<const __half*>(&rb));
        } else {
          const uint8_t* cp = reinterpret_cast<const uint8_t*>(cbase) + ((size_t)src * n_kv + h) * hd * FMT / 8;
          const __half2* mp = reinterpret_cast<const __half2*>(cmeta) + ((size_t)src * n_kv + h) * (hd / 64);
          const int d2 = half + d;
          const uint32_t qa = (cp[d * FMT / 8] >> ((d * FMT) & 7)) & ((1u << FMT) - 1u);
          const uint32_t qb = (cp[d2 * FMT / 8] >> ((d2 * FMT) & 7)) & ((1u << FMT) - 1u);
          const __half2 ma = mp[d / 64], mb = mp[d2 / 64];
          lo[0] = __fmaf_rn((float)qa, __low2float(ma), __high2float(ma));
          hi[0] = __fmaf_rn((float)qb, __low2float(mb), __high2float(mb));
        }
      }
      if (!is_v) {
        const float2 t = rot[d];
        const float rl = lo[0] * t.x - hi[0] * t.y, rh = hi[0] * t.x + lo[0] * t.y;
        lo[0] = rl;
        hi[0] = rh;
      }
      const T* fp = fresh + ((size_t)j * n_kv + h) * hd;
      const float r_lo = to_f(fp[d]) - lo[0], r_hi = to_f(fp[half + d]) - hi[0];
      s_lo[i] = fmaf(sj, r_lo, s_lo[i]);
      s_hi[i] = fmaf(sj, r_hi, s_hi[i]);
      t_acc += r_lo * r_lo + r_hi * r_hi;
      const float c_lo = r_lo - wj * m_lo[i], c_hi = r_hi - wj * m_hi[i];
      r_acc += c_lo * c_lo + c_hi * c_hi;
    }
    tot += (double)t_acc;
    rem += (double)r_acc;
  }
  float* mean = is_v ? mean_v : mean_k;
  if (mean) {
    const float inv = ssum > 0.f ? 1.f / ssum : 0.f;
#pragma unroll
    for (int i = 0; i < RS_PAIRS; ++i) {
      const int p = threadIdx.x + i * RS_THREADS;
      if (p >= P) break;
      const int h = p / half, d = p - h * half;
      mean[((size_t)u * n_kv + h) * hd + d] = s_lo[i] * inv;
      mean[((size_t)u * n_kv + h) * hd + half + d] = s_hi[i] * inv;
    }
  }
  // block sums in a fixed order: lanes by shuffle, warps by thread 0
  for (int o = 16; o > 0; o >>= 1) {
    tot += __shfl_down_sync(0xFFFFFFFFu, tot, o);
    rem += __shfl_down_sync(0xFFFFFFFFu, rem, o);
  }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = tot; red[1][threadIdx.x >> 5] = rem; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t2 = 0.0, r2 = 0.0;
    for (int i = 0; i < RS_THREADS / 32; ++i) { t2 += red[0][i]; r2 += red[1][i]; }
    energy[(size_t)u * 4 + is_v * 2] = (float)t2;
    energy[(size_t)u * 4 + is_v * 2 + 1] = (float)r2;
  }
}

int32_t launch_residual_stats(int dtype, const KvLayer& kv, const int32_t* ctx_off, const int32_t* tok_src,
                              const void* k_fresh, const void* v_fresh, int M, int n_kv, int hd, const float2* table,
                              const float* sel_k, const float* sel_v, const float* mu_k, const float* mu_v,
                              const float* w_k, const float* w_v, float* mean_k, float* mean_v, float* energy,
                              cudaStream_t st) {
  if (M == 0) return AKVS_OK;
  AKVS_TRY(check_kv_shape(dtype, kv, hd));
  if (n_kv * (hd / 2) > RS_THREADS * RS_PAIRS) return AKVS_ERR_TOO_LARGE;
  const dim3 grid(M, 2);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    return dispatch_fmt(kv.fmt, [&](auto f) -> int32_t {
      residual_stats_kernel<T, decltype(f)::value><<<grid, RS_THREADS, 0, st>>>(
          kv, ctx_off, tok_src, (const T*)k_fresh, (const T*)v_fresh, n_kv, hd, table, sel_k, sel_v, mu_k, mu_v, w_k,
          w_v, mean_k, mean_v, energy);
      AKVS_LAUNCHED();
      return AKVS_OK;
    });
  });
}
