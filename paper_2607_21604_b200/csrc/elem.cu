// Elementwise and row-wise steps of the decoder: embedding lookup, row gather, RMSNorm,
// RoPE table + rotation, and the cache group quantiser.  All are HBM-bound; every global
// access is a 16-byte vector where the layout allows it.
#include "common.cuh"
#include <cuda_fp8.h>

// ---------------------------------------------------------------------------------------
// h[r][:] = float(tok_emb[ids[gather ? gather[r] : r]][:])
// ---------------------------------------------------------------------------------------
// A token id outside [0, vocab) (ids are caller data) raises AKVS_ERR_INVALID_ARG in the status
// word and the row is written as zeros: the table is never read out of range.
template <typename T>
__global__ void embed_kernel(const T* __restrict__ emb, const int32_t* __restrict__ ids,
                             const int32_t* __restrict__ gather, int n, int d, int vocab, int32_t* status,
                             float* __restrict__ h) {
  constexpr int V = VecOf<T>::N;
  const int r = blockIdx.x;
  const int id = ids[gather ? gather[r] : r];
  const bool ok = id >= 0 && id < vocab;
  if (!ok && threadIdx.x == 0) set_status(status, AKVS_ERR_INVALID_ARG);
  const T* src = emb + (size_t)(ok ? id : 0) * d;
  float* dst = h + (size_t)r * d;
  for (int c = threadIdx.x * V; c < d; c += blockDim.x * V) {
    float v[V];
    if (ok) {
      ld16(src + c, v);
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i) v[i] = 0.f;
    }
#pragma unroll
    for (int i = 0; i < V; i += 4) {
      float t[4] = {v[i], v[i + 1], v[i + 2], v[i + 3]};
      st16(dst + c + i, t);
    }
  }
}

int32_t launch_embed(int dtype, const void* tok_emb, const int32_t* ids, const int32_t* gather, int n, int d,
                     int vocab, int32_t* status, float* h, cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    embed_kernel<T><<<n, 128, 0, st>>>((const T*)tok_emb, ids, gather, n, d, vocab, status, h);
    AKVS_LAUNCHED();
    return AKVS_OK;
  });
}

// rows[] may have been written by the caller (akvs_probes.rows): an entry outside [0, n_src)
// raises AKVS_ERR_INVALID_ARG and yields a row of zeros instead of an out-of-range read.
__global__ void gather_rows_kernel(const float* __restrict__ src, const int32_t* __restrict__ rows, int d, int n_src,
                                   int32_t* status, float* __restrict__ dst) {
  const int r = blockIdx.x;
  const int j = rows[r];
  const bool ok = j >= 0 && j < n_src;
  if (!ok && threadIdx.x == 0) set_status(status, AKVS_ERR_INVALID_ARG);
  const float4* s = reinterpret_cast<const float4*>(src + (size_t)(ok ? j : 0) * d);
  float4* t = reinterpret_cast<float4*>(dst + (size_t)r * d);
  for (int c = threadIdx.x; c < d / 4; c += blockDim.x) t[c] = ok ? s[c] : make_float4(0.f, 0.f, 0.f, 0.f);
}

int32_t launch_gather_rows(const float* src, const int32_t* rows, int n, int d, int n_src, int32_t* status, float* dst,
                           cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  gather_rows_kernel<<<n, 256, 0, st>>>(src, rows, d, n_src, status, dst);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

__global__ void iota_kernel(int32_t* p, int n, int start) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = start + i;
}
int32_t launch_iota(int32_t* p, int n, int start, cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  iota_kernel<<<akvs_cdiv(n, 256), 256, 0, st>>>(p, n, start);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

// ---------------------------------------------------------------------------------------
// RMSNorm: x = h * rsqrt(mean(h^2) + eps) * gain.  One CTA per row; the row (float) is read
// once into registers (d <= 256 threads * 4 * RMS_MAX_V elements).
// ---------------------------------------------------------------------------------------
constexpr int RMS_THREADS = 256;
constexpr int RMS_MAX_V = 8;           // float4 per thread: d <= 8192

template <typename TO>
__global__ void __launch_bounds__(RMS_THREADS)
rmsnorm_kernel(const float* __restrict__ h, const float* __restrict__ gain, float eps, int d, TO* __restrict__ x) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x;
  const float4* hp = reinterpret_cast<const float4*>(h + (size_t)r * d);
  const float4* gp = reinterpret_cast<const float4*>(gain);
  const int nv = d / 4;
  float4 v[RMS_MAX_V];
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < RMS_MAX_V; ++i) {
    const int c = threadIdx.x + i * RMS_THREADS;
    if (c < nv) {
      v[i] = hp[c];
      ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
    }
  }
  __shared__ float part[RMS_THREADS / 32];
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < RMS_THREADS / 32; ++i) tot += part[i];
  const float scale = rsqrtf(tot / (float)d + eps);
  TO* xp = x + (size_t)r * d;
#pragma unroll
  for (int i = 0; i < RMS_MAX_V; ++i) {
    const int c = threadIdx.x + i * RMS_THREADS;
    if (c < nv) {
      const float4 g = gp[c];
      const float o0 = v[i].x * scale * g.x, o1 = v[i].y * scale * g.y;
      const float o2 = v[i].z * scale * g.z, o3 = v[i].w * scale * g.w;
      if constexpr (sizeof(TO) == 4) {
        reinterpret_cast<float4*>(xp)[c] = make_float4(o0, o1, o2, o3);
      } else {
        uint2 pk;
        pk.x = pack2<TO>(o0, o1);
        pk.y = pack2<TO>(o2, o3);
        reinterpret_cast<uint2*>(xp)[c] = pk;
      }
    }
  }
}

int32_t launch_rmsnorm(int out_dtype, const float* h, const float* gain, float eps, int n, int d, void* x,
                       cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  if (d % 4 != 0 || d > RMS_THREADS * 4 * RMS_MAX_V) return AKVS_ERR_UNSUPPORTED;
  ProfScope prof(4, 0, (double)n * d * (4.0 + (out_dtype == AKVS_F32 ? 4.0 : 2.0)), st);
  return dispatch_dtype(out_dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    AKVS_CUDA(launch_pdl(rmsnorm_kernel<T>, dim3(n), dim3(RMS_THREADS), 0, st, h, gain, eps, d, (T*)x));
    AKVS_LAUNCHED();
    return AKVS_OK;
  });
}

// ---------------------------------------------------------------------------------------
// RoPE.  table[p][i] = (cos, sin)(p * base^(-2i/hd)), angle formed in double so that the
// float table is the correctly rounded value for every position the request can reach.
// ---------------------------------------------------------------------------------------
__global__ void rope_table_kernel(double base, int hd, int n_pos, float2* __restrict__ table) {
  const int half = hd / 2;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pos * half) return;
  const int p = idx / half, i = idx % half;
  const double inv_freq = pow(base, -2.0 * (double)i / (double)hd);
  double s, c;
  sincos((double)p * inv_freq, &s, &c);
  table[idx] = make_float2((float)c, (float)s);
}

int32_t launch_rope_table(float base, int hd, int n_pos, float2* table, cudaStream_t st) {
  if (n_pos == 0) return AKVS_OK;
  rope_table_kernel<<<akvs_cdiv((int64_t)n_pos * (hd / 2), 256), 256, 0, st>>>((double)base, hd, n_pos, table);
  AKVS_LAUNCHED();
  return AKVS_OK;
}

// In place on x[n][n_heads][hd] (row stride ld elements).  One thread per 16-byte chunk of
// the lower half; it also owns the partner chunk in the upper half.
template <typename T>
__global__ void rope_kernel(T* __restrict__ x, const int32_t* __restrict__ pos, int n, int n_heads, int hd, int ld,
                            const float2* __restrict__ table, int n_pos, int32_t* status, double base) {
  constexpr int V = VecOf<T>::N;
  pdl_trigger();
  pdl_wait();
  const int half = hd / 2, ch = half / V;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n * n_heads * ch) return;
  const int c = (int)(idx % ch);
  const int hh = (int)((idx / ch) % n_heads);
  const int r = (int)(idx / ((int64_t)ch * n_heads));
  int p = pos[r];
  if (table && (p < 0 || p >= n_pos)) {           // positions may be caller data: never index past the table
    set_status(status, AKVS_ERR_INVALID_ARG);
    p = 0;
  }
  T* lo_p = x + (size_t)r * ld + (size_t)hh * hd + c * V;
  T* hi_p = lo_p + half;
  float lo[V], hi[V], olo[V], ohi[V];
  ld16(lo_p, lo);
  ld16(hi_p, hi);
#pragma unroll
  for (int i = 0; i < V; ++i) {
    float cs, sn;
    if (table) {
      const float2 t = table[(size_t)p * half + c * V + i];
      cs = t.x;
      sn = t.y;
    } else {
      const double inv_freq = pow(base, -2.0 * (double)(c * V + i) / (double)hd);
      double s_, c_;
      sincos((double)p * inv_freq, &s_, &c_);
      cs = (float)c_;
      sn = (float)s_;
    }
    olo[i] = lo[i] * cs - hi[i] * sn;
    ohi[i] = hi[i] * cs + lo[i] * sn;
  }
  st16(lo_p, olo);
  st16(hi_p, ohi);
}

int32_t launch_rope(int dtype, void* x, const int32_t* pos, int n, int n_heads, int hd, int ld,
                    const float2* table, int n_pos, int32_t* status, float base, cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  const int V = dtype == AKVS_F32 ? 4 : 8;
  if (hd % (2 * V) != 0) return AKVS_ERR_UNSUPPORTED;
  const int64_t total = (int64_t)n * n_heads * (hd / 2 / V);
  const int blocks = akvs_cdiv(total, 256);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    AKVS_CUDA(launch_pdl(rope_kernel<T>, dim3(blocks), dim3(256), 0, st, (T*)x, pos, n, n_heads, hd, ld, table, n_pos, status,
                         (double)base));
    AKVS_LAUNCHED();
    return AKVS_OK;
  });
}

// ---------------------------------------------------------------------------------------
// Group quantiser of the cache (asymmetric min-max, 64 consecutive dims, float16 scale and
// minimum).  One warp per group: lane l owns elements 2l and 2l+1.  All decisions are
// float32 round-to-nearest operations with no contraction, so codes are reproducible:
//   scale = half((max - min) / levels); min16 = half(min);
//   code  = clamp(rint((x - min16) / scale), 0, levels), 0 when scale == 0.
// Packing: little-endian within a byte, dimension ascending.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void quantize_kernel(const T* __restrict__ x, int64_t n_groups, int bits, uint8_t* __restrict__ codes,
                                __half2* __restrict__ meta) {
  const int64_t g = (int64_t)blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5);
  if (g >= n_groups) return;
  const int lane = threadIdx.x & 31;
  const T* xp = x + g * 64 + 2 * lane;
  const float a = to_f(xp[0]), b = to_f(xp[1]);
  const float mn = warp_min(fminf(a, b));
  const float mx = warp_max(fmaxf(a, b));
  const float levels = (float)((1 << bits) - 1);
  const __half s16 = __float2half_rn(__fdiv_rn(__fsub_rn(mx, mn), levels));
  const __half m16 = __float2half_rn(mn);
  const float s = __half2float(s16), m = __half2float(m16);
  uint32_t c0 = 0, c1 = 0;
  if (s != 0.f) {
    c0 = (uint32_t)fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(a, m), s)), 0.f), levels);
    c1 = (uint32_t)fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(b, m), s)), 0.f), levels);
  }
  if (bits == 4) {
    codes[g * 32 + lane] = (uint8_t)(c0 | (c1 << 4));
  } else {
    const uint32_t nib = c0 | (c1 << 2);
    const uint32_t other = __shfl_down_sync(0xFFFFFFFFu, nib, 1);
    if ((lane & 1) == 0) codes[g * 16 + (lane >> 1)] = (uint8_t)(nib | (other << 4));
  }
  if (lane == 0) meta[g] = __halves2half2(s16, m16);
}

// FP8 (E4M3) cache: every value cast by itself, round to nearest even, saturating at 448.
template <typename T>
__global__ void fp8_cast_kernel(const T* __restrict__ x, int64_t n, uint8_t* __restrict__ codes) {
  const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= n) return;
  uint8_t c[4];
#pragma unroll
  for (int e = 0; e < 4; ++e)
    c[e] = i + e < n ? (uint8_t)__nv_cvt_float_to_fp8(to_f(x[i + e]), __NV_SATFINITE, __NV_E4M3) : 0;
  if (i + 3 < n) {
    *reinterpret_cast<uchar4*>(codes + i) = make_uchar4(c[0], c[1], c[2], c[3]);
  } else {
    for (int e = 0; i + e < n; ++e) codes[i + e] = c[e];
  }
}

int32_t launch_quantize(int dtype, const void* x, int n, int n_kv, int hd, int bits, void* codes, void* meta,
                        cudaStream_t st) {
  if (n == 0) return AKVS_OK;
  if (bits == AKVS_KV_FP8) {
    const int64_t total = (int64_t)n * n_kv * hd;          // rows of n_kv * hd bytes: 4-byte stores stay aligned
    if ((n_kv * hd) % 4 != 0) return AKVS_ERR_UNSUPPORTED;
    return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
      using T = decltype(tag);
      fp8_cast_kernel<T><<<akvs_cdiv((total + 3) / 4, 256), 256, 0, st>>>((const T*)x, total, (uint8_t*)codes);
      AKVS_LAUNCHED();
      return AKVS_OK;
    });
  }
  if (hd % 64 != 0 || (bits != 2 && bits != 4)) return AKVS_ERR_UNSUPPORTED;
  const int64_t n_groups = (int64_t)n * n_kv * (hd / 64);
  const int blocks = akvs_cdiv(n_groups, 8);
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    quantize_kernel<T><<<blocks, 256, 0, st>>>((const T*)x, n_groups, bits, (uint8_t*)codes, (__half2*)meta);
    AKVS_LAUNCHED();
    return AKVS_OK;
  });
}
