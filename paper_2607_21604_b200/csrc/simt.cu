// CUDA-core versions of the two contractions.  They are the float (AKVS_F32) path, whose
// 2e-3 tolerance rules out reduced-precision tensor-core inputs, and an independent
// cross-check of the tensor-core kernels in the tests (algo = 1).
#include "common.cuh"

// ---------------------------------------------------------------------------------------
// y[M][N] = x[M][K] w[N][K]^T   (optionally: y = silu(x w^T) * (x w2^T);  or resid += x w^T)
// 64x64 tile, 16-wide k slab, 256 threads, 4x4 outputs per thread, float accumulation.
// ---------------------------------------------------------------------------------------
constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

template <typename T, typename TW, bool DUAL>
__global__ void __launch_bounds__(256)
linear_simt_kernel(const T* __restrict__ x, const TW* __restrict__ w, const TW* __restrict__ w2, T* __restrict__ y,
                   float* __restrict__ resid, int M, int N, int K, int ldy) {
  __shared__ float xs[SG_BK][SG_BM + 4];
  pdl_trigger();
  pdl_wait();
  __shared__ float ws[SG_BK][SG_BN + 4];
  __shared__ float ws2[DUAL ? SG_BK : 1][SG_BN + 4];
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {}, acc2[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
    for (int i = threadIdx.x; i < SG_BM * SG_BK; i += 256) {
      const int r = i / SG_BK, kk = i % SG_BK;
      const int gr = m0 + r, gk = k0 + kk;
      xs[kk][r] = (gr < M && gk < K) ? to_f(x[(size_t)gr * K + gk]) : 0.f;
      const int gn = n0 + r;
      ws[kk][r] = (gn < N && gk < K) ? to_f(w[(size_t)gn * K + gk]) : 0.f;
      if constexpr (DUAL) ws2[kk][r] = (gn < N && gk < K) ? to_f(w2[(size_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < SG_BK; ++kk) {
      float a[4], b[4], b2[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = xs[kk][ty * 4 + i];
        b[i] = ws[kk][tx * 4 + i];
        if constexpr (DUAL) b2[i] = ws2[kk][tx * 4 + i];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
          if constexpr (DUAL) acc2[i][j] = fmaf(a[i], b2[j], acc2[i][j]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gr = m0 + ty * 4 + i;
    if (gr >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = acc[i][j];
      if constexpr (DUAL) v = v / (1.f + __expf(-v)) * acc2[i][j];
      if (resid) resid[(size_t)gr * ldy + gn] += v;
      else y[(size_t)gr * ldy + gn] = from_f<T>(v);
    }
  }
}

int32_t launch_linear_simt(int dtype, const void* x, const void* w, const void* w2, void* y, float* resid,
                           int M, int N, int K, int ldy, cudaStream_t st) {
  if (M == 0 || N == 0) return AKVS_OK;
  const dim3 grid(akvs_cdiv(N, SG_BN), akvs_cdiv(M, SG_BM));
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    if (w2) AKVS_CUDA(launch_pdl(linear_simt_kernel<T, T, true>, grid, dim3(256), 0, st, (const T*)x, (const T*)w, (const T*)w2, (T*)y, resid, M, N, K, ldy));
    else AKVS_CUDA(launch_pdl(linear_simt_kernel<T, T, false>, grid, dim3(256), 0, st, (const T*)x, (const T*)w, (const T*)nullptr, (T*)y, resid, M, N, K, ldy));
    AKVS_LAUNCHED();
    return AKVS_OK;
  });
}

// ---------------------------------------------------------------------------------------
// GQA attention on CUDA cores with an online softmax.
// CTA = 4 warps = 16 query rows of one q head; keys in tiles of 32.  Score phase: lane =
// key; value phase: lane = output dims.  Row r sees keys k_lo[r]..k_hi[r] (inclusive).
// ---------------------------------------------------------------------------------------
constexpr int SA_ROWS = 16, SA_KEYS = 32, SA_RPW = 4;   // rows per CTA, keys per tile, rows per warp

template <typename T, int HD>
__global__ void __launch_bounds__(128)
attention_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ out,
                      const int32_t* __restrict__ k_lo, const int32_t* __restrict__ k_hi,
                      const int32_t* __restrict__ k_lo2, const int32_t* __restrict__ k_hi2, int R, int n_q, int n_kv) {
  extern __shared__ float smem[];
  pdl_trigger();
  pdl_wait();
  float* qs = smem;                               // [SA_ROWS][HD]
  float* ks = qs + SA_ROWS * HD;                  // [SA_KEYS][HD + 1]
  float* vs = ks + SA_KEYS * (HD + 1);            // [SA_KEYS][HD]
  float* ps = vs + SA_KEYS * HD;                  // [SA_ROWS][SA_KEYS]
  constexpr int DPL = HD / 32;                    // output dims per lane
  const int r0 = blockIdx.x * SA_ROWS, hq = blockIdx.y, hk = hq / (n_q / n_kv);
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int nrows = min(SA_ROWS, R - r0);
  const float scale = rsqrtf((float)HD);

  for (int i = threadIdx.x; i < SA_ROWS * HD; i += 128) {
    const int r = i / HD, e = i % HD;
    qs[i] = r < nrows ? to_f(q[((size_t)(r0 + r) * n_q + hq) * HD + e]) * scale : 0.f;
  }
  int lo_r[SA_RPW], hi_r[SA_RPW];
  float m_r[SA_RPW], l_r[SA_RPW], o_r[SA_RPW][DPL];
#pragma unroll
  for (int i = 0; i < SA_RPW; ++i) {
    m_r[i] = -INFINITY;
    l_r[i] = 0.f;
#pragma unroll
    for (int d = 0; d < DPL; ++d) o_r[i][d] = 0.f;
  }
  // A row sees the keys of its first range and, when second-range arrays are given (batched
  // requests: a query row's own context and its own query tokens are not adjacent), of its
  // second range.  Each range is walked over the hull of the block's rows.
  for (int seg = 0; seg < (k_lo2 ? 2 : 1); ++seg) {
  const int32_t* klo = seg ? k_lo2 : k_lo;
  const int32_t* khi = seg ? k_hi2 : k_hi;
  int key_lo = 0x7fffffff, key_hi = -1;
  for (int r = 0; r < nrows; ++r) {
    const int a = klo[r0 + r], b = khi[r0 + r];
    if (a <= b) { key_lo = min(key_lo, a); key_hi = max(key_hi, b); }
  }
#pragma unroll
  for (int i = 0; i < SA_RPW; ++i) {
    const int r = wid * SA_RPW + i;
    lo_r[i] = r < nrows ? klo[r0 + r] : 1;
    hi_r[i] = r < nrows ? khi[r0 + r] : 0;
  }
  for (int t0 = key_lo; t0 <= key_hi; t0 += SA_KEYS) {
    __syncthreads();
    for (int i = threadIdx.x; i < SA_KEYS * HD; i += 128) {
      const int jj = i / HD, e = i % HD;
      const int j = t0 + jj;
      const bool ok = j <= key_hi;
      ks[jj * (HD + 1) + e] = ok ? to_f(k[((size_t)j * n_kv + hk) * HD + e]) : 0.f;
      vs[jj * HD + e] = ok ? to_f(v[((size_t)j * n_kv + hk) * HD + e]) : 0.f;
    }
    __syncthreads();
    const int j = t0 + lane;
#pragma unroll
    for (int i = 0; i < SA_RPW; ++i) {
      const int r = wid * SA_RPW + i;
      float s = 0.f;
      const float* qp = qs + r * HD;
      const float* kp = ks + lane * (HD + 1);
#pragma unroll 16
      for (int e = 0; e < HD; ++e) s = fmaf(qp[e], kp[e], s);
      const bool vis = j >= lo_r[i] && j <= hi_r[i];
      s = vis ? s : -INFINITY;
      const float tmax = warp_max(s);
      const float m_new = fmaxf(m_r[i], tmax);
      // a row with nothing visible so far keeps m = -inf; guard the exponentials
      const float corr = m_new == -INFINITY ? 1.f : __expf(m_r[i] - m_new);
      const float p = vis ? __expf(s - m_new) : 0.f;
      l_r[i] = l_r[i] * corr + warp_sum(p);
      m_r[i] = m_new;
      ps[r * SA_KEYS + lane] = p;
#pragma unroll
      for (int d = 0; d < DPL; ++d) o_r[i][d] *= corr;
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < SA_RPW; ++i) {
      const float* pp = ps + (wid * SA_RPW + i) * SA_KEYS;
#pragma unroll 8
      for (int jj = 0; jj < SA_KEYS; ++jj) {
        const float p = pp[jj];
#pragma unroll
        for (int d = 0; d < DPL; ++d) o_r[i][d] = fmaf(p, vs[jj * HD + lane + 32 * d], o_r[i][d]);
      }
    }
  }
  }
#pragma unroll
  for (int i = 0; i < SA_RPW; ++i) {
    const int r = wid * SA_RPW + i;
    if (r >= nrows) continue;
    const float inv = l_r[i] > 0.f ? 1.f / l_r[i] : 0.f;
#pragma unroll
    for (int d = 0; d < DPL; ++d)
      out[((size_t)(r0 + r) * n_q + hq) * HD + lane + 32 * d] = from_f<T>(o_r[i][d] * inv);
  }
}

template <typename T, int HD>
static int32_t launch_attention_simt_t(const void* q, const void* k, const void* v, void* out, const int32_t* k_lo,
                                       const int32_t* k_hi, const int32_t* k_lo2, const int32_t* k_hi2, int R, int n_q,
                                       int n_kv, cudaStream_t st) {
  const size_t smem = sizeof(float) * (SA_ROWS * HD + SA_KEYS * (HD + 1) + SA_KEYS * HD + SA_ROWS * SA_KEYS);
  const dim3 grid(akvs_cdiv(R, SA_ROWS), n_q);
  AKVS_CUDA(launch_pdl(attention_simt_kernel<T, HD>, grid, dim3(128), smem, st, (const T*)q, (const T*)k, (const T*)v, (T*)out,
                       k_lo, k_hi, k_lo2, k_hi2, R, n_q, n_kv));
  AKVS_LAUNCHED();
  return AKVS_OK;
}

int32_t launch_attention_simt(int dtype, const void* q, const void* k, const void* v, void* out,
                              const int32_t* k_lo, const int32_t* k_hi, const int32_t* k_lo2, const int32_t* k_hi2,
                              int R, int n_q, int n_kv, int hd, cudaStream_t st) {
  if (R == 0) return AKVS_OK;
  if (n_kv <= 0 || n_q % n_kv != 0) return AKVS_ERR_SHAPE;
  return dispatch_dtype(dtype, [&](auto tag) -> int32_t {
    using T = decltype(tag);
    if (hd == 64) return launch_attention_simt_t<T, 64>(q, k, v, out, k_lo, k_hi, k_lo2, k_hi2, R, n_q, n_kv, st);
    if (hd == 128) return launch_attention_simt_t<T, 128>(q, k, v, out, k_lo, k_hi, k_lo2, k_hi2, R, n_q, n_kv, st);
    return AKVS_ERR_UNSUPPORTED;
  });
}
