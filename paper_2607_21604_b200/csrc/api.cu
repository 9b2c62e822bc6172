// C ABI of the library and the per-layer schedule behind it.  Host code only enqueues
// kernels on the caller's stream; the single host<-device read is the row count at the end
// of akvs_select_probes.
#include <vector>
#include <functional>
#include <new>

#include "common.cuh"

unsigned long long g_akvs_launches = 0;

// ----------------------------------------------------------------------------- profiling hooks
namespace {
struct ProfRec { cudaEvent_t a, b; int sub; double work; };
int g_prof_kind = 0;
std::vector<ProfRec> g_prof;
size_t g_prof_used = 0;
}  // namespace

void akvs_prof_mark(int kind, int sub, double work, bool begin, cudaStream_t st) {
  if (!((g_prof_kind >> kind) & 1) || g_prof_used >= g_prof.size()) return;
  ProfRec& r = g_prof[g_prof_used];
  if (begin) {
    r.sub = (kind << 8) | sub;
    r.work = work;
    cudaEventRecord(r.a, st);
  } else {
    cudaEventRecord(r.b, st);
    ++g_prof_used;
  }
}

namespace {

constexpr uint32_t kCtxMagic = 0x616B7673u;   // "akvs"

struct Dims {
  int L, d, nq, nkv, hd, f, vocab, dq, dkv, dtype;
  size_t es;                                  // element size of the model dtype
};

int32_t check_model(const akvs_model_desc* m, Dims& D) {
  if (!m) return AKVS_ERR_INVALID_ARG;
  if (m->dtype != AKVS_F32 && m->dtype != AKVS_BF16 && m->dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  if (m->n_layers <= 0 || m->d_model <= 0 || m->n_q_heads <= 0 || m->n_kv_heads <= 0 || m->head_dim <= 0 ||
      m->d_ff <= 0 || m->vocab <= 0)
    return AKVS_ERR_INVALID_ARG;
  if (m->n_q_heads % m->n_kv_heads != 0) return AKVS_ERR_SHAPE;
  if (m->head_dim != 64 && m->head_dim != 128) return AKVS_ERR_UNSUPPORTED;
  if (m->d_model % 8 != 0 || m->d_ff % 8 != 0) return AKVS_ERR_SHAPE;
  if (!m->tok_emb || !m->final_norm || !m->attn_norm || !m->wq || !m->wk || !m->wv || !m->wo || !m->mlp_norm ||
      !m->w_gate || !m->w_up || !m->w_down)
    return AKVS_ERR_INVALID_ARG;
  for (int l = 0; l < m->n_layers; ++l)
    if (!m->attn_norm[l] || !m->wq[l] || !m->wk[l] || !m->wv[l] || !m->wo[l] || !m->mlp_norm[l] || !m->w_gate[l] ||
        !m->w_up[l] || !m->w_down[l])
      return AKVS_ERR_INVALID_ARG;
  D.L = m->n_layers; D.d = m->d_model; D.nq = m->n_q_heads; D.nkv = m->n_kv_heads; D.hd = m->head_dim;
  D.f = m->d_ff; D.vocab = m->vocab; D.dq = D.nq * D.hd; D.dkv = D.nkv * D.hd; D.dtype = m->dtype;
  D.es = dtype_size(m->dtype);
  return AKVS_OK;
}

// Bump allocator over the caller's workspace.  With base == nullptr it only measures.
struct Carver {
  char* base;
  int64_t off = 0;
  explicit Carver(void* b) : base(reinterpret_cast<char*>(b)) {}
  template <typename T> T* take(int64_t count) {
    off = akvs_align_up(off, 256);
    T* p = base ? reinterpret_cast<T*>(base + off) : nullptr;
    off += count * (int64_t)sizeof(T);
    return p;
  }
  void* take_bytes(int64_t bytes) { return take<char>(bytes); }
};

struct Workspace {
  int32_t* status;          // [16]: [0] status word, [4..5] row counts
  int32_t* ctx_off;         // [M+1]
  int32_t* slot_src_off;    // [M]
  int32_t* probe_off;       // [M+1]
  int32_t* tok_unit;        // [N]
  int32_t* tok_src;         // [N]
  int32_t* row_of_pos;      // [T]
  int4* tok_meta;           // [2][T] K and V records of the correction pass
  uint8_t* flags;           // [2N]: kflag, vflag
  uint64_t* keys;           // [2N]
  int32_t* pos;             // [T] 0..T-1 (or unit-local positions while encoding)
  int32_t* lo;              // [T] attention lower bounds
  int32_t* zeros;           // [T]
  int32_t* unit_pos;        // [M+1] batched requests: position of a unit inside its own request
  int32_t* tok_pos;         // [T]   batched requests: position of a token inside its own request
  int32_t* tok_rng;         // [4][T] batched requests: visible key ranges (lo1, hi1, lo2, hi2) per token
  int32_t* row_meta;        // [5][T] the same five arrays gathered for the recomputed rows
  float2* rope;             // [T][hd/2]
  float* mu_k;              // [M][dkv]
  float* mu_v;
  float* h;                 // [T][d] residual stream
  float* stash_h;           // [T][d] hidden state entering the check layer
  void* x;                  // [T][d]
  void* q;                  // [T][dq]
  void* k;                  // [T][dkv]
  void* v;
  void* ao;                 // [T][dq]
  void* act;                // [T][f]
  void* stash_k;            // [check_layer-1][T][dkv]
  void* stash_v;
  int64_t bytes;
  int rope_n;               // positions the RoPE table was built for (host-side note for the bounds guards)
};

Workspace carve(const Dims& D, int N, int nq, int M, int check_layer, void* base) {
  const int64_t T = (int64_t)N + nq;
  Carver c(base);
  Workspace w;
  w.status = c.take<int32_t>(16);
  w.ctx_off = c.take<int32_t>(M + 1);
  w.slot_src_off = c.take<int32_t>(M + 1);
  w.probe_off = c.take<int32_t>(M + 1);
  w.tok_unit = c.take<int32_t>(N);
  w.tok_src = c.take<int32_t>(N);
  w.row_of_pos = c.take<int32_t>(T);
  w.tok_meta = c.take<int4>(2 * T);
  w.flags = c.take<uint8_t>(2 * (int64_t)N);
  w.keys = c.take<uint64_t>(2 * (int64_t)N);
  w.pos = c.take<int32_t>(T);
  w.lo = c.take<int32_t>(T);
  w.zeros = c.take<int32_t>(T);
  w.unit_pos = c.take<int32_t>(M + 1);
  w.tok_pos = c.take<int32_t>(T);
  w.tok_rng = c.take<int32_t>(4 * T);
  w.row_meta = c.take<int32_t>(5 * T);
  w.rope = c.take<float2>(T * (D.hd / 2));
  w.mu_k = c.take<float>((int64_t)M * D.dkv);
  w.mu_v = c.take<float>((int64_t)M * D.dkv);
  w.h = c.take<float>(T * D.d);
  w.stash_h = c.take<float>(T * D.d);
  w.x = c.take_bytes(T * D.d * D.es);
  w.q = c.take_bytes(T * D.dq * D.es);
  w.k = c.take_bytes(T * D.dkv * D.es);
  w.v = c.take_bytes(T * D.dkv * D.es);
  w.ao = c.take_bytes(T * D.dq * D.es);
  w.act = c.take_bytes(T * D.f * D.es);
  const int64_t nd = check_layer > 1 ? check_layer - 1 : 0;
  w.stash_k = c.take_bytes(nd * T * D.dkv * D.es);
  w.stash_v = c.take_bytes(nd * T * D.dkv * D.es);
  w.bytes = akvs_align_up(c.off, 256);
  w.rope_n = (int)T;
  return w;
}

int32_t check_workspace(const void* ws, int64_t have, int64_t need) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return AKVS_ERR_WORKSPACE;
  if (have < need) return AKVS_ERR_WORKSPACE;
  return AKVS_OK;
}

struct Ctx {                   // host object that carries a request from selection to prefill
  uint32_t magic;
  int N, nq, M, B, check_layer, n_probe_total;
  void* workspace;
};

// ----------------------------------------------------------------------------- linear layers
int g_bf16_linear_algo = 0;    // 16-bit models: 0 = tcgen05; 1 = CUDA cores (kept for cross-checking)
int g_linear_tiling = 0;       // tcgen05 linear layers: 0 = by shape; 1 = single CTAs; 2 = CTA pairs (cross-checking)
int g_linear_splits = 0;       // residual linear layers: 0 = split-K by the cost model; 1..4 = forced (comparisons)

// Projections that share the input x.  Segments whose bit is set in rope_mask are [M][heads][hd]
// tensors that get RoPE at pos[row]: fused into the tensor-core epilogue when hd == 128,
// otherwise done by the rotation kernel afterwards.
int32_t linear_multi(const Dims& D, const void* x, int M, int K, int n_seg, const void* const* w, const int* n,
                     void* const* out, const int* ldc, int32_t* status, cudaStream_t st,
                     const float2* rope = nullptr, const int32_t* pos = nullptr, int rope_mask = 0,
                     float rope_base = 0.f, int n_pos = 0) {
  bool tc_ok = D.dtype != AKVS_F32 && g_bf16_linear_algo == 0 && K % 8 == 0;
  for (int i = 0; i < n_seg; ++i) tc_ok = tc_ok && n[i] % 128 == 0;
  const bool fuse = tc_ok && D.hd == 128;
  if (tc_ok) {
    AKVS_TRY(launch_linear_tc(D.dtype, 0, x, M, K, n_seg, w, n, out, ldc, status, st, fuse ? rope : nullptr, pos,
                              rope_mask, g_linear_tiling, n_pos));
  } else {
    for (int i = 0; i < n_seg; ++i)
      AKVS_TRY(launch_linear_simt(D.dtype, x, w[i], nullptr, out[i], nullptr, M, n[i], K, ldc[i], st));
  }
  if (!fuse)
    for (int i = 0; i < n_seg; ++i)
      if ((rope_mask >> i) & 1)
        AKVS_TRY(launch_rope(D.dtype, out[i], pos, M, n[i] / D.hd, D.hd, ldc[i], rope, n_pos, status, rope_base, st));
  return AKVS_OK;
}
// split_ok: the k range may be cut into ordered partial sums where that fills the device.  Off
// for the unit encoder and the dense front, whose K/V of a unit at offset 0 are then the same
// bits (one accumulation chain per element whatever the launch shape), so that such a unit scores
// exactly zero at the check layer, as in exact arithmetic.
int32_t linear_resid(const Dims& D, const void* x, int M, int K, const void* w, int n, float* h, int32_t* status,
                     cudaStream_t st, bool split_ok) {
  if (D.dtype != AKVS_F32 && g_bf16_linear_algo == 0 && K % 8 == 0 && n % 128 == 0) {
    void* out = h;
    return launch_linear_tc(D.dtype, 1, x, M, K, 1, &w, &n, &out, &n, status, st, nullptr, nullptr, 0, g_linear_tiling, 0,
                            split_ok ? g_linear_splits : 1);
  }
  return launch_linear_simt(D.dtype, x, w, nullptr, nullptr, h, M, n, K, n, st);
}
int32_t linear_swiglu(const Dims& D, const void* x, int M, int K, const void* wg, const void* wu, int n, void* act,
                      int32_t* status, cudaStream_t st) {
  if (D.dtype != AKVS_F32 && g_bf16_linear_algo == 0 && K % 8 == 0 && n % 128 == 0) {
    const void* w[2] = {wg, wu};
    const int ns[2] = {n, n};
    void* out[2] = {act, act};
    const int ld[2] = {n, n};
    return launch_linear_tc(D.dtype, 2, x, M, K, 2, w, ns, out, ld, status, st, nullptr, nullptr, 0, g_linear_tiling);
  }
  return launch_linear_simt(D.dtype, x, wg, wu, act, nullptr, M, n, K, n, st);
}

// One decoder layer over `n` rows held in ws.h.  k_dst/v_dst receive the rows' fresh K
// (rotated at `pos`) and V; `between` runs after RoPE and before attention (store to the
// cache, or estimate offsets and assemble the corrected K/V); attention then reads
// attn_k/attn_v with per-row key ranges [lo, hi].
int g_attention_algo = 0;       // 16-bit models with head_dim 128: 0 = tcgen05; 1 = CUDA cores

// Per-row geometry of a set of rows: RoPE position and visible key ranges.  lo2/hi2 are null
// for a single request (one contiguous causal range per row).
struct RowGeom {
  const int32_t* pos;
  const int32_t* lo;
  const int32_t* hi;
  const int32_t* lo2;
  const int32_t* hi2;
};

int32_t attention(const Dims& D, const void* q, const void* k, const void* v, void* out, const RowGeom& g, int n,
                  int n_keys, int32_t* status, cudaStream_t st) {
  if (D.dtype != AKVS_F32 && D.hd == 128 && g_attention_algo == 0)
    return launch_attention_tc(D.dtype, q, k, v, out, g.lo, g.hi, g.lo2, g.hi2, n, n_keys, D.nq, D.nkv, status, st);
  return launch_attention_simt(D.dtype, q, k, v, out, g.lo, g.hi, g.lo2, g.hi2, n, D.nq, D.nkv, D.hd, st);
}

int32_t run_layer(const akvs_model_desc* m, const Dims& D, int l, const Workspace& ws, int n, const RowGeom& g,
                  void* k_dst, void* v_dst, const void* attn_k, const void* attn_v, int n_keys,
                  const std::function<int32_t()>& between, cudaStream_t st, bool split_ok = false) {
  if (n == 0) return between ? between() : AKVS_OK;
  AKVS_TRY(launch_rmsnorm(D.dtype, ws.h, m->attn_norm[l], m->rms_eps, n, D.d, ws.x, st));
  {
    const void* w[3] = {m->wq[l], m->wk[l], m->wv[l]};
    const int ns[3] = {D.dq, D.dkv, D.dkv};
    void* out[3] = {ws.q, k_dst, v_dst};
    AKVS_TRY(linear_multi(D, ws.x, n, D.d, 3, w, ns, out, ns, ws.status, st, ws.rope, g.pos, 0b011, m->rope_base,
                          ws.rope_n));
  }
  if (between) AKVS_TRY(between());
  AKVS_TRY(attention(D, ws.q, attn_k, attn_v, ws.ao, g, n, n_keys, ws.status, st));
  AKVS_TRY(linear_resid(D, ws.ao, n, D.dq, m->wo[l], D.d, ws.h, ws.status, st, split_ok));
  AKVS_TRY(launch_rmsnorm(D.dtype, ws.h, m->mlp_norm[l], m->rms_eps, n, D.d, ws.x, st));
  AKVS_TRY(linear_swiglu(D, ws.x, n, D.d, m->w_gate[l], m->w_up[l], D.f, ws.act, ws.status, st));
  AKVS_TRY(linear_resid(D, ws.act, n, D.f, m->w_down[l], D.d, ws.h, ws.status, st, split_ok));
  return AKVS_OK;
}

size_t kv_row_bytes(const Dims& D, int fmt) {
  return fmt == AKVS_KV_NATIVE ? (size_t)D.dkv * D.es : (size_t)D.dkv * fmt / 8;
}

KvLayer cache_layer(const akvs_cache* c, const Dims& D, int l) {
  KvLayer kv;
  const size_t stride = (size_t)c->n_tokens * kv_row_bytes(D, c->kv_format);
  kv.k = reinterpret_cast<const char*>(c->k) + l * stride;
  kv.v = reinterpret_cast<const char*>(c->v) + l * stride;
  kv.fmt = c->kv_format;
  if (c->kv_format == AKVS_KV_NATIVE || c->kv_format == AKVS_KV_FP8) {
    kv.k_meta = kv.v_meta = nullptr;
  } else {
    const size_t ms = (size_t)c->n_tokens * D.nkv * (D.hd / 64) * 4;
    kv.k_meta = reinterpret_cast<const char*>(c->k_meta) + l * ms;
    kv.v_meta = reinterpret_cast<const char*>(c->v_meta) + l * ms;
  }
  return kv;
}

// The caller may be streaming layer l of the cache in on another stream: wait for its event.
int32_t wait_layer(const akvs_cache* c, int l, cudaStream_t st) {
  if (c->layer_ready && c->layer_ready[l])
    AKVS_CUDA(cudaStreamWaitEvent(st, reinterpret_cast<cudaEvent_t>(c->layer_ready[l]), 0));
  return AKVS_OK;
}

int32_t check_cache(const akvs_cache* c, const Dims& D, bool need_kv) {
  if (!c || !c->unit_off || !c->token_ids) return AKVS_ERR_INVALID_ARG;
  if (c->n_units < 0 || c->n_tokens < 0) return AKVS_ERR_INVALID_ARG;
  const bool grouped = c->kv_format == AKVS_KV_Q4 || c->kv_format == AKVS_KV_Q2;
  if (c->kv_format != AKVS_KV_NATIVE && c->kv_format != AKVS_KV_FP8 && !grouped) return AKVS_ERR_UNSUPPORTED;
  if (grouped && D.hd % 64 != 0) return AKVS_ERR_UNSUPPORTED;
  if (c->unit_off[0] != 0 || c->unit_off[c->n_units] != c->n_tokens) return AKVS_ERR_SHAPE;
  for (int u = 0; u < c->n_units; ++u)
    if (c->unit_off[u + 1] < c->unit_off[u]) return AKVS_ERR_SHAPE;
  if (need_kv) {
    if (!c->k || !c->v) return AKVS_ERR_INVALID_ARG;
    if (grouped && (!c->k_meta || !c->v_meta)) return AKVS_ERR_INVALID_ARG;
  }
  return AKVS_OK;
}

// Boundaries of the requests of a batch in the merged token order (all context tokens, request
// after request, then all query tokens, request after request).  B == 1: a single request.
struct Batch {
  int B = 1;
  std::vector<int32_t> unit_off;    // [B+1] into the unit list
  std::vector<int32_t> ctx_start;   // [B+1] into the context tokens
  std::vector<int32_t> qry_start;   // [B+1] into the query tokens
};

int32_t check_batch(const akvs_request* r, const std::vector<int32_t>& ctx_off, Batch& b) {
  b.B = r->n_requests > 1 ? r->n_requests : 1;
  if (r->n_requests < 0) return AKVS_ERR_INVALID_ARG;
  if (b.B == 1) {
    b.unit_off = {0, r->n_units};
    b.ctx_start = {0, ctx_off[r->n_units]};
    b.qry_start = {0, r->n_query};
    return AKVS_OK;
  }
  if (!r->req_unit_off || !r->req_query_off) return AKVS_ERR_INVALID_ARG;
  if (r->req_unit_off[0] != 0 || r->req_unit_off[b.B] != r->n_units) return AKVS_ERR_SHAPE;
  if (r->req_query_off[0] != 0 || r->req_query_off[b.B] != r->n_query) return AKVS_ERR_SHAPE;
  b.unit_off.assign(r->req_unit_off, r->req_unit_off + b.B + 1);
  b.qry_start.assign(r->req_query_off, r->req_query_off + b.B + 1);
  b.ctx_start.assign(b.B + 1, 0);
  for (int i = 0; i < b.B; ++i) {
    if (b.unit_off[i + 1] < b.unit_off[i] || b.qry_start[i + 1] < b.qry_start[i]) return AKVS_ERR_SHAPE;
    b.ctx_start[i + 1] = ctx_off[b.unit_off[i + 1]];
  }
  return AKVS_OK;
}

int32_t check_request(const akvs_request* r, const akvs_cache* c, std::vector<int32_t>& ctx_off,
                      std::vector<int32_t>& slot_src) {
  if (!r || r->n_units < 0 || r->n_query < 0) return AKVS_ERR_INVALID_ARG;
  if (r->n_units > 0 && !r->unit_ids) return AKVS_ERR_INVALID_ARG;
  if (r->n_query > 0 && !r->query_ids) return AKVS_ERR_INVALID_ARG;
  ctx_off.assign(r->n_units + 1, 0);
  slot_src.assign(r->n_units + 1, 0);
  for (int s = 0; s < r->n_units; ++s) {
    const int u = r->unit_ids[s];
    if (u < 0 || u >= c->n_units) return AKVS_ERR_INVALID_ARG;
    ctx_off[s + 1] = ctx_off[s] + (c->unit_off[u + 1] - c->unit_off[u]);
    slot_src[s] = c->unit_off[u];
  }
  return AKVS_OK;
}

__global__ void local_pos_kernel(const int32_t* __restrict__ ctx_off, const int32_t* __restrict__ tok_unit, int N,
                                 int32_t* __restrict__ pos, int32_t* __restrict__ lo) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= N) return;
  const int a = ctx_off[tok_unit[j]];
  pos[j] = j - a;
  lo[j] = a;
}

// Uploads the request's offsets and builds the maps every mode needs.
__global__ void gather_i32_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ idx, int n, int n_src,
                                  int stride_src, int stride_dst, int n_arrays, int32_t* status,
                                  int32_t* __restrict__ dst) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  int j = idx[i];
  if (j < 0 || j >= n_src) {                    // idx may be caller data (akvs_probes.rows)
    set_status(status, AKVS_ERR_INVALID_ARG);
    j = 0;
  }
  for (int a = 0; a < n_arrays; ++a) dst[(size_t)a * stride_dst + i] = src[(size_t)a * stride_src + j];
}

// Batched requests: per-token position inside the token's own request and the key ranges it
// sees in the merged order.  Context token j of request b sees [ctx_start_b, j]; query token
// t = N + i of request b sees its whole context [ctx_start_b, ctx_start_{b+1}) and the query
// tokens [N + qry_start_b, t].  tok_pos and the four range arrays are contiguous (5 x T).
int32_t setup_batch(const Workspace& ws, const std::vector<int32_t>& ctx_off, const Batch& b, int M, int N, int nq,
                    cudaStream_t st) {
  const int T = N + nq;
  std::vector<int32_t> unit_pos(M + 1, 0), arr((size_t)5 * T);
  int32_t* pos = arr.data();
  int32_t* lo1 = pos + T;
  int32_t* hi1 = lo1 + T;
  int32_t* lo2 = hi1 + T;
  int32_t* hi2 = lo2 + T;
  for (int r = 0; r < b.B; ++r) {
    const int cs = b.ctx_start[r], ce = b.ctx_start[r + 1], qs = b.qry_start[r], qe = b.qry_start[r + 1];
    for (int u = b.unit_off[r]; u < b.unit_off[r + 1]; ++u) unit_pos[u] = ctx_off[u] - cs;
    for (int j = cs; j < ce; ++j) { pos[j] = j - cs; lo1[j] = cs; hi1[j] = j; lo2[j] = 1; hi2[j] = 0; }
    for (int i = qs; i < qe; ++i) {
      const int t = N + i;
      pos[t] = (ce - cs) + (i - qs); lo1[t] = cs; hi1[t] = ce - 1; lo2[t] = N + qs; hi2[t] = t;
    }
  }
  AKVS_CUDA(cudaMemcpyAsync(ws.unit_pos, unit_pos.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  if (T > 0) {
    AKVS_CUDA(cudaMemcpyAsync(ws.tok_pos, pos, (size_t)T * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    AKVS_CUDA(cudaMemcpyAsync(ws.tok_rng, lo1, (size_t)4 * T * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    // the vectors die with this frame: pageable copies are staged before the call returns, but do not rely on it
    AKVS_CUDA(cudaStreamSynchronize(st));
  }
  return AKVS_OK;
}

// Geometry of all T tokens taken as rows (dense layers, full recompute).
RowGeom token_geom(const Workspace& ws, const Batch& b, int T) {
  if (b.B == 1) return RowGeom{ws.pos, ws.zeros, ws.pos, nullptr, nullptr};
  return RowGeom{ws.tok_pos, ws.tok_rng, ws.tok_rng + T, ws.tok_rng + 2 * (size_t)T, ws.tok_rng + 3 * (size_t)T};
}

// Geometry of the recomputed rows `rows[0..R)` (merged token indices, device).
int32_t row_geom(const Workspace& ws, const Batch& b, const int32_t* rows, int R, int T, RowGeom& g, cudaStream_t st) {
  if (b.B == 1) { g = RowGeom{rows, ws.zeros, rows, nullptr, nullptr}; return AKVS_OK; }
  if (R > 0) {
    gather_i32_kernel<<<akvs_cdiv(R, 256), 256, 0, st>>>(ws.tok_pos, rows, R, T, 0, 0, 1, ws.status, ws.row_meta);
    AKVS_LAUNCHED();
    gather_i32_kernel<<<akvs_cdiv(R, 256), 256, 0, st>>>(ws.tok_rng, rows, R, T, T, T, 4, ws.status, ws.row_meta + T);
    AKVS_LAUNCHED();
  }
  g = RowGeom{ws.row_meta, ws.row_meta + T, ws.row_meta + 2 * (size_t)T, ws.row_meta + 3 * (size_t)T,
              ws.row_meta + 4 * (size_t)T};
  return AKVS_OK;
}

int32_t setup_request(const Dims& D, const Workspace& ws, const std::vector<int32_t>& ctx_off,
                      const std::vector<int32_t>& slot_src, int M, int N, int nq, cudaStream_t st) {
  const int T = N + nq;
  AKVS_CUDA(cudaMemsetAsync(ws.status, 0, 16 * sizeof(int32_t), st));
  AKVS_CUDA(cudaMemcpyAsync(ws.ctx_off, ctx_off.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_CUDA(cudaMemcpyAsync(ws.slot_src_off, slot_src.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_TRY(launch_tok_maps(ws.ctx_off, ws.slot_src_off, M, N, ws.tok_unit, ws.tok_src, st));
  AKVS_TRY(launch_iota(ws.pos, T, 0, st));
  if (T > 0) AKVS_CUDA(cudaMemsetAsync(ws.zeros, 0, (size_t)T * sizeof(int32_t), st));
  return AKVS_OK;
}

ReqMaps req_maps(const Workspace& ws, int N, bool batched = false) {
  ReqMaps mp;
  mp.ctx_off = ws.ctx_off;
  mp.unit_pos = batched ? ws.unit_pos : ws.ctx_off;
  mp.tok_unit = ws.tok_unit;
  mp.tok_src = ws.tok_src;
  mp.row_of_pos = ws.row_of_pos;
  mp.kflag = ws.flags;
  mp.vflag = ws.flags + N;
  mp.tok_meta = ws.tok_meta;
  return mp;
}

// Embeds context (through the store's token ids) and query rows into ws.h.
int32_t embed_all(const akvs_model_desc* m, const Dims& D, const akvs_cache* c, const akvs_request* r,
                  const Workspace& ws, int N, cudaStream_t st) {
  AKVS_TRY(launch_embed(D.dtype, m->tok_emb, c->token_ids, ws.tok_src, N, D.d, D.vocab, ws.status, ws.h, st));
  AKVS_TRY(launch_embed(D.dtype, m->tok_emb, r->query_ids, nullptr, r->n_query, D.d, D.vocab, ws.status,
                        ws.h + (size_t)N * D.d, st));
  return AKVS_OK;
}

}  // namespace

// =========================================================================================
extern "C" {

int32_t akvs_debug_set_linear_algo(int32_t algo) {
  g_bf16_linear_algo = algo & 1;
  g_attention_algo = (algo >> 1) & 1;
  g_linear_tiling = (algo >> 2) & 3;
  if (g_linear_tiling == 3) g_linear_tiling = 0;
  g_linear_splits = (algo >> 4) & 7;
  if (g_linear_splits > 4) g_linear_splits = 0;
  return AKVS_OK;
}

int64_t akvs_launch_count(void) { return (int64_t)g_akvs_launches; }

int32_t akvs_prof_enable(int32_t kind, int32_t max_records) {
  for (ProfRec& r : g_prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  g_prof.clear();
  g_prof_used = 0;
  g_prof_kind = kind;
  if (kind == 0) return AKVS_OK;
  if (max_records < 0) return AKVS_ERR_INVALID_ARG;
  g_prof.resize(max_records);
  for (ProfRec& r : g_prof)
    if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return AKVS_ERR_CUDA;
  return AKVS_OK;
}

int32_t akvs_prof_reset(void) {
  g_prof_used = 0;
  return AKVS_OK;
}

int32_t akvs_prof_read(int32_t capacity, float* ms, double* work, int32_t* sub, int32_t* n_out) {
  if (!ms || !work || !sub || !n_out || capacity < 0) return AKVS_ERR_INVALID_ARG;
  const size_t n = g_prof_used < (size_t)capacity ? g_prof_used : (size_t)capacity;
  for (size_t i = 0; i < n; ++i) {
    if (cudaEventSynchronize(g_prof[i].b) != cudaSuccess) return AKVS_ERR_CUDA;
    if (cudaEventElapsedTime(&ms[i], g_prof[i].a, g_prof[i].b) != cudaSuccess) return AKVS_ERR_CUDA;
    work[i] = g_prof[i].work;
    sub[i] = g_prof[i].sub;
  }
  *n_out = (int32_t)n;
  return AKVS_OK;
}

int32_t akvs_workspace_bytes(const akvs_model_desc* model, int32_t n_ctx, int32_t n_query, int32_t n_units,
                             int32_t check_layer, int64_t* out_bytes) {
  Dims D;
  AKVS_TRY(check_model(model, D));
  if (!out_bytes || n_ctx < 0 || n_query < 0 || n_units < 0 || check_layer < 1 || check_layer > D.L)
    return AKVS_ERR_INVALID_ARG;
  *out_bytes = carve(D, n_ctx, n_query, n_units, check_layer, nullptr).bytes;
  return AKVS_OK;
}

int32_t akvs_encode_units(const akvs_model_desc* model, akvs_cache* cache, void* workspace, int64_t ws_bytes,
                          void* stream) {
  Dims D;
  AKVS_TRY(check_model(model, D));
  AKVS_TRY(check_cache(cache, D, true));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int N = cache->n_tokens, M = cache->n_units;
  Workspace ws = carve(D, N, 0, M, 1, workspace);
  AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
  std::vector<int32_t> off(cache->unit_off, cache->unit_off + M + 1), src(M + 1, 0);
  for (int u = 0; u < M; ++u) src[u] = off[u];
  AKVS_TRY(setup_request(D, ws, off, src, M, N, 0, st));
  if (N == 0) return AKVS_OK;
  int max_len = 0;
  for (int u = 0; u < M; ++u) max_len = off[u + 1] - off[u] > max_len ? off[u + 1] - off[u] : max_len;
  AKVS_TRY(launch_rope_table(model->rope_base, D.hd, max_len, ws.rope, st));
  ws.rope_n = max_len;
  local_pos_kernel<<<akvs_cdiv(N, 256), 256, 0, st>>>(ws.ctx_off, ws.tok_unit, N, ws.row_of_pos, ws.lo);
  AKVS_LAUNCHED();
  const int32_t* local_pos = ws.row_of_pos;     // unit-local positions; ws.pos stays 0..N-1 = row index
  AKVS_TRY(launch_embed(D.dtype, model->tok_emb, cache->token_ids, nullptr, N, D.d, D.vocab, ws.status, ws.h, st));
  const bool native = cache->kv_format == AKVS_KV_NATIVE;
  const size_t lstride = (size_t)N * kv_row_bytes(D, cache->kv_format);
  const size_t mstride = (size_t)N * D.nkv * (D.hd / 64) * 4;
  for (int l = 0; l < D.L; ++l) {
    // native cache: the layer's K/V go straight into the store; quantised cache: attention
    // inside the unit reads the unquantised K/V and the codes are written beside
    void* k_dst = native ? reinterpret_cast<char*>(cache->k) + l * lstride : ws.k;
    void* v_dst = native ? reinterpret_cast<char*>(cache->v) + l * lstride : ws.v;
    std::function<int32_t()> store;
    if (!native)
      store = [&, l]() -> int32_t {
        const bool has_meta = cache->kv_format != AKVS_KV_FP8;
        AKVS_TRY(launch_quantize(D.dtype, ws.k, N, D.nkv, D.hd, cache->kv_format,
                                 reinterpret_cast<char*>(cache->k) + l * lstride,
                                 has_meta ? reinterpret_cast<char*>(cache->k_meta) + l * mstride : nullptr, st));
        return launch_quantize(D.dtype, ws.v, N, D.nkv, D.hd, cache->kv_format,
                               reinterpret_cast<char*>(cache->v) + l * lstride,
                               has_meta ? reinterpret_cast<char*>(cache->v_meta) + l * mstride : nullptr, st);
      };
    AKVS_TRY(run_layer(model, D, l, ws, N, RowGeom{local_pos, ws.lo, ws.pos, nullptr, nullptr}, k_dst, v_dst, k_dst,
                       v_dst, N, store, st));
  }
  return AKVS_OK;
}

int32_t akvs_select_probes(const akvs_model_desc* model, const akvs_cache* cache, const akvs_request* req,
                           int32_t refresh_bp, int32_t check_layer, akvs_probes* out, void** ctx_inout,
                           void* workspace, int64_t ws_bytes, void* stream) {
  Dims D;
  AKVS_TRY(check_model(model, D));
  AKVS_TRY(check_cache(cache, D, true));
  if (!out || !ctx_inout || refresh_bp < 0 || refresh_bp > 10000 || check_layer < 1 || check_layer > D.L)
    return AKVS_ERR_INVALID_ARG;
  if (!out->ctx_off || !out->probe_off || !out->sk_idx || !out->sv_idx || !out->w_k || !out->w_v || !out->d_k ||
      !out->d_v || !out->rows)
    return AKVS_ERR_INVALID_ARG;
  std::vector<int32_t> ctx_off, slot_src;
  AKVS_TRY(check_request(req, cache, ctx_off, slot_src));
  Batch batch;
  AKVS_TRY(check_batch(req, ctx_off, batch));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int M = req->n_units, N = ctx_off[M], nq = req->n_query, T = N + nq;
  Workspace ws = carve(D, N, nq, M, check_layer, workspace);
  AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
  if (*ctx_inout && reinterpret_cast<Ctx*>(*ctx_inout)->magic != kCtxMagic) return AKVS_ERR_INVALID_ARG;

  std::vector<int32_t> probe_off(M + 1, 0);
  for (int u = 0; u < M; ++u) {
    const int64_t n = ctx_off[u + 1] - ctx_off[u];
    int64_t b = (n * refresh_bp + 9999) / 10000;          // ceil(r n) in integers
    b = b < 0 ? 0 : (b > n ? n : b);
    probe_off[u + 1] = probe_off[u] + (int32_t)b;
  }
  AKVS_TRY(setup_request(D, ws, ctx_off, slot_src, M, N, nq, st));
  if (batch.B > 1) AKVS_TRY(setup_batch(ws, ctx_off, batch, M, N, nq, st));
  const RowGeom all_tokens = token_geom(ws, batch, T);
  AKVS_CUDA(cudaMemcpyAsync(ws.probe_off, probe_off.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_CUDA(cudaMemcpyAsync(out->ctx_off, ctx_off.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_CUDA(cudaMemcpyAsync(out->probe_off, probe_off.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_TRY(launch_rope_table(model->rope_base, D.hd, T, ws.rope, st));

  // dense front: layers before the check layer on every row; their K/V are fresh
  AKVS_TRY(embed_all(model, D, cache, req, ws, N, st));
  const size_t kv_l = (size_t)T * D.dkv * D.es;
  for (int l = 0; l < check_layer - 1; ++l) {
    void* kd = reinterpret_cast<char*>(ws.stash_k) + l * kv_l;
    void* vd = reinterpret_cast<char*>(ws.stash_v) + l * kv_l;
    AKVS_TRY(run_layer(model, D, l, ws, T, all_tokens, kd, vd, kd, vd, T, nullptr, st));
  }
  if (T > 0)
    AKVS_CUDA(cudaMemcpyAsync(ws.stash_h, ws.h, (size_t)T * D.d * sizeof(float), cudaMemcpyDeviceToDevice, st));

  // check layer: fresh K/V of every context row, scores against the re-aligned cache
  const int lc = check_layer - 1;
  if (N > 0) {
    AKVS_TRY(launch_rmsnorm(D.dtype, ws.h, model->attn_norm[lc], model->rms_eps, N, D.d, ws.x, st));
    const void* w[2] = {model->wk[lc], model->wv[lc]};
    const int ns[2] = {D.dkv, D.dkv};
    void* o[2] = {ws.k, ws.v};
    AKVS_TRY(linear_multi(D, ws.x, N, D.d, 2, w, ns, o, ns, ws.status, st, ws.rope, all_tokens.pos, 0b01,
                          model->rope_base, ws.rope_n));
    AKVS_TRY(wait_layer(cache, lc, st));
    AKVS_TRY(launch_scores(D.dtype, cache_layer(cache, D, lc), req_maps(ws, N, batch.B > 1), ws.k, ws.v, N, D.nkv, D.hd, ws.rope,
                           out->d_k, out->d_v, st));
  }
  AKVS_TRY(launch_select(out->d_k, out->d_v, ws.ctx_off, ws.probe_off, M, N, nq, out->sk_idx, out->sv_idx, out->w_k,
                         out->w_v, out->rows, ws.keys, ws.flags, ws.status + 4, ws.status, st));
  int32_t host[8] = {0};
  AKVS_CUDA(cudaMemcpyAsync(host, ws.status, sizeof(host), cudaMemcpyDeviceToHost, st));
  AKVS_CUDA(cudaStreamSynchronize(st));
  if (host[0] != 0) return host[0];
  out->n_ctx = N;
  out->n_probe_rows = host[4];
  out->n_rows = host[5];

  Ctx* ctx = reinterpret_cast<Ctx*>(*ctx_inout);
  if (!ctx) {
    ctx = new (std::nothrow) Ctx;
    if (!ctx) return AKVS_ERR_INVALID_ARG;
    *ctx_inout = ctx;
  }
  ctx->magic = kCtxMagic;
  ctx->N = N; ctx->nq = nq; ctx->M = M; ctx->B = batch.B; ctx->check_layer = check_layer;
  ctx->n_probe_total = probe_off[M];
  ctx->workspace = workspace;
  return AKVS_OK;
}

int32_t akvs_prefill_corrected(const akvs_model_desc* model, const akvs_cache* cache, const akvs_request* req,
                               const akvs_probes* probes, int32_t mode, float* out_hidden, void* out_k, void* out_v,
                               void* ctx_v, void* workspace, int64_t ws_bytes, void* stream) {
  Dims D;
  AKVS_TRY(check_model(model, D));
  if (mode != AKVS_MODE_CORRECTED && mode != AKVS_MODE_NAIVE && mode != AKVS_MODE_FULL) return AKVS_ERR_INVALID_ARG;
  AKVS_TRY(check_cache(cache, D, mode != AKVS_MODE_FULL));
  if (!out_hidden || !out_k || !out_v) return AKVS_ERR_INVALID_ARG;
  std::vector<int32_t> ctx_off, slot_src;
  AKVS_TRY(check_request(req, cache, ctx_off, slot_src));
  Batch batch;
  AKVS_TRY(check_batch(req, ctx_off, batch));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int M = req->n_units, N = ctx_off[M], nq = req->n_query, T = N + nq;
  const size_t kv_l = (size_t)T * D.dkv * D.es;
  char* ok = reinterpret_cast<char*>(out_k);
  char* ov = reinterpret_cast<char*>(out_v);

  if (mode == AKVS_MODE_FULL) {
    Workspace ws = carve(D, N, nq, M, 1, workspace);
    AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
    AKVS_TRY(setup_request(D, ws, ctx_off, slot_src, M, N, nq, st));
    if (batch.B > 1) AKVS_TRY(setup_batch(ws, ctx_off, batch, M, N, nq, st));
    AKVS_TRY(launch_rope_table(model->rope_base, D.hd, T, ws.rope, st));
    AKVS_TRY(embed_all(model, D, cache, req, ws, N, st));
    const RowGeom all_tokens = token_geom(ws, batch, T);
    for (int l = 0; l < D.L; ++l)
      AKVS_TRY(run_layer(model, D, l, ws, T, all_tokens, ok + l * kv_l, ov + l * kv_l, ok + l * kv_l, ov + l * kv_l, T,
                         nullptr, st));
    return launch_rmsnorm(AKVS_F32, ws.h + (size_t)N * D.d, model->final_norm, model->rms_eps, nq, D.d, out_hidden, st);
  }

  int first_layer = 0, P = 0, R = nq, n_probe_total = 0;
  const int32_t* rows = nullptr;
  Workspace ws;
  if (mode == AKVS_MODE_NAIVE) {
    ws = carve(D, N, nq, M, 1, workspace);
    AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
    AKVS_TRY(setup_request(D, ws, ctx_off, slot_src, M, N, nq, st));
    if (batch.B > 1) AKVS_TRY(setup_batch(ws, ctx_off, batch, M, N, nq, st));
    AKVS_TRY(launch_rope_table(model->rope_base, D.hd, T, ws.rope, st));
    rows = ws.pos + N;                                   // the query positions N..T-1
    AKVS_TRY(launch_row_maps(rows, nq, nullptr, nullptr, 0, N, T, ws.row_of_pos, ws.flags, ws.flags + N, st));
    AKVS_TRY(launch_tok_meta(ws.tok_unit, ws.tok_src, ws.row_of_pos, ws.flags, ws.flags + N, nullptr, nullptr, N, T, 0,
                             ws.tok_meta, st));
    AKVS_TRY(launch_embed(D.dtype, model->tok_emb, req->query_ids, nullptr, nq, D.d, D.vocab, ws.status, ws.h, st));
  } else {
    const Ctx* ctx = reinterpret_cast<const Ctx*>(ctx_v);
    if (!ctx || ctx->magic != kCtxMagic || !probes) return AKVS_ERR_INVALID_ARG;
    if (ctx->N != N || ctx->nq != nq || ctx->M != M || ctx->B != batch.B || ctx->workspace != workspace)
      return AKVS_ERR_SHAPE;
    if (probes->n_ctx != N || probes->n_probe_rows < 0 || probes->n_probe_rows > N ||
        probes->n_rows != probes->n_probe_rows + nq)
      return AKVS_ERR_SHAPE;
    if (!probes->sk_idx || !probes->sv_idx || !probes->w_k || !probes->w_v || !probes->rows || !probes->probe_off)
      return AKVS_ERR_INVALID_ARG;
    ws = carve(D, N, nq, M, ctx->check_layer, workspace);
    AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
    first_layer = ctx->check_layer - 1;
    n_probe_total = ctx->n_probe_total;
    P = probes->n_probe_rows;
    R = probes->n_rows;
    rows = probes->rows;
    AKVS_TRY(launch_row_maps(rows, R, probes->sk_idx, probes->sv_idx, ctx->n_probe_total, N, T, ws.row_of_pos,
                             ws.flags, ws.flags + N, st));
    AKVS_TRY(launch_tok_meta(ws.tok_unit, ws.tok_src, ws.row_of_pos, ws.flags, ws.flags + N, probes->w_k, probes->w_v, N,
                             T, P, ws.tok_meta, st));
    for (int l = 0; l < first_layer; ++l) {
      AKVS_CUDA(cudaMemcpyAsync(ok + l * kv_l, reinterpret_cast<char*>(ws.stash_k) + l * kv_l, kv_l,
                                cudaMemcpyDeviceToDevice, st));
      AKVS_CUDA(cudaMemcpyAsync(ov + l * kv_l, reinterpret_cast<char*>(ws.stash_v) + l * kv_l, kv_l,
                                cudaMemcpyDeviceToDevice, st));
    }
    AKVS_TRY(launch_gather_rows(ws.stash_h, rows, R, D.d, T, ws.status, ws.h, st));
  }

  const ReqMaps maps = req_maps(ws, N, batch.B > 1);
  RowGeom geom;
  AKVS_TRY(row_geom(ws, batch, rows, R, T, geom, st));
  const bool corrected = mode == AKVS_MODE_CORRECTED;
  for (int l = first_layer; l < D.L; ++l) {
    const KvLayer kv = cache_layer(cache, D, l);
    auto assemble = [&, l]() -> int32_t {
      AKVS_TRY(wait_layer(cache, l, st));
      if (corrected)
        AKVS_TRY(launch_offsets(D.dtype, kv, maps, probes->probe_off, probes->sk_idx, probes->sv_idx, ws.k, ws.v, M,
                                N, n_probe_total, D.nkv, D.hd, ws.rope, ws.mu_k, ws.mu_v, ws.status, st));
      return launch_correct(D.dtype, kv, maps, ws.k, ws.v, corrected, ws.mu_k, ws.mu_v, N, nq, D.nkv, D.hd, ws.rope,
                            ok + l * kv_l, ov + l * kv_l, st);
    };
    AKVS_TRY(run_layer(model, D, l, ws, R, geom, ws.k, ws.v, ok + l * kv_l, ov + l * kv_l, T, assemble, st,
                       /*split_ok=*/true));
  }
  return launch_rmsnorm(AKVS_F32, ws.h + (size_t)P * D.d, model->final_norm, model->rms_eps, nq, D.d, out_hidden, st);
}

int32_t akvs_debug_correct_repeat(const akvs_model_desc* model, const akvs_cache* cache, const akvs_request* req,
                                  const akvs_probes* probes, void* out_k, void* out_v, void* ctx_v, void* workspace,
                                  int64_t ws_bytes, void* stream) {
  Dims D;
  AKVS_TRY(check_model(model, D));
  AKVS_TRY(check_cache(cache, D, true));
  if (!out_k || !out_v || !probes) return AKVS_ERR_INVALID_ARG;
  std::vector<int32_t> ctx_off, slot_src;
  AKVS_TRY(check_request(req, cache, ctx_off, slot_src));
  Batch batch;
  AKVS_TRY(check_batch(req, ctx_off, batch));
  const Ctx* ctx = reinterpret_cast<const Ctx*>(ctx_v);
  const int M = req->n_units, N = ctx_off[M], nq = req->n_query, T = N + nq;
  if (!ctx || ctx->magic != kCtxMagic) return AKVS_ERR_INVALID_ARG;
  if (ctx->N != N || ctx->nq != nq || ctx->M != M || ctx->B != batch.B || ctx->workspace != workspace)
    return AKVS_ERR_SHAPE;
  Workspace ws = carve(D, N, nq, M, ctx->check_layer, workspace);
  AKVS_TRY(check_workspace(workspace, ws_bytes, ws.bytes));
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const size_t kv_l = (size_t)T * D.dkv * D.es;
  const ReqMaps maps = req_maps(ws, N, batch.B > 1);
  for (int l = ctx->check_layer - 1; l < D.L; ++l)
    AKVS_TRY(launch_correct(D.dtype, cache_layer(cache, D, l), maps, ws.k, ws.v, true, ws.mu_k, ws.mu_v, N, nq, D.nkv,
                            D.hd, ws.rope, reinterpret_cast<char*>(out_k) + l * kv_l,
                            reinterpret_cast<char*>(out_v) + l * kv_l, st));
  return AKVS_OK;
}

void akvs_free(void* ctx) {
  Ctx* c = reinterpret_cast<Ctx*>(ctx);
  if (c && c->magic == kCtxMagic) {
    c->magic = 0;
    delete c;
  }
}

int32_t akvs_check(void* workspace, void* stream) {
  if (!workspace) return AKVS_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int32_t s = 0;
  AKVS_CUDA(cudaMemcpyAsync(&s, workspace, sizeof(s), cudaMemcpyDeviceToHost, st));
  AKVS_CUDA(cudaStreamSynchronize(st));
  AKVS_CUDA(cudaMemsetAsync(workspace, 0, sizeof(int32_t), st));
  if (cudaGetLastError() != cudaSuccess) return AKVS_ERR_CUDA;
  return s;
}

// ----------------------------------------------------------------------------- single steps

int32_t akvs_op_linear(int32_t dtype, const void* x, const void* w, void* y, int32_t M, int32_t N, int32_t K,
                       int32_t algo, void* stream) {
  if (!x || !w || !y || M < 0 || N <= 0 || K <= 0) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (algo < 0 || algo > 3) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && algo != 1) {
    if (N % 128 != 0 || K % 8 != 0) return AKVS_ERR_SHAPE;
    return launch_linear_tc(dtype, 0, x, M, K, 1, &w, &N, &y, &N, nullptr, st, nullptr, nullptr, 0,
                            algo == 0 ? 0 : algo - 1);
  }
  return launch_linear_simt(dtype, x, w, nullptr, y, nullptr, M, N, K, N, st);
}

int32_t akvs_op_linear_residual(int32_t dtype, const void* x, const void* w, float* h, int32_t M, int32_t N, int32_t K,
                                int32_t algo, int32_t splits, void* stream) {
  if (!x || !w || !h || M < 0 || N <= 0 || K <= 0 || splits < 0 || splits > 4) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (algo < 0 || algo > 3) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && algo != 1) {
    if (N % 128 != 0 || K % 8 != 0) return AKVS_ERR_SHAPE;
    void* out = h;
    return launch_linear_tc(dtype, 1, x, M, K, 1, &w, &N, &out, &N, nullptr, st, nullptr, nullptr, 0,
                            algo == 0 ? 0 : algo - 1, 0, splits);
  }
  if (splits > 1) return AKVS_ERR_UNSUPPORTED;
  return launch_linear_simt(dtype, x, w, nullptr, nullptr, h, M, N, K, N, st);
}

int32_t akvs_op_rope(int32_t dtype, void* x, const int32_t* pos, int32_t n, int32_t n_heads, int32_t head_dim,
                     float rope_base, void* stream) {
  if (!x || !pos || n < 0 || n_heads <= 0 || head_dim <= 0) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  return launch_rope(dtype, x, pos, n, n_heads, head_dim, n_heads * head_dim, nullptr, 0, nullptr, rope_base,
                     reinterpret_cast<cudaStream_t>(stream));
}

int32_t akvs_op_attention(int32_t dtype, const void* q, const void* k, const void* v, void* out, const int32_t* k_lo,
                          const int32_t* k_hi, int32_t R, int32_t T, int32_t n_q_heads, int32_t n_kv_heads,
                          int32_t head_dim, int32_t algo, void* stream) {
  if (!q || !k || !v || !out || !k_lo || !k_hi || R < 0 || T < 0) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (dtype != AKVS_F32 && head_dim == 128 && algo == 0)
    return launch_attention_tc(dtype, q, k, v, out, k_lo, k_hi, nullptr, nullptr, R, T, n_q_heads, n_kv_heads, nullptr, st);
  return launch_attention_simt(dtype, q, k, v, out, k_lo, k_hi, nullptr, nullptr, R, n_q_heads, n_kv_heads, head_dim, st);
}

int64_t akvs_op_scratch_bytes(int32_t n_ctx, int32_t n_query, int32_t n_units, int32_t head_dim) {
  const int64_t T = (int64_t)n_ctx + n_query;
  return 4096 + 256 * 12 + T * (4 + 32 + head_dim * 4) + (int64_t)n_ctx * (4 + 2 + 16) + (int64_t)(n_units + 1) * 8;
}

int32_t akvs_op_select(const float* d_k, const float* d_v, const int32_t* ctx_off_host, int32_t n_units,
                       int32_t n_query, int32_t refresh_bp, akvs_probes* out, void* scratch, void* stream) {
  if (!d_k || !d_v || !ctx_off_host || !out || !scratch || n_units < 0 || n_query < 0 || refresh_bp < 0 ||
      refresh_bp > 10000)
    return AKVS_ERR_INVALID_ARG;
  if (!out->ctx_off || !out->probe_off || !out->sk_idx || !out->sv_idx || !out->w_k || !out->w_v || !out->rows)
    return AKVS_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int M = n_units;
  if (ctx_off_host[0] != 0) return AKVS_ERR_SHAPE;
  for (int u = 0; u < M; ++u)
    if (ctx_off_host[u + 1] < ctx_off_host[u]) return AKVS_ERR_SHAPE;      // before N is used for anything
  const int N = ctx_off_host[M];
  std::vector<int32_t> probe_off(M + 1, 0);
  for (int u = 0; u < M; ++u) {
    const int64_t n = ctx_off_host[u + 1] - ctx_off_host[u];
    int64_t b = (n * refresh_bp + 9999) / 10000;
    b = b > n ? n : b;
    probe_off[u + 1] = probe_off[u] + (int32_t)b;
  }
  Carver c(scratch);
  int32_t* status = c.take<int32_t>(16);
  uint64_t* keys = c.take<uint64_t>(2 * (int64_t)N);
  uint8_t* flags = c.take<uint8_t>(2 * (int64_t)N);
  AKVS_CUDA(cudaMemsetAsync(status, 0, 16 * sizeof(int32_t), st));
  AKVS_CUDA(cudaMemcpyAsync(out->ctx_off, ctx_off_host, (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_CUDA(cudaMemcpyAsync(out->probe_off, probe_off.data(), (M + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_TRY(launch_select(d_k, d_v, out->ctx_off, out->probe_off, M, N, n_query, out->sk_idx, out->sv_idx, out->w_k,
                         out->w_v, out->rows, keys, flags, status + 4, status, st));
  int32_t host[8] = {0};
  AKVS_CUDA(cudaMemcpyAsync(host, status, sizeof(host), cudaMemcpyDeviceToHost, st));
  AKVS_CUDA(cudaStreamSynchronize(st));
  if (host[0] != 0) return host[0];
  out->n_ctx = N;
  out->n_probe_rows = host[4];
  out->n_rows = host[5];
  return AKVS_OK;
}

int32_t akvs_op_correct_layer(int32_t dtype, int32_t kv_format, const void* cache_k, const void* cache_v,
                              const void* k_meta, const void* v_meta, const int32_t* src_tok, const void* fresh_k,
                              const void* fresh_v, const akvs_probes* probes, int32_t n_units, int32_t n_query,
                              int32_t n_kv_heads, int32_t head_dim, float rope_base, void* out_k, void* out_v,
                              float* mu_k, float* mu_v, void* scratch, void* stream) {
  if (!probes || !out_k || !out_v || !mu_k || !mu_v || !scratch || n_units < 0 || n_query < 0)
    return AKVS_ERR_INVALID_ARG;
  if (probes->n_ctx > 0 && (!cache_k || !cache_v || !src_tok)) return AKVS_ERR_INVALID_ARG;
  if (probes->n_rows > 0 && (!fresh_k || !fresh_v)) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int N = probes->n_ctx, T = N + n_query, M = n_units;
  if (probes->n_rows != probes->n_probe_rows + n_query) return AKVS_ERR_SHAPE;
  Carver c(scratch);
  int32_t* poff_host_dev = c.take<int32_t>(16);
  int32_t* tok_unit = c.take<int32_t>(N);
  int32_t* row_of_pos = c.take<int32_t>(T);
  uint8_t* flags = c.take<uint8_t>(2 * (int64_t)N);
  int32_t* zero_src = c.take<int32_t>(M + 1);
  int32_t* dummy_src = c.take<int32_t>(N);
  float2* table = c.take<float2>((int64_t)T * (head_dim / 2));
  int4* tok_meta = c.take<int4>(2 * (int64_t)T);
  // the number of probe indices is probe_off[M]; read it back (this helper may synchronise)
  int32_t n_probe = 0;
  AKVS_CUDA(cudaMemcpyAsync(&n_probe, probes->probe_off + M, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  AKVS_CUDA(cudaStreamSynchronize(st));
  if (n_probe < 0 || n_probe > N) return AKVS_ERR_SHAPE;
  AKVS_CUDA(cudaMemsetAsync(zero_src, 0, (M + 1) * sizeof(int32_t), st));
  AKVS_TRY(launch_tok_maps(probes->ctx_off, zero_src, M, N, tok_unit, dummy_src, st));
  AKVS_TRY(launch_row_maps(probes->rows, probes->n_rows, probes->sk_idx, probes->sv_idx, n_probe, N, T, row_of_pos,
                           flags, flags + N, st));
  AKVS_TRY(launch_rope_table(rope_base, head_dim, T, table, st));
  AKVS_TRY(launch_tok_meta(tok_unit, src_tok, row_of_pos, flags, flags + N, probes->w_k, probes->w_v, N, T,
                           probes->n_probe_rows, tok_meta, st));
  KvLayer kv{cache_k, cache_v, k_meta, v_meta, kv_format};
  ReqMaps maps{probes->ctx_off, probes->ctx_off, tok_unit, src_tok, row_of_pos, flags, flags + N, tok_meta};
  int32_t* status = poff_host_dev;                 // first words of the scratch: the status word of this call
  AKVS_CUDA(cudaMemsetAsync(status, 0, 16 * sizeof(int32_t), st));
  AKVS_TRY(launch_offsets(dtype, kv, maps, probes->probe_off, probes->sk_idx, probes->sv_idx, fresh_k, fresh_v, M, N,
                          n_probe, n_kv_heads, head_dim, table, mu_k, mu_v, status, st));
  return launch_correct(dtype, kv, maps, fresh_k, fresh_v, true, mu_k, mu_v, N, n_query, n_kv_heads, head_dim, table,
                        out_k, out_v, st);
}

int32_t akvs_op_residual_stats(int32_t dtype, int32_t kv_format, const void* cache_k, const void* cache_v,
                               const void* k_meta, const void* v_meta, const int32_t* src_tok, const void* fresh_k,
                               const void* fresh_v, const int32_t* ctx_off_host, int32_t n_units, int32_t n_kv_heads,
                               int32_t head_dim, float rope_base, const float* sel_k, const float* sel_v,
                               const float* mu_k, const float* mu_v, const float* w_k, const float* w_v, float* mean_k,
                               float* mean_v, float* energy, void* scratch, void* stream) {
  if (!ctx_off_host || !energy || !scratch || n_units < 0) return AKVS_ERR_INVALID_ARG;
  if ((mu_k == nullptr) != (mu_v == nullptr) || (mean_k == nullptr) != (mean_v == nullptr)) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  if (ctx_off_host[0] != 0) return AKVS_ERR_SHAPE;
  for (int u = 0; u < n_units; ++u)
    if (ctx_off_host[u + 1] < ctx_off_host[u]) return AKVS_ERR_SHAPE;
  const int N = ctx_off_host[n_units];
  if (N > 0 && (!cache_k || !cache_v || !src_tok || !fresh_k || !fresh_v)) return AKVS_ERR_INVALID_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  Carver c(scratch);
  int32_t* ctx_off = c.take<int32_t>(n_units + 1);
  float2* table = c.take<float2>((int64_t)N * (head_dim / 2));
  AKVS_CUDA(cudaMemcpyAsync(ctx_off, ctx_off_host, (n_units + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  AKVS_TRY(launch_rope_table(rope_base, head_dim, N, table, st));
  KvLayer kv{cache_k, cache_v, k_meta, v_meta, kv_format};
  return launch_residual_stats(dtype, kv, ctx_off, src_tok, fresh_k, fresh_v, n_units, n_kv_heads, head_dim, table,
                               sel_k, sel_v, mu_k, mu_v, w_k, w_v, mean_k, mean_v, energy, st);
}

int32_t akvs_op_quantize(int32_t dtype, const void* x, int32_t n, int32_t n_kv_heads, int32_t head_dim, int32_t bits,
                         void* codes, void* meta, void* stream) {
  if (!x || !codes || (!meta && bits != AKVS_KV_FP8) || n < 0) return AKVS_ERR_INVALID_ARG;
  if (dtype != AKVS_F32 && dtype != AKVS_BF16 && dtype != AKVS_F16) return AKVS_ERR_UNSUPPORTED;
  return launch_quantize(dtype, x, n, n_kv_heads, head_dim, bits, codes, meta, reinterpret_cast<cudaStream_t>(stream));
}

}  // extern "C"
