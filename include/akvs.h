/*
 * akvs -- selective-recompute prefill with probe-guided per-unit KV offset correction,
 * for one NVIDIA B200 (sm_100a).  Plain C ABI: POD structs, raw pointers, sizes.
 *
 * The method (paper Section 3, Algorithm 1): every memory unit is encoded once, alone, and
 * its per-layer K/V cached.  For a request the retrieved units are concatenated in
 * retrieval order and followed by the query.  At a check layer, per-token divergence
 * scores between fresh and reused K/V pick, per unit, the top-b tokens by K score and the
 * top-b by V score (b = ceil(r n)) and fix per-token weights w = min(score, 1).  From the
 * check layer on only those probe tokens (and the query) are recomputed; per layer and
 * unit the mean residual (fresh - reused) over the probes is the unit's offset, and every
 * non-probe token of the unit gets reused + w * offset while probes keep their fresh state.
 *
 * Conventions
 *  - every function returns AKVS_OK or a negative AKVS_ERR_*; nothing is launched when
 *    validation fails; no exception or abort crosses this boundary;
 *  - "device" pointers are CUDA global memory owned by the caller, "host" pointers are
 *    ordinary host memory owned by the caller; the library allocates no device memory
 *    (scratch comes from the caller's workspace);
 *  - all work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL is
 *    the default stream).  These calls synchronise it (each says so below): akvs_select_probes
 *    and akvs_check; akvs_op_select, akvs_op_select_static and akvs_op_correct_layer; and
 *    akvs_select_probes / akvs_prefill_corrected (NAIVE and FULL modes) with n_requests > 1,
 *    which upload per-token tables of a batch from host vectors;
 *  - a process drives ONE device through this library (one process per GPU): kernel
 *    attributes are set once per process on the device current at the first call, the
 *    measurement hooks keep process-wide state, and calls are not re-entrant across host
 *    threads that share a workspace;
 *  - linear weights are row-major [out_features][in_features] (y = x W^T), no biases;
 *  - model dtype AKVS_F32 / AKVS_BF16 / AKVS_F16: weights, the native unit cache, every
 *    activation tensor and the K/V outputs have that type; accumulation, the residual
 *    stream and `out_hidden` are float in every mode.  The 16-bit modes run the linear
 *    layers on the tensor cores at the same rate; float16 keeps three more mantissa bits
 *    (conversions saturate instead of producing infinities);
 *  - K is cached AFTER RoPE at unit-local positions 0..n-1 (rotate-half pairing
 *    (i, i + head_dim/2), angle p * rope_base^(-2i/head_dim)); reuse turns it through the
 *    unit's global offset.  Residuals, offsets and corrected K live at global positions.
 */
#ifndef AKVS_H
#define AKVS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AKVS_OK               0
#define AKVS_ERR_INVALID_ARG (-1)  /* null pointer, negative size, value out of range      */
#define AKVS_ERR_SHAPE       (-2)  /* model/cache/request shapes inconsistent or unsupported */
#define AKVS_ERR_WORKSPACE   (-3)  /* workspace missing, misaligned (256 B) or too small     */
#define AKVS_ERR_UNSUPPORTED (-4)  /* dtype / kv format / head_dim not handled               */
#define AKVS_ERR_CUDA        (-5)  /* a CUDA runtime or driver call failed                    */
#define AKVS_ERR_TIMEOUT     (-6)  /* a bounded device-side wait ran out (no hang, no trap)  */
#define AKVS_ERR_NAN_SCORE   (-7)  /* a divergence score was NaN                             */
#define AKVS_ERR_TOO_LARGE   (-8)  /* request exceeds a fixed capacity of the entry point    */

#define AKVS_F32   0
#define AKVS_BF16  1
#define AKVS_F16   2

#define AKVS_KV_NATIVE 0           /* cache holds the model dtype                            */
#define AKVS_KV_Q2     2           /* 2-bit codes, asymmetric min-max, groups of 64 along head_dim */
#define AKVS_KV_Q4     4           /* 4-bit codes, same scheme                               */
#define AKVS_KV_FP8    8           /* FP8 E4M3 bytes (Section 4.5 names the format; no scale: a saturating
                                      round-to-nearest-even cast of each value), no k_meta / v_meta */

#define AKVS_MODE_CORRECTED 0      /* Algorithm 1                                            */
#define AKVS_MODE_NAIVE     1      /* direct reuse (Section 3.1): only the query is computed */
#define AKVS_MODE_FULL      2      /* full recompute of context + query (what is approximated) */

/* Decoder description.  All pointers borrowed.  The nine per-layer arrays are HOST arrays
 * of n_layers DEVICE pointers.  Pre-norm RMSNorm (gain vectors are float), GQA with
 * q head i reading kv head i / (n_q_heads / n_kv_heads), SwiGLU MLP. */
typedef struct akvs_model_desc {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab;
  int32_t dtype;                      /* AKVS_F32 | AKVS_BF16 | AKVS_F16                    */
  float   rope_base, rms_eps;
  const void*  tok_emb;               /* device [vocab][d_model], model dtype                */
  const float* final_norm;            /* device [d_model]                                    */
  const float* const* attn_norm;      /* [L] -> device [d_model]                             */
  const void* const* wq;              /* [L] -> device [n_q_heads*head_dim][d_model]         */
  const void* const* wk;              /* [L] -> device [n_kv_heads*head_dim][d_model]        */
  const void* const* wv;              /* [L] -> device [n_kv_heads*head_dim][d_model]        */
  const void* const* wo;              /* [L] -> device [d_model][n_q_heads*head_dim]         */
  const float* const* mlp_norm;       /* [L] -> device [d_model]                             */
  const void* const* w_gate;          /* [L] -> device [d_ff][d_model]                       */
  const void* const* w_up;            /* [L] -> device [d_ff][d_model]                       */
  const void* const* w_down;          /* [L] -> device [d_model][d_ff]                       */
} akvs_model_desc;

/* Unit store (Section 3.1: "encoded once").  Filled by akvs_encode_units, read-only to
 * every other call (the same unit is reused under other contexts). */
typedef struct akvs_cache {
  int32_t n_units, n_tokens, kv_format;
  const int32_t* unit_off;   /* host   [n_units+1], prefix sums of unit lengths, unit_off[0]=0 */
  const int32_t* token_ids;  /* device [n_tokens], units back to back in store order          */
  void* k;                   /* device [L][n_tokens][n_kv][head_dim] model dtype, or packed codes
                                [L][n_tokens][n_kv][head_dim*bits/8] bytes (little-endian in a byte) */
  void* v;                   /* same layout                                                    */
  void* k_meta;              /* device half2 (scale, min) [L][n_tokens][n_kv][head_dim/64]; NULL if native */
  void* v_meta;
  void* const* layer_ready;  /* host [L] of cudaEvent_t, or NULL.  When set, the library makes its stream wait
                                for layer_ready[l] before the first read of layer l of k/v/meta, so a caller
                                that streams an offloaded cache in over PCIe (one copy + event record per layer,
                                on its own stream, enqueued before the call) overlaps the transfer with the
                                prefill.  Ignored by akvs_encode_units. */
} akvs_cache;

/* One request: which units, in which order (retrieval order differs per query), and the query.
 *
 * A batch of requests that share the model (Section 4.4 measures batch sizes 4-16) is one
 * akvs_request with n_requests > 1: unit_ids and query_ids hold the requests' lists one after
 * the other and req_unit_off / req_query_off give the boundaries.  Every linear layer then
 * runs once over the recomputed rows of all requests; attention, offsets and corrections stay
 * per request (a row only sees its own request's context and query tokens, positions restart
 * at 0 in every request, offsets are per unit as before).  Token order of every per-token
 * argument and output (akvs_probes arrays, out_k / out_v rows, out_hidden rows): all context
 * tokens, request after request, then all query tokens, request after request.  The results of
 * a request do not depend on the other requests of its batch. */
typedef struct akvs_request {
  int32_t n_units;           /* total over the batch                                          */
  const int32_t* unit_ids;   /* host   [n_units], indices into the unit store                 */
  int32_t n_query;           /* total over the batch                                          */
  const int32_t* query_ids;  /* device [n_query]                                              */
  int32_t n_requests;        /* 0 or 1: a single request (the two arrays below are ignored)   */
  const int32_t* req_unit_off;   /* host [n_requests + 1] boundaries in unit_ids, first 0, last n_units  */
  const int32_t* req_query_off;  /* host [n_requests + 1] boundaries in query_ids, first 0, last n_query */
} akvs_request;

/* Probe sets and weights (Section 3.3).  Every array is device memory allocated by the
 * caller for n_ctx = total context tokens of the request; akvs_select_probes fills them and
 * the three host counters.  A caller may overwrite the contents (for instance with sets
 * chosen elsewhere) before akvs_prefill_corrected as long as the counters stay consistent. */
typedef struct akvs_probes {
  int32_t  n_ctx;            /* out: N                                                        */
  int32_t  n_probe_rows;     /* out: P = | union of all S^K and S^V |                         */
  int32_t  n_rows;           /* out: P + n_query                                              */
  int32_t* ctx_off;          /* [n_units+1] global offset of each unit in this request        */
  int32_t* probe_off;        /* [n_units+1] prefix sums of b_u (same for K and V sets)        */
  int32_t* sk_idx;           /* [n_ctx] first probe_off[n_units] valid: S^K, global positions, ascending per unit */
  int32_t* sv_idx;           /* [n_ctx] S^V likewise                                          */
  float*   w_k;              /* [n_ctx] min(d_K, 1)                                           */
  float*   w_v;              /* [n_ctx] min(d_V, 1)                                           */
  float*   d_k;              /* [n_ctx] divergence scores at the check layer                  */
  float*   d_v;              /* [n_ctx]                                                       */
  int32_t* rows;             /* [n_ctx + n_query] recomputed rows: sorted probe positions, then the query positions */
} akvs_probes;

/* Bytes of workspace a request of this size needs (monotone in every argument).
 * Workspace must be 256-byte aligned device memory; its contents carry state from
 * akvs_select_probes to akvs_prefill_corrected of the same request. */
int32_t akvs_workspace_bytes(const akvs_model_desc* model, int32_t n_ctx, int32_t n_query,
                             int32_t n_units, int32_t check_layer, int64_t* out_bytes);

/* Section 3.1 -- isolated encoding.  Runs every unit of cache->token_ids alone (positions
 * 0..n_u-1, causal within the unit) through all layers and stores, per layer, K after RoPE
 * at local positions and V, in cache->kv_format.  cache->unit_off/token_ids are inputs;
 * cache->k/v (and *_meta when quantised) are outputs.  Asynchronous. */
int32_t akvs_encode_units(const akvs_model_desc* model, akvs_cache* cache,
                          void* workspace, int64_t ws_bytes, void* stream);

/* Section 3.3, Algorithm 1 line 2 -- probe selection.  Computes layers 1..check_layer-1
 * densely for all rows (context + query), then at the check layer the fresh K/V of every
 * context token, the scores d_K, d_V against the re-aligned cache, per unit the top-b sets
 * (b = ceil(n_u * refresh_bp / 10000), ties to the smaller index, indices ascending), the
 * weights and the sorted row list.  check_layer is 1-based, 1 <= check_layer <= n_layers.
 * Synchronises the stream once to return the row counts.  *ctx_inout: pass NULL-initialised
 * storage the first time; the library creates (or reuses) a small host object that carries
 * the request's state to akvs_prefill_corrected; release it with akvs_free. */
int32_t akvs_select_probes(const akvs_model_desc* model, const akvs_cache* cache,
                           const akvs_request* req, int32_t refresh_bp, int32_t check_layer,
                           akvs_probes* out, void** ctx_inout,
                           void* workspace, int64_t ws_bytes, void* stream);

/* Algorithm 1 lines 3-9 around the decoder -- the prefill.
 *  AKVS_MODE_CORRECTED: needs `probes` and the `ctx` of a preceding akvs_select_probes on
 *    the same workspace.  From the check layer on, recomputes the rows in probes->rows,
 *    estimates per-unit offsets from the probes, writes corrected K/V for the whole context.
 *  AKVS_MODE_NAIVE: probes/ctx may be NULL; context K/V are the re-aligned cache.
 *  AKVS_MODE_FULL:  probes/ctx may be NULL; everything recomputed (cache K/V unused).
 * Outputs: out_hidden float [n_query][d_model] (after the final RMSNorm);
 *          out_k, out_v [L][n_ctx+n_query][n_kv][head_dim] in the model dtype, K after
 *          RoPE at global positions.  Asynchronous.
 * In AKVS_MODE_CORRECTED the call only enqueues work on `stream` (kernels and device-to-device
 * copies; no host reads, no host buffers of its own), so after one eager call with the same
 * model (which sets the kernels' function attributes) it may be recorded into a CUDA graph by
 * stream capture and replayed, as long as every pointer argument, the probe counts and the
 * cache's layer_ready events stay what they were at capture.  The other two modes upload small
 * host tables and are not meant for capture. */
int32_t akvs_prefill_corrected(const akvs_model_desc* model, const akvs_cache* cache,
                               const akvs_request* req, const akvs_probes* probes, int32_t mode,
                               float* out_hidden, void* out_k, void* out_v,
                               void* ctx, void* workspace, int64_t ws_bytes, void* stream);

/* Releases the host object created by akvs_select_probes.  NULL is allowed. */
void akvs_free(void* ctx);

/* Synchronises `stream` and returns the device status word kept in `workspace`
 * (AKVS_OK, AKVS_ERR_TIMEOUT, AKVS_ERR_NAN_SCORE), then clears it. */
int32_t akvs_check(void* workspace, void* stream);

/* ------------------------------------------------------------------------------------
 * Single steps of the path, exported so that each kernel can be checked on its own.
 * dtype names the element type of every `void*` tensor.  Asynchronous on `stream` unless stated.
 * ------------------------------------------------------------------------------------ */

/* y[M][N] = x[M][K] * w[N][K]^T, float accumulation.  algo 0: the path's default for the
 * dtype (tcgen05 tensor cores for the 16-bit types, CUDA cores for float); algo 1: CUDA cores;
 * algo 2 / 3 (16-bit types): the tensor-core kernel forced onto single CTAs / onto CTA pairs
 * (pairs need M > 128; otherwise single CTAs run) - the default picks between them by shape. */
int32_t akvs_op_linear(int32_t dtype, const void* x, const void* w, void* y,
                       int32_t M, int32_t N, int32_t K, int32_t algo, void* stream);

/* h[M][N] (float, read and written) += x[M][K] * w[N][K]^T: the residual form of the linear
 * layers after attention and after the MLP (the decoder layer of the models the paper serves;
 * the paper itself only says the probes are "recomputed", Algorithm 1).  algo as above.
 * splits (tensor-core kernel only): the k range is cut into that many work items per output
 * tile, each adding its partial sum into h with a vector reduction at the L2 - 0 lets the
 * library choose (it splits launches that would leave SMs idle), 1..4 force the count
 * (AKVS_ERR_SHAPE when K holds fewer 64-wide slabs than that).  With more than one split the
 * order in which partial sums reach an element is not fixed, so results may differ in the last
 * bit from run to run.  Errors: AKVS_ERR_INVALID_ARG (null pointer, bad size, splits outside
 * 0..4), AKVS_ERR_SHAPE (16-bit: N not a multiple of 128, K not of 8), AKVS_ERR_UNSUPPORTED
 * (dtype; splits > 1 on the CUDA-core kernel). */
int32_t akvs_op_linear_residual(int32_t dtype, const void* x, const void* w, float* h,
                                int32_t M, int32_t N, int32_t K, int32_t algo, int32_t splits,
                                void* stream);

/* Rotate-half RoPE in place on x[n][n_heads][head_dim] at positions pos[n] (device). */
int32_t akvs_op_rope(int32_t dtype, void* x, const int32_t* pos, int32_t n, int32_t n_heads,
                     int32_t head_dim, float rope_base, void* stream);

/* GQA attention: query row r sees key j iff k_lo[r] <= j <= k_hi[r] (device arrays, both
 * non-decreasing in r).  q [R][n_q][hd], k/v [T][n_kv][hd], out [R][n_q][hd].
 * algo 0: the path's default (tcgen05 for 16-bit types with head_dim 128, else CUDA cores);
 * algo 1: CUDA cores. */
int32_t akvs_op_attention(int32_t dtype, const void* q, const void* k, const void* v, void* out,
                          const int32_t* k_lo, const int32_t* k_hi, int32_t R, int32_t T,
                          int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int32_t algo, void* stream);

/* Bytes of scratch that akvs_op_select and akvs_op_correct_layer need for these sizes. */
int64_t akvs_op_scratch_bytes(int32_t n_ctx, int32_t n_query, int32_t n_units, int32_t head_dim);

/* Section 3.3 selection from given scores: fills probe_off, sk_idx, sv_idx, w_k, w_v, rows
 * (device) exactly as akvs_select_probes does; ctx_off is a HOST array [n_units+1].
 * scratch: device, 256-byte aligned, akvs_op_scratch_bytes(...) bytes.  Synchronises the stream. */
int32_t akvs_op_select(const float* d_k, const float* d_v, const int32_t* ctx_off_host, int32_t n_units,
                       int32_t n_query, int32_t refresh_bp, akvs_probes* out, void* scratch, void* stream);

/* akvs_op_select for callers that cannot allocate device memory.  (The paper has no
 * counterpart to this entry point; it exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is not an option -- a serving loop whose
 * device memory pool is carved up at start-up, a process whose remaining memory belongs to
 * another allocator, a request path on which allocation is forbidden -- and that therefore
 * has no scratch buffer to hand to akvs_op_select.  Here the scratch (sort keys, selection
 * flags, counters; about 0.3 MB) is a fixed array inside the library's device image, held
 * on every GPU that loads the library until the process exits.  The call itself allocates
 * nothing on the device or on the host heap.
 *
 * Same arguments, outputs and bit-exact results as akvs_op_select, minus `scratch`.
 * Limits: ctx_off_host[n_units] <= AKVS_STATIC_MAX_CTX context tokens and
 * n_units <= AKVS_STATIC_MAX_UNITS; beyond either the call returns AKVS_ERR_TOO_LARGE and
 * launches nothing.
 * First call per device: it resolves the device address of the array (with that device
 * current); make that first call outside any stream capture.
 * Sharing: every call on a device uses the one array, which keeps the previous call's
 * contents; the call clears what has to start at zero itself.  Two calls that overlap on the
 * GPU (different streams, different host threads) race on it: run them one after another.
 * Synchronises `stream` once, like akvs_op_select. */
#define AKVS_STATIC_MAX_CTX   16384
#define AKVS_STATIC_MAX_UNITS 1024
int32_t akvs_op_select_static(const float* d_k, const float* d_v, const int32_t* ctx_off_host, int32_t n_units,
                              int32_t n_query, int32_t refresh_bp, akvs_probes* out, void* stream);

/* One layer of Algorithm 1 lines 5-8 (mean estimation + correction) over a whole context.
 * fresh_k/fresh_v [n_rows][n_kv][hd] hold the recomputed rows listed in probes->rows (K
 * already rotated at global positions).  cache_k/cache_v (+meta) are ONE layer of a unit
 * store; the request's token j reads store row src_tok[j] (device [n_ctx]).  Writes
 * out_k/out_v [n_ctx+n_query][n_kv][hd] and the offsets mu_k, mu_v float [n_units][n_kv*hd].
 * scratch: device, 256-byte aligned, akvs_op_scratch_bytes(...) bytes.  Synchronises the stream
 * once (it reads the probe count back) before the kernels are enqueued. */
int32_t akvs_op_correct_layer(int32_t dtype, int32_t kv_format,
                              const void* cache_k, const void* cache_v, const void* k_meta, const void* v_meta,
                              const int32_t* src_tok, const void* fresh_k, const void* fresh_v,
                              const akvs_probes* probes, int32_t n_units, int32_t n_query,
                              int32_t n_kv_heads, int32_t head_dim, float rope_base,
                              void* out_k, void* out_v, float* mu_k, float* mu_v,
                              void* scratch, void* stream);

/* Diagnostics of the residual model r_i = mu + xi_i (Section 3.4; the appendix's mean-explained
 * residual energy), for one layer of one request.  fresh_k / fresh_v: device [N][n_kv][hd],
 * the fresh K (rotated at global positions) and V of EVERY context token, e.g. from
 * AKVS_MODE_FULL; the cache arguments as in akvs_op_correct_layer; ctx_off: host [n_units+1].
 * Per unit u and per K | V, with r_i = fresh_i - reuse_i (K re-aligned to the unit's offset):
 *   mean[u]   = sum_i sel_i r_i / sum_i sel_i   (sel NULL: 1 -> the exact unit mean; sample
 *               multiplicities -> a probe-mean estimate with replacement; 0 if the sum is 0)
 *   energy[u] = { sum_i |r_i^K|^2, sum_i |r_i^K - w_i^K mu_K[u]|^2, the same two for V }
 * mu_k / mu_v: device [n_units][n_kv*hd] or both NULL (zero); w_k / w_v: device [N] or NULL (1);
 * sel_k / sel_v: device [N] or NULL; mean_k / mean_v: device [n_units][n_kv*hd] outputs or both
 * NULL; energy: device [n_units][4] float.  The mean-explained energy of a correction vector is
 * 1 - remaining / total.  scratch: akvs_op_scratch_bytes(N, 0, n_units, head_dim) bytes.
 * Returns AKVS_ERR_TOO_LARGE when n_kv * hd exceeds 4096. */
int32_t akvs_op_residual_stats(int32_t dtype, int32_t kv_format, const void* cache_k, const void* cache_v,
                               const void* k_meta, const void* v_meta, const int32_t* src_tok, const void* fresh_k,
                               const void* fresh_v, const int32_t* ctx_off, int32_t n_units, int32_t n_kv_heads,
                               int32_t head_dim, float rope_base, const float* sel_k, const float* sel_v,
                               const float* mu_k, const float* mu_v, const float* w_k, const float* w_v, float* mean_k,
                               float* mean_v, float* energy, void* scratch, void* stream);

/* Group quantiser of the cache (asymmetric min-max, groups of 64 along head_dim, float16
 * scale and minimum): x [n][n_kv][hd] -> codes [n][n_kv][hd*bits/8], meta half2 [n][n_kv][hd/64].
 * bits = 8 is the FP8 (E4M3) cast: one byte per value, meta unused (may be NULL). */
int32_t akvs_op_quantize(int32_t dtype, const void* x, int32_t n, int32_t n_kv_heads, int32_t head_dim,
                         int32_t bits, void* codes, void* meta, void* stream);

/* ====================================================================================
 * NOT PART OF THE SERVING SURFACE.  Test and measurement hooks: process-wide state, not
 * thread-safe, no paper passage behind any of them.  A serving caller needs none of these.
 * ==================================================================================== */

/* Cross-check switch for the tests: bit 0 set routes the 16-bit linear layers, bit 1 set the
 * 16-bit attention, to the CUDA-core kernels instead of the tcgen05 ones (default 0: tensor
 * cores for both).  Bits 2-3: tiling of the tcgen05 linear layers - 0 picked by shape
 * (default), 1 single CTAs, 2 CTA pairs wherever M > 128.  Bits 4-6: split-K of the residual
 * linear layers - 0 by the library's cost model (default), 1..4 that many splits.
 * Process-wide; not part of the serving surface. */
int32_t akvs_debug_set_linear_algo(int32_t algo);

/* Number of kernels this library has launched in this process so far. */
int64_t akvs_launch_count(void);

/* Per-launch device timing of kernel classes with CUDA events recorded on the launching
 * stream.  kind_mask has bit k set for class k: 1 = tensor-core linear layers (sub =
 * epilogue: 0 store, 1 residual, 2 SwiGLU; work = flops), 2 = correction pass (sub = kv
 * format; work = algorithmic bytes), 3 = tensor-core attention (work not filled in),
 * 4 = RMSNorm (work = bytes read and written), 5 = offset estimation (work not filled in);
 * 0 = off.  akvs_prof_enable allocates max_records event pairs (host objects only);
 * akvs_prof_read waits for the recorded events and returns per launch the elapsed ms, the
 * work and (class << 8 | sub); akvs_prof_reset forgets the records but keeps the events.
 * Not thread-safe. */
int32_t akvs_prof_enable(int32_t kind_mask, int32_t max_records);
int32_t akvs_prof_reset(void);
int32_t akvs_prof_read(int32_t capacity, float* ms, double* work, int32_t* sub, int32_t* n_out);

/* Launches ONLY the correction kernel of every layer from the check layer on, one after the
 * other, with exactly the arguments akvs_prefill_corrected(AKVS_MODE_CORRECTED) gives it: the
 * layer's cache slice in, the layer's out_k / out_v slice out, the request maps, offsets and
 * fresh rows that the preceding prefill left in `workspace`.  For timing the kernel back to
 * back over distinct buffers; the K/V it writes are those of the LAST layer's offsets and rows
 * and are not meant to be used.  Arguments as for the prefill it follows.  Asynchronous. */
int32_t akvs_debug_correct_repeat(const akvs_model_desc* model, const akvs_cache* cache, const akvs_request* req,
                                  const akvs_probes* probes, void* out_k, void* out_v, void* ctx,
                                  void* workspace, int64_t ws_bytes, void* stream);

/* Makes one bounded device-side wait run out, to exercise AKVS_ERR_TIMEOUT without a hang, a
 * trap or a fault: one CTA of one warp waits, with the same bounded wait the tensor-core kernels
 * use on their barriers, on a shared-memory barrier that nothing ever arrives at; after
 * `limit_cycles` SM clock cycles (clamped to [1000, 2e8], i.e. at most about 0.1 s) the wait gives
 * up, the kernel writes AKVS_ERR_TIMEOUT to the status word at the start of `workspace` (the word
 * akvs_check returns and clears) and exits normally.  The context stays usable.  Asynchronous. */
int32_t akvs_debug_wait_timeout(void* workspace, int64_t limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AKVS_H */
