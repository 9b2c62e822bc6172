"""ctypes binding of libakvs.so: argument marshalling only.

Every step of the path runs inside the library's CUDA kernels; torch is used here for
device memory and for the current stream, nothing else.  There is no CPU fallback: if the
shared library is missing or was not built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libakvs.so")

OK = 0
ERR = {0: "AKVS_OK", -1: "AKVS_ERR_INVALID_ARG", -2: "AKVS_ERR_SHAPE", -3: "AKVS_ERR_WORKSPACE",
       -4: "AKVS_ERR_UNSUPPORTED", -5: "AKVS_ERR_CUDA", -6: "AKVS_ERR_TIMEOUT", -7: "AKVS_ERR_NAN_SCORE",
       -8: "AKVS_ERR_TOO_LARGE"}
F32, BF16, F16 = 0, 1, 2
KV_NATIVE, KV_Q2, KV_Q4, KV_FP8 = 0, 2, 4, 8
MODE_CORRECTED, MODE_NAIVE, MODE_FULL = 0, 1, 2

EXPORTS = ["akvs_workspace_bytes", "akvs_debug_set_linear_algo", "akvs_launch_count", "akvs_prof_enable",
           "akvs_prof_reset", "akvs_prof_read", "akvs_encode_units", "akvs_select_probes", "akvs_prefill_corrected",
           "akvs_free", "akvs_check", "akvs_op_linear", "akvs_op_linear_residual", "akvs_op_rope", "akvs_op_attention",
           "akvs_op_scratch_bytes", "akvs_op_select", "akvs_op_select_static", "akvs_op_correct_layer",
           "akvs_op_quantize", "akvs_op_residual_stats", "akvs_debug_correct_repeat", "akvs_debug_wait_timeout"]
STATIC_MAX_CTX, STATIC_MAX_UNITS = 16384, 1024


class AkvsError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {ERR.get(code, code)}")
        self.code = code


class ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ff",
                                         "vocab", "dtype")] + \
               [("rope_base", C.c_float), ("rms_eps", C.c_float), ("tok_emb", C.c_void_p),
                ("final_norm", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate",
                                                     "w_up", "w_down")]


class CacheDesc(C.Structure):
    _fields_ = [("n_units", C.c_int32), ("n_tokens", C.c_int32), ("kv_format", C.c_int32),
                ("unit_off", C.POINTER(C.c_int32)), ("token_ids", C.c_void_p), ("k", C.c_void_p),
                ("v", C.c_void_p), ("k_meta", C.c_void_p), ("v_meta", C.c_void_p),
                ("layer_ready", C.POINTER(C.c_void_p))]


class RequestDesc(C.Structure):
    _fields_ = [("n_units", C.c_int32), ("unit_ids", C.POINTER(C.c_int32)), ("n_query", C.c_int32),
                ("query_ids", C.c_void_p), ("n_requests", C.c_int32), ("req_unit_off", C.POINTER(C.c_int32)),
                ("req_query_off", C.POINTER(C.c_int32))]


class ProbesDesc(C.Structure):
    _fields_ = [("n_ctx", C.c_int32), ("n_probe_rows", C.c_int32), ("n_rows", C.c_int32)] + \
               [(n, C.c_void_p) for n in ("ctx_off", "probe_off", "sk_idx", "sv_idx", "w_k", "w_v", "d_k", "d_v",
                                          "rows")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2607_21604_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    for name in EXPORTS:
        getattr(lib, name)                       # raises AttributeError if a symbol is absent
    lib.akvs_op_scratch_bytes.restype = C.c_int64
    lib.akvs_launch_count.restype = C.c_int64
    lib.akvs_free.restype = None
    return lib


lib = _load()


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _chk(code, where):
    if code != OK:
        raise AkvsError(code, where)


_TORCH = {F32: torch.float32, BF16: torch.bfloat16, F16: torch.float16}


def torch_dtype(dtype):
    return _TORCH[dtype]


_tdtype = torch_dtype


class Model:
    """Device-resident weights + the POD description the library reads.

    `layers[l]` maps attn_norm, wq, wk, wv, wo, mlp_norm, w_gate, w_up, w_down to CUDA tensors
    (projections [out][in] in the model dtype, norm gains float32)."""
    NAMES = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")

    def __init__(self, cfg, tok_emb, layers, final_norm, dtype):
        self.cfg, self.tok_emb, self.layers, self.final_norm, self.dtype = cfg, tok_emb, layers, final_norm, dtype
        L = len(layers)
        self._arrays = {}
        d = ModelDesc()
        d.n_layers, d.d_model, d.n_q_heads, d.n_kv_heads = L, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads
        d.head_dim, d.d_ff, d.vocab, d.dtype = cfg.head_dim, cfg.d_ff, cfg.vocab, dtype
        d.rope_base, d.rms_eps = cfg.rope_base, cfg.rms_eps
        d.tok_emb, d.final_norm = tok_emb.data_ptr(), final_norm.data_ptr()
        for n in self.NAMES:
            arr = (C.c_void_p * L)(*[layers[l][n].data_ptr() for l in range(L)])
            self._arrays[n] = arr
            setattr(d, n, C.cast(arr, C.POINTER(C.c_void_p)))
        self.desc = d

    @classmethod
    def from_layer_fn(cls, cfg, tok_emb, layer_fn, n_threads=8, device="cuda"):
        """Uploads a model layer by layer: `layer_fn(l)` returns the host arrays of layer l.  At
        most `n_threads` layers are resident on the host at a time (the 32B-class model does
        not fit in host memory as float32)."""
        from concurrent.futures import ThreadPoolExecutor
        dtype = {"f32": F32, "bf16": BF16, "f16": F16}[cfg.dtype]
        td = _tdtype(dtype)
        up = lambda a, t: torch.from_numpy(a).to(device=device, dtype=t).contiguous()
        dl = [None] * cfg.n_layers
        with ThreadPoolExecutor(n_threads) as ex:
            pending = {}
            nxt = 0
            for l in range(cfg.n_layers):
                while nxt < cfg.n_layers and len(pending) < n_threads:
                    pending[nxt] = ex.submit(layer_fn, nxt)
                    nxt += 1
                lw = pending.pop(l).result()
                dl[l] = {n: up(lw[n], torch.float32 if "norm" in n else td) for n in cls.NAMES}
                del lw
        fn = torch.ones(cfg.d_model, dtype=torch.float32, device=device)
        return cls(cfg, up(tok_emb, td), dl, fn, dtype)

    @classmethod
    def from_numpy(cls, cfg, tok_emb, layers, final_norm=None, device="cuda"):
        """Uploads host arrays (float32 values, bf16-representable for bf16 models)."""
        dtype = {"f32": F32, "bf16": BF16, "f16": F16}[cfg.dtype]
        td = _tdtype(dtype)
        up = lambda a, t: torch.from_numpy(a).to(device=device, dtype=t).contiguous()
        dl = [{n: up(lw[n], torch.float32 if "norm" in n else td) for n in cls.NAMES} for lw in layers]
        fn = torch.ones(cfg.d_model, dtype=torch.float32, device=device) if final_norm is None else up(final_norm, torch.float32)
        return cls(cfg, up(tok_emb, td), dl, fn, dtype)


class UnitStore:
    """The unit cache: token ids and unit offsets in, per-layer K/V out (akvs_encode_units)."""

    def __init__(self, model, unit_lengths, token_ids, kv_format=KV_NATIVE, device="cuda"):
        cfg = model.cfg
        self.model, self.kv_format = model, kv_format
        self.n_units = len(unit_lengths)
        off = [0]
        for n in unit_lengths:
            off.append(off[-1] + int(n))
        self.unit_off = (C.c_int32 * (self.n_units + 1))(*off)
        self.n_tokens = off[-1]
        self.token_ids = torch.as_tensor(token_ids, dtype=torch.int32).to(device).contiguous()
        L, N, dkv = len(model.layers), self.n_tokens, cfg.n_kv_heads * cfg.head_dim
        if kv_format == KV_NATIVE:
            td = _tdtype(model.dtype)
            self.k = torch.zeros((L, N, cfg.n_kv_heads, cfg.head_dim), dtype=td, device=device)
            self.v = torch.zeros_like(self.k)
            self.k_meta = self.v_meta = None
        elif kv_format == KV_FP8:
            self.k = torch.zeros((L, N, cfg.n_kv_heads, cfg.head_dim), dtype=torch.uint8, device=device)
            self.v = torch.zeros_like(self.k)
            self.k_meta = self.v_meta = None
        else:
            self.k = torch.zeros((L, N, cfg.n_kv_heads, cfg.head_dim * kv_format // 8), dtype=torch.uint8, device=device)
            self.v = torch.zeros_like(self.k)
            self.k_meta = torch.zeros((L, N, cfg.n_kv_heads, cfg.head_dim // 64, 2), dtype=torch.float16, device=device)
            self.v_meta = torch.zeros_like(self.k_meta)
        d = CacheDesc()
        d.n_units, d.n_tokens, d.kv_format = self.n_units, self.n_tokens, kv_format
        d.unit_off = C.cast(self.unit_off, C.POINTER(C.c_int32))
        d.token_ids, d.k, d.v = self.token_ids.data_ptr(), self.k.data_ptr(), self.v.data_ptr()
        d.k_meta = self.k_meta.data_ptr() if self.k_meta is not None else None
        d.v_meta = self.v_meta.data_ptr() if self.v_meta is not None else None
        self.desc = d
        self._events = None

    def set_layer_events(self, events):
        """`events`: one recorded torch.cuda.Event per layer (or None to clear).  The library then
        waits for events[l] before it first reads layer l (a cache streamed in from the host)."""
        if events is None:
            self._events = None
            self.desc.layer_ready = None
            return
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        self._events = (arr, events)
        self.desc.layer_ready = C.cast(arr, C.POINTER(C.c_void_p))


class Probes:
    """Caller-owned probe arrays for a request with n_ctx context tokens."""
    INT = ("ctx_off", "probe_off", "sk_idx", "sv_idx", "rows")
    FLT = ("w_k", "w_v", "d_k", "d_v")

    def __init__(self, n_ctx, n_units, n_query, device="cuda"):
        sizes = {"ctx_off": n_units + 1, "probe_off": n_units + 1, "sk_idx": n_ctx, "sv_idx": n_ctx,
                 "rows": n_ctx + n_query, "w_k": n_ctx, "w_v": n_ctx, "d_k": n_ctx, "d_v": n_ctx}
        d = ProbesDesc()
        for n in self.INT:
            setattr(self, n, torch.zeros(max(1, sizes[n]), dtype=torch.int32, device=device))
        for n in self.FLT:
            setattr(self, n, torch.zeros(max(1, sizes[n]), dtype=torch.float32, device=device))
        for n in self.INT + self.FLT:
            setattr(d, n, getattr(self, n).data_ptr())
        self.desc = d

    n_ctx = property(lambda s: s.desc.n_ctx)
    n_probe_rows = property(lambda s: s.desc.n_probe_rows)
    n_rows = property(lambda s: s.desc.n_rows)


class Request:
    """One request (unit ids in retrieval order + query ids) or, with `batch`, several requests
    that share the model: `Request.batch([(unit_ids, query_ids), ...])`."""

    def __init__(self, unit_ids, query_ids, device="cuda", unit_off=None, query_off=None):
        self.unit_ids = (C.c_int32 * max(1, len(unit_ids)))(*[int(u) for u in unit_ids])
        self.query_ids = torch.as_tensor(query_ids, dtype=torch.int32).to(device).contiguous()
        d = RequestDesc()
        d.n_units, d.n_query = len(unit_ids), int(self.query_ids.numel())
        d.unit_ids = C.cast(self.unit_ids, C.POINTER(C.c_int32))
        d.query_ids = self.query_ids.data_ptr()
        d.n_requests = 0
        if unit_off is not None:
            assert query_off is not None and len(unit_off) == len(query_off) >= 2
            self.unit_off = (C.c_int32 * len(unit_off))(*[int(x) for x in unit_off])
            self.query_off = (C.c_int32 * len(query_off))(*[int(x) for x in query_off])
            d.n_requests = len(unit_off) - 1
            d.req_unit_off = C.cast(self.unit_off, C.POINTER(C.c_int32))
            d.req_query_off = C.cast(self.query_off, C.POINTER(C.c_int32))
        self.desc = d

    @classmethod
    def batch(cls, requests, device="cuda"):
        units, queries, uo, qo = [], [], [0], [0]
        for u, q in requests:
            units += [int(x) for x in u]
            queries += [int(x) for x in q]
            uo.append(len(units))
            qo.append(len(queries))
        return cls(units, queries, device=device, unit_off=uo, query_off=qo)


def workspace_bytes(model, n_ctx, n_query, n_units, check_layer):
    out = C.c_int64(0)
    _chk(lib.akvs_workspace_bytes(C.byref(model.desc), n_ctx, n_query, n_units, check_layer, C.byref(out)),
         "akvs_workspace_bytes")
    return out.value


def alloc_workspace(nbytes, device="cuda"):
    return torch.empty(max(256, nbytes), dtype=torch.uint8, device=device)


def encode_units(model, store, workspace):
    _chk(lib.akvs_encode_units(C.byref(model.desc), C.byref(store.desc), _ptr(workspace),
                               C.c_int64(workspace.numel()), _stream()), "akvs_encode_units")


def select_probes(model, store, req, refresh_bp, check_layer, probes, ctx, workspace):
    """`ctx` is a ctypes.c_void_p holder (initially empty) that the library fills."""
    _chk(lib.akvs_select_probes(C.byref(model.desc), C.byref(store.desc), C.byref(req.desc), refresh_bp, check_layer,
                                C.byref(probes.desc), C.byref(ctx), _ptr(workspace), C.c_int64(workspace.numel()),
                                _stream()), "akvs_select_probes")


def prefill_corrected(model, store, req, probes, mode, out_hidden, out_k, out_v, ctx, workspace):
    _chk(lib.akvs_prefill_corrected(C.byref(model.desc), C.byref(store.desc), C.byref(req.desc),
                                    C.byref(probes.desc) if probes is not None else None, mode, _ptr(out_hidden),
                                    _ptr(out_k), _ptr(out_v), ctx if ctx is not None else None, _ptr(workspace),
                                    C.c_int64(workspace.numel()), _stream()), "akvs_prefill_corrected")


def free(ctx):
    if ctx is not None and ctx.value:
        lib.akvs_free(ctx)
        ctx.value = None


def check(workspace):
    return lib.akvs_check(_ptr(workspace), _stream())


def launch_count():
    return int(lib.akvs_launch_count())


def prof_enable(kind, max_records=0):
    _chk(lib.akvs_prof_enable(kind, max_records), "akvs_prof_enable")


def prof_reset():
    lib.akvs_prof_reset()


def prof_read(capacity=1 << 16):
    ms = (C.c_float * capacity)()
    work = (C.c_double * capacity)()
    sub = (C.c_int32 * capacity)()
    n = C.c_int32(0)
    _chk(lib.akvs_prof_read(capacity, ms, work, sub, C.byref(n)), "akvs_prof_read")
    return [(ms[i], work[i], sub[i]) for i in range(n.value)]


def debug_correct_repeat(model, store, req, probes, out_k, out_v, ctx, workspace):
    """Measurement hook: the correction kernel of every selective layer, back to back."""
    _chk(lib.akvs_debug_correct_repeat(C.byref(model.desc), C.byref(store.desc), C.byref(req.desc),
                                       C.byref(probes.desc), _ptr(out_k), _ptr(out_v), ctx, _ptr(workspace),
                                       C.c_int64(workspace.numel()), _stream()), "akvs_debug_correct_repeat")


def debug_wait_timeout(workspace, limit_cycles):
    """Test hook: a bounded device wait that runs out and reports AKVS_ERR_TIMEOUT through `check`."""
    _chk(lib.akvs_debug_wait_timeout(_ptr(workspace), C.c_int64(limit_cycles), _stream()), "akvs_debug_wait_timeout")


def alloc_outputs(model, n_ctx, n_query, device="cuda"):
    cfg = model.cfg
    td = _tdtype(model.dtype)
    T = n_ctx + n_query
    hid = torch.zeros((n_query, cfg.d_model), dtype=torch.float32, device=device)
    k = torch.zeros((len(model.layers), T, cfg.n_kv_heads, cfg.head_dim), dtype=td, device=device)
    return hid, k, torch.zeros_like(k)


# ------------------------------------------------------------------------------- single steps

def _dt(t):
    return {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}[t.dtype]


def op_linear(x, w, algo=0):
    dtype = _dt(x)
    M, K = x.shape
    N = w.shape[0]
    y = torch.empty((M, N), dtype=x.dtype, device=x.device)
    _chk(lib.akvs_op_linear(dtype, _ptr(x), _ptr(w), _ptr(y), M, N, K, algo, _stream()), "akvs_op_linear")
    return y


def op_linear_residual(x, w, h, algo=0, splits=0):
    """h (float32 [M][N], in place) += x w^T."""
    dtype = _dt(x)
    M, K = x.shape
    N = w.shape[0]
    assert h.dtype == torch.float32 and tuple(h.shape) == (M, N) and h.is_contiguous()
    _chk(lib.akvs_op_linear_residual(dtype, _ptr(x), _ptr(w), _ptr(h), M, N, K, algo, splits, _stream()),
         "akvs_op_linear_residual")
    return h


def op_rope(x, pos, base):
    dtype = _dt(x)
    n, H, hd = x.shape
    _chk(lib.akvs_op_rope(dtype, _ptr(x), _ptr(pos), n, H, hd, C.c_float(base), _stream()), "akvs_op_rope")
    return x


def op_attention(q, k, v, k_lo, k_hi, algo=0):
    dtype = _dt(q)
    R, nq, hd = q.shape
    T, nkv, _ = k.shape
    out = torch.empty_like(q)
    _chk(lib.akvs_op_attention(dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(k_lo), _ptr(k_hi), R, T, nq, nkv, hd,
                               algo, _stream()), "akvs_op_attention")
    return out


def op_scratch(n_ctx, n_query, n_units, head_dim, device="cuda"):
    return alloc_workspace(lib.akvs_op_scratch_bytes(n_ctx, n_query, n_units, head_dim), device)


def op_select(d_k, d_v, ctx_off, n_query, refresh_bp):
    M = len(ctx_off) - 1
    N = int(ctx_off[-1])
    probes = Probes(N, M, n_query, d_k.device)
    off = (C.c_int32 * (M + 1))(*[int(x) for x in ctx_off])
    scratch = op_scratch(N, n_query, M, 128, d_k.device)
    _chk(lib.akvs_op_select(_ptr(d_k), _ptr(d_v), off, M, n_query, refresh_bp, C.byref(probes.desc), _ptr(scratch),
                            _stream()), "akvs_op_select")
    return probes


def op_select_static(d_k, d_v, ctx_off, n_query, refresh_bp, probes=None):
    """Selection without a scratch buffer, for callers that must not allocate device memory:
    the library's built-in array is used (limits STATIC_MAX_CTX / STATIC_MAX_UNITS).  Pass
    `probes` to reuse output arrays; this wrapper only allocates them when none are given."""
    M = len(ctx_off) - 1
    N = int(ctx_off[-1])
    if probes is None:
        probes = Probes(N, M, n_query, d_k.device)
    off = (C.c_int32 * (M + 1))(*[int(x) for x in ctx_off])
    _chk(lib.akvs_op_select_static(_ptr(d_k), _ptr(d_v), off, M, n_query, refresh_bp, C.byref(probes.desc),
                                   _stream()), "akvs_op_select_static")
    return probes


def op_correct_layer(dtype, kv_format, cache_k, cache_v, k_meta, v_meta, src_tok, fresh_k, fresh_v, probes, n_units,
                     n_query, n_kv, hd, base, scratch=None):
    N = probes.n_ctx
    T = N + n_query
    td = _tdtype(dtype)
    out_k = torch.empty((T, n_kv, hd), dtype=td, device=fresh_k.device)
    out_v = torch.empty_like(out_k)
    mu_k = torch.empty((n_units, n_kv * hd), dtype=torch.float32, device=fresh_k.device)
    mu_v = torch.empty_like(mu_k)
    if scratch is None:
        scratch = op_scratch(N, n_query, n_units, hd, fresh_k.device)
    _chk(lib.akvs_op_correct_layer(dtype, kv_format, _ptr(cache_k), _ptr(cache_v), _ptr(k_meta), _ptr(v_meta),
                                   _ptr(src_tok), _ptr(fresh_k), _ptr(fresh_v), C.byref(probes.desc), n_units,
                                   n_query, n_kv, hd, C.c_float(base), _ptr(out_k), _ptr(out_v), _ptr(mu_k),
                                   _ptr(mu_v), _ptr(scratch), _stream()), "akvs_op_correct_layer")
    return out_k, out_v, mu_k, mu_v


def op_residual_stats(dtype, kv_format, cache_k, cache_v, k_meta, v_meta, src_tok, fresh_k, fresh_v, ctx_off, n_kv, hd,
                      base, sel_k=None, sel_v=None, mu_k=None, mu_v=None, w_k=None, w_v=None):
    """Unit means of the residual (under selection weights) and total / remaining residual energy.
    Returns (mean_k, mean_v [M][n_kv*hd], energy [M][4] = K total, K remaining, V total, V remaining)."""
    M = len(ctx_off) - 1
    N = int(ctx_off[-1])
    dev_ = fresh_k.device
    off = (C.c_int32 * (M + 1))(*[int(x) for x in ctx_off])
    mean_k = torch.zeros((M, n_kv * hd), dtype=torch.float32, device=dev_)
    mean_v = torch.zeros_like(mean_k)
    energy = torch.zeros((M, 4), dtype=torch.float32, device=dev_)
    scratch = op_scratch(N, 0, M, hd, dev_)
    _chk(lib.akvs_op_residual_stats(dtype, kv_format, _ptr(cache_k), _ptr(cache_v), _ptr(k_meta), _ptr(v_meta),
                                    _ptr(src_tok), _ptr(fresh_k), _ptr(fresh_v), off, M, n_kv, hd, C.c_float(base),
                                    _ptr(sel_k), _ptr(sel_v), _ptr(mu_k), _ptr(mu_v), _ptr(w_k), _ptr(w_v),
                                    _ptr(mean_k), _ptr(mean_v), _ptr(energy), _ptr(scratch), _stream()),
         "akvs_op_residual_stats")
    return mean_k, mean_v, energy


def op_quantize(x, bits):
    dtype = _dt(x)
    n, nkv, hd = x.shape
    codes = torch.empty((n, nkv, hd * bits // 8), dtype=torch.uint8, device=x.device)
    meta = None if bits == KV_FP8 else torch.empty((n, nkv, hd // 64, 2), dtype=torch.float16, device=x.device)
    _chk(lib.akvs_op_quantize(dtype, _ptr(x), n, nkv, hd, bits, _ptr(codes), _ptr(meta), _stream()),
         "akvs_op_quantize")
    return codes, meta
