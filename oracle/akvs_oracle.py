"""CPU oracle for probe-guided per-unit KV offset correction (TEST INFRASTRUCTURE ONLY).

This file is the slow, plain restatement of the method that the CUDA library is checked
against.  It is imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg; the product path never calls it.  It shares no code, tables or helpers
with the CUDA path.

What it follows
---------------
* Section 3.1 (motivation): a memory unit is encoded once, alone; at layer l direct reuse
  substitutes the cached K/V for the fresh ones, leaving residuals R = fresh - reuse.
* Section 3.3, "Probe selection": per-token divergence scores d_K, d_V at the check layer
  (the unnumbered equation there), top-b probe sets S^K, S^V per unit with b = ceil(r n),
  per-token weights w = min(d, 1), all fixed for every later layer.
* Section 3.3, "Mean estimation": the per-unit, per-layer offset is the plain mean of the
  probe residuals (unnumbered equation; Algorithm 1 line 5).
* Algorithm 1 lines 3-9 and the "correction" paragraph: a token in S^K keeps its fresh K,
  every other token of the unit gets K_reuse + w_K * mu_K; the same for V with S^V.

What the paper leaves open, and the reading taken here (each is listed in the design
notes too): the transformer itself (pre-norm RMSNorm, rotate-half RoPE, causal GQA
attention, SwiGLU MLP, no biases); keys are cached after RoPE at unit-local positions and
re-aligned by rotating through the unit's offset; residuals, offsets and corrections live
in that post-RoPE, global-position space; the score is one norm per token over all kv
heads; `check_layer` is 1-based and layers before it are computed densely for every row;
ties in the top-b are broken towards the smaller token index; b is computed from the
ratio in integer basis points.

* Section 4.5 (quantised caches): 2/4-bit asymmetric groups of 64 and the FP8 (E4M3) cast,
  the paper naming only the formats.
* Section 3.4 and the appendix on mean-explained residual energy: `residual_stats`.

Run-time plumbing that changes no arithmetic: `ATTENTION_WORKERS` > 1 computes the query
heads of one attention call in that many threads (each head is the same sequence of numpy
calls on the same data); `Model.w` converts a layer's weights to the working precision once
and keeps the last layer converted, and `encode_units` walks layer by layer over all units so
that this happens once per layer.

Arithmetic: float64 by default (`dtype=np.float32` gives the single-precision variant).
The quantisers are the exception: their decisions are taken on float32 values (float16
scale and minimum for the groups), because those decide integer codes.

Pins (tests/test_oracle_*.py): closed forms for the mean and the correction, brute-force
top-b, brute-force attention, an independent composition of stock library ops for the
transformer, Lemma 1's inequality, the Proposition 2 residual identity, quantiser error
bounds, the E4M3 cast by brute force over every code, hand-computed ties and an independent
library cast, the residual statistics by the variance identity and hand-computed weighted
means, and the invariants 100 % refresh == full recompute, first unit has zero
residual, 0 % refresh == naive reuse, exact constant-offset caches are recovered exactly.
No function here is "parity unpinned".
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ATTENTION_WORKERS = 1        # threads over query heads inside attention(); 1 = plain loop

# --------------------------------------------------------------------------- transformer parts


def rmsnorm(h, gain, eps, dtype=np.float64):
    """x_i = h_i / sqrt(mean(h^2) + eps) * gain_i, per row."""
    h = np.asarray(h, dtype)
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + dtype(eps)) * np.asarray(gain, dtype)


def rope_cos_sin(positions, head_dim, base):
    """cos/sin of p * base^(-2i/head_dim), i = 0..head_dim/2-1, in float64.

    `positions` may be negative (a rotation back)."""
    half = head_dim // 2
    inv_freq = np.float64(base) ** (-2.0 * np.arange(half, dtype=np.float64) / head_dim)
    ang = np.asarray(positions, np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def rope_rotate(x, positions, base, dtype=np.float64):
    """Rotate-half RoPE: pairs (i, i + hd/2) of every head of x [n][heads][hd] are turned
    through positions[n] * theta_i."""
    x = np.asarray(x, dtype)
    hd = x.shape[-1]
    half = hd // 2
    c, s = rope_cos_sin(positions, hd, base)
    c = c.astype(dtype)[:, None, :]
    s = s.astype(dtype)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def attention(q, k, v, q_pos, k_pos, k_first=None, dtype=np.float64, row_block=1024):
    """softmax(q k^T / sqrt(hd)) v for GQA heads.

    q [R][n_q][hd]; k, v [T][n_kv][hd]; query row r sees key j iff
    k_first[r] <= k_pos[j] <= q_pos[r]   (k_first defaults to -inf: plain causal).
    q head i reads kv head i // (n_q / n_kv).  Softmax subtracts the row maximum."""
    q = np.asarray(q, dtype)
    k = np.asarray(k, dtype)
    v = np.asarray(v, dtype)
    R, nq, hd = q.shape
    nkv = k.shape[1]
    g = nq // nkv
    q_pos = np.asarray(q_pos, np.int64)
    k_pos = np.asarray(k_pos, np.int64)
    lo = np.full(R, np.iinfo(np.int64).min, np.int64) if k_first is None else np.asarray(k_first, np.int64)
    out = np.empty((R, nq, hd), dtype)
    scale = dtype(1.0 / math.sqrt(hd))
    for r0 in range(0, R, row_block):
        r1 = min(R, r0 + row_block)
        visible = (k_pos[None, :] <= q_pos[r0:r1, None]) & (k_pos[None, :] >= lo[r0:r1, None])

        def one_head(hq):
            hk = hq // g
            s = (q[r0:r1, hq, :] @ k[:, hk, :].T) * scale
            s = np.where(visible, s, -np.inf)
            s = s - np.max(s, axis=1, keepdims=True)
            p = np.exp(s)
            p = p / np.sum(p, axis=1, keepdims=True)
            out[r0:r1, hq, :] = p @ v[:, hk, :]

        if ATTENTION_WORKERS > 1 and nq > 1:
            with ThreadPoolExecutor(ATTENTION_WORKERS) as ex:
                list(ex.map(one_head, range(nq)))
        else:
            for hq in range(nq):
                one_head(hq)
    return out


def silu(x):
    return x / (1.0 + np.exp(-x))


class Model:
    """Borrowed arrays of a decoder: `cfg` has n_layers, d_model, n_q_heads, n_kv_heads,
    head_dim, d_ff, rope_base, rms_eps; `layers[l]` is a dict of attn_norm, wq, wk, wv, wo,
    mlp_norm, w_gate, w_up, w_down, every projection stored [out][in]."""

    def __init__(self, cfg, tok_emb, layers, final_norm=None):
        self.cfg = cfg
        self.tok_emb = tok_emb
        self.layers = layers
        self.final_norm = np.ones(cfg.d_model, np.float32) if final_norm is None else final_norm
        self._conv = (None, None, {})

    def w(self, l, name, dtype=np.float64):
        """Layer l's array `name` in the working precision; the last layer asked for stays converted."""
        if self._conv[0] != l or self._conv[1] != dtype:
            self._conv = (l, dtype, {})
        c = self._conv[2]
        if name not in c:
            c[name] = np.asarray(self.layers[l][name], dtype)
        return c[name]


def embed(model, ids, dtype=np.float64):
    return np.asarray(model.tok_emb, dtype)[np.asarray(ids, np.int64)]


def layer_qkv(model, l, h, positions, dtype=np.float64):
    """Pre-norm, q/k/v projections, RoPE on q and k at `positions`."""
    c = model.cfg
    x = rmsnorm(h, model.w(l, "attn_norm", dtype), c.rms_eps, dtype)
    n = x.shape[0]
    q = (x @ model.w(l, "wq", dtype).T).reshape(n, c.n_q_heads, c.head_dim)
    k = (x @ model.w(l, "wk", dtype).T).reshape(n, c.n_kv_heads, c.head_dim)
    v = (x @ model.w(l, "wv", dtype).T).reshape(n, c.n_kv_heads, c.head_dim)
    q = rope_rotate(q, positions, c.rope_base, dtype)
    k = rope_rotate(k, positions, c.rope_base, dtype)
    return q, k, v


def layer_out(model, l, h, attn, dtype=np.float64):
    """h + attn W_o, then the SwiGLU MLP with its own pre-norm and residual."""
    c = model.cfg
    n = h.shape[0]
    h = h + attn.reshape(n, c.n_q_heads * c.head_dim) @ model.w(l, "wo", dtype).T
    x = rmsnorm(h, model.w(l, "mlp_norm", dtype), c.rms_eps, dtype)
    a = silu(x @ model.w(l, "w_gate", dtype).T) * (x @ model.w(l, "w_up", dtype).T)
    return h + a @ model.w(l, "w_down", dtype).T


def dense_layer(model, l, h, positions, k_first=None, dtype=np.float64):
    """One full layer over rows that are all present: returns (h', k, v)."""
    q, k, v = layer_qkv(model, l, h, positions, dtype)
    a = attention(q, k, v, positions, positions, k_first, dtype)
    return layer_out(model, l, h, a, dtype), k, v


# --------------------------------------------------------------------------- group quantiser

def quantize_groups(x, bits, group=64):
    """Asymmetric min-max quantisation of consecutive groups of `group` values along the
    last axis (the head dimension).  All decisions in float32; scale and minimum are
    rounded to float16 BEFORE they are used, so that codes and reconstructions are a
    function of stored values only.

        scale = (max - min) / (2^bits - 1);  code = clamp(rint((x - min16) / scale16), 0, 2^bits-1)
        scale16 == 0  ->  code = 0
    Returns (codes uint8 [..., hd], scale float16 [..., hd/group], minimum float16 [...])."""
    x = np.asarray(x, np.float32)
    shp = x.shape
    xg = x.reshape(shp[:-1] + (shp[-1] // group, group))
    levels = np.float32((1 << bits) - 1)
    mn = xg.min(axis=-1)
    mx = xg.max(axis=-1)
    scale16 = ((mx - mn) / levels).astype(np.float32).astype(np.float16)
    mn16 = mn.astype(np.float16)
    s = scale16.astype(np.float32)[..., None]
    m = mn16.astype(np.float32)[..., None]
    with np.errstate(divide="ignore", invalid="ignore"):
        t = ((xg - m).astype(np.float32) / s).astype(np.float32)
    code = np.rint(t)                       # round half to even
    code = np.clip(code, 0.0, levels)
    code = np.where(s == 0, np.float32(0), code)
    return code.astype(np.uint8).reshape(shp), scale16, mn16


def dequantize_groups(codes, scale16, mn16, group=64):
    """x = fma(code, scale, min) evaluated in float32 (one rounding)."""
    shp = codes.shape
    cg = codes.reshape(shp[:-1] + (shp[-1] // group, group)).astype(np.float64)
    s = scale16.astype(np.float64)[..., None]
    m = mn16.astype(np.float64)[..., None]
    # a float64 multiply-add of (<=4-bit integer) * float16 + float16 is exact, so rounding
    # it once to float32 is the fused multiply-add result
    return (cg * s + m).astype(np.float32).reshape(shp)


def pack_codes(codes, bits):
    """Little-endian packing within a byte, dimension ascending: element e of a row sits in
    byte e*bits//8 at bit offset (e*bits) % 8."""
    per = 8 // bits
    c = codes.reshape(codes.shape[:-1] + (codes.shape[-1] // per, per)).astype(np.uint16)
    out = np.zeros(c.shape[:-1], np.uint16)
    for i in range(per):
        out |= c[..., i] << (bits * i)
    return out.astype(np.uint8)


# --------------------------------------------------------------------------- residual diagnostics

def residual_stats(fresh, reuse, ctx_off, sel=None, mu=None, w=None):
    """Diagnostics of the residual model r_i = mu + xi_i (Section 3.4 and the appendix on
    mean-explained energy), per unit u with tokens a..e-1 and residual rows r_i = fresh_i -
    reuse_i (flattened over heads):

        mean[u]      = sum_i sel_i r_i / sum_i sel_i      (sel = 1: the exact unit mean; sel =
                       sample multiplicities: a probe-mean estimate; 0 where the sum is 0)
        total[u]     = sum_i |r_i|^2
        remaining[u] = sum_i |r_i - w_i mu[u]|^2          (mu = 0, w = 1 when not given)

    The mean-explained energy of a correction vector is 1 - remaining / total."""
    ctx_off = np.asarray(ctx_off, np.int64)
    M, N = len(ctx_off) - 1, int(ctx_off[-1])
    r = (np.asarray(fresh, np.float64) - np.asarray(reuse, np.float64)).reshape(N, -1)
    D = r.shape[1]
    sel = np.ones(N) if sel is None else np.asarray(sel, np.float64)
    w = np.ones(N) if w is None else np.asarray(w, np.float64)
    mu = np.zeros((M, D)) if mu is None else np.asarray(mu, np.float64).reshape(M, D)
    mean, total, remaining = np.zeros((M, D)), np.zeros(M), np.zeros(M)
    for u in range(M):
        a, e = int(ctx_off[u]), int(ctx_off[u + 1])
        ssum = sel[a:e].sum()
        if ssum > 0:
            mean[u] = (sel[a:e, None] * r[a:e]).sum(axis=0) / ssum
        total[u] = (r[a:e] ** 2).sum()
        remaining[u] = ((r[a:e] - w[a:e, None] * mu[u]) ** 2).sum()
    return mean, total, remaining


# --------------------------------------------------------------------------- FP8 cache

E4M3_MAX = 448.0


def e4m3_encode(x):
    """Element-wise cast to FP8 E4M3 (the format the quantisation study of Section 4.5 names:
    1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value
    448, subnormals in steps of 2^-9).  The paper gives no scaling, so the reading is a plain
    cast of the value (first rounded to float32): round to nearest, ties to the even mantissa,
    magnitudes above 448 saturate to 448.  Returns the uint8 bit patterns."""
    x = np.asarray(x, np.float32).astype(np.float64)
    if not np.all(np.isfinite(x)):
        raise ValueError("e4m3_encode: non-finite input")
    sign = np.signbit(x)
    a = np.minimum(np.abs(x), E4M3_MAX)
    _, ex = np.frexp(a)                              # a = m 2^ex, m in [0.5, 1)
    e = np.clip(ex - 1, -6, 8)                       # binade; everything below 2^-6 is subnormal
    q = np.exp2(e - 3.0)                             # spacing of the grid in that binade
    v = np.rint(a / q) * q                           # half to even; may land on the next binade's first value
    _, ex2 = np.frexp(v)
    e2 = ex2 - 1
    normal = v >= 2.0 ** -6
    ebits = np.where(normal, e2 + 7, 0).astype(np.int64)
    mant = np.where(normal, np.rint((v / np.exp2(np.where(normal, e2, 0).astype(np.float64)) - 1.0) * 8.0),
                    np.rint(v / 2.0 ** -9)).astype(np.int64)
    return ((sign.astype(np.int64) << 7) | (ebits << 3) | mant).astype(np.uint8)


def e4m3_decode(code):
    """Value of an E4M3 bit pattern (the two NaN patterns 0x7f / 0xff never occur here)."""
    c = np.asarray(code, np.uint8).astype(np.int64)
    s = np.where(c & 0x80, -1.0, 1.0)
    ebits, m = (c >> 3) & 15, c & 7
    return s * np.where(ebits == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * np.exp2(ebits - 7.0))


# --------------------------------------------------------------------------- the four modes

def encode_units(model, unit_ids_list, kv_bits=0, dtype=np.float64):
    """Section 3.1: each unit alone, positions 0..n-1, causal.  Returns a list (one entry
    per unit) of dicts with K [L][n][n_kv][hd] (post-RoPE at LOCAL positions) and V.
    With kv_bits in (2, 4) the cached values are the dequantised reconstructions and the
    codes/scale/minimum are kept beside them; kv_bits = 8 is the FP8 (E4M3) cache: the cached
    values are the decoded bytes, kept beside them as codes."""
    c = model.cfg
    out = []
    # every unit is its own sequence; the walk is layer by layer over all of them (the units do
    # not interact, so the order of the two loops changes nothing)
    hs = [embed(model, ids, dtype) for ids in unit_ids_list]
    Ks = [[] for _ in unit_ids_list]
    Vs = [[] for _ in unit_ids_list]
    for l in range(c.n_layers):
        for i, ids in enumerate(unit_ids_list):
            hs[i], k, v = dense_layer(model, l, hs[i], np.arange(len(ids)), None, dtype)
            Ks[i].append(k)
            Vs[i].append(v)
    for i in range(len(unit_ids_list)):
        unit = {"K": np.stack(Ks[i]), "V": np.stack(Vs[i]), "hidden": hs[i]}
        if kv_bits == 8:
            for name in ("K", "V"):
                unit[name + "_codes"] = e4m3_encode(unit[name])
                unit[name] = e4m3_decode(unit[name + "_codes"]).astype(dtype)
        elif kv_bits:
            for name in ("K", "V"):
                codes, s16, m16 = quantize_groups(unit[name], kv_bits)
                unit[name + "_codes"], unit[name + "_scale"], unit[name + "_min"] = codes, s16, m16
                unit[name] = dequantize_groups(codes, s16, m16).astype(dtype)
        out.append(unit)
    return out


def context_offsets(lengths):
    off = np.zeros(len(lengths) + 1, np.int64)
    off[1:] = np.cumsum(np.asarray(lengths, np.int64))
    return off


def full_recompute(model, ctx_ids, query_ids, dtype=np.float64, n_dense=None, h0=None):
    """The thing the method approximates: the concatenated context followed by the query,
    global positions 0..T-1, every row through every layer.  Returns final-normed query
    hidden [n_q][d], K, V [L][T][n_kv][hd].  `n_dense` stops after that many layers and
    returns the raw hidden state of all rows instead (used for the dense front)."""
    c = model.cfg
    ids = np.concatenate([np.asarray(ctx_ids, np.int64), np.asarray(query_ids, np.int64)])
    T = len(ids)
    pos = np.arange(T)
    h = embed(model, ids, dtype) if h0 is None else h0
    Ks, Vs = [], []
    L = c.n_layers if n_dense is None else n_dense
    for l in range(L):
        h, k, v = dense_layer(model, l, h, pos, None, dtype)
        Ks.append(k)
        Vs.append(v)
    if n_dense is not None:
        return h, Ks, Vs
    nq = len(query_ids)
    out = rmsnorm(h[T - nq:], model.final_norm, c.rms_eps, dtype)
    return out, np.stack(Ks), np.stack(Vs)


def reuse_kv(model, units, order, l, dtype=np.float64):
    """K_reuse, V_reuse of layer l for the context `order` (Section 3.1): the cached V as
    is, the cached K turned through the unit's global offset."""
    c = model.cfg
    lens = [units[u]["K"].shape[1] for u in order]
    off = context_offsets(lens)
    Ks, Vs = [], []
    for s, u in enumerate(order):
        n = lens[s]
        Ks.append(rope_rotate(units[u]["K"][l], np.full(n, off[s]), c.rope_base, dtype))
        Vs.append(np.asarray(units[u]["V"][l], dtype))
    return np.concatenate(Ks), np.concatenate(Vs)


def probe_budget(n, refresh_bp):
    """b = ceil(r n) with r = refresh_bp / 10000, in integers; clamped to [0, n]."""
    return int(min(n, max(0, (int(n) * int(refresh_bp) + 9999) // 10000)))


def divergence_scores(k_fresh, k_reuse, dtype=np.float64):
    """d_j = || fresh_j - reuse_j ||_2 over the token's whole [n_kv * hd] vector
    (Section 3.3, probe selection)."""
    diff = (np.asarray(k_fresh, dtype) - np.asarray(k_reuse, dtype)).reshape(len(k_fresh), -1)
    return np.sqrt(np.sum(diff * diff, axis=1))


def top_b(scores, b):
    """Indices of the b largest scores, larger first, equal scores by smaller index;
    returned ascending."""
    s = np.asarray(scores) + 0.0            # -0.0 -> +0.0
    if np.isnan(s).any():
        raise ValueError("NaN divergence score")
    order = np.argsort(-s, kind="stable")
    return np.sort(order[:b]).astype(np.int64)


def select_probes(d_k, d_v, ctx_off, refresh_bp):
    """Section 3.3 / Algorithm 1 line 2.  Per unit: S^K = top-b of d_K, S^V = top-b of d_V
    (global token indices, ascending within the unit); weights w = min(d, 1); `ctx_rows` =
    sorted union of all probes."""
    M = len(ctx_off) - 1
    sk, sv, off = [], [], [0]
    for u in range(M):
        a, e = int(ctx_off[u]), int(ctx_off[u + 1])
        b = probe_budget(e - a, refresh_bp)
        sk.append(a + top_b(d_k[a:e], b))
        sv.append(a + top_b(d_v[a:e], b))
        off.append(off[-1] + b)
    sk_idx = np.concatenate(sk) if sk else np.zeros(0, np.int64)
    sv_idx = np.concatenate(sv) if sv else np.zeros(0, np.int64)
    return {
        "sk_idx": sk_idx, "sv_idx": sv_idx, "probe_off": np.asarray(off, np.int64),
        "w_k": np.minimum(np.asarray(d_k), 1.0), "w_v": np.minimum(np.asarray(d_v), 1.0),
        "ctx_rows": np.union1d(sk_idx, sv_idx).astype(np.int64),
    }


def probe_offsets(fresh, reuse, s_idx, probe_off, dtype=np.float64):
    """mu_u = (1/b_u) * sum_{j in S_u} (fresh_j - reuse_j), per unit (mean estimation).
    `fresh` and `reuse` are indexed by global token position; b_u = 0 gives mu_u = 0."""
    M = len(probe_off) - 1
    mu = np.zeros((M,) + fresh.shape[1:], dtype)
    for u in range(M):
        S = s_idx[probe_off[u]:probe_off[u + 1]]
        if len(S):
            mu[u] = np.sum(np.asarray(fresh[S], dtype) - np.asarray(reuse[S], dtype), axis=0) / dtype(len(S))
    return mu


def apply_correction(fresh, reuse, s_idx, w, mu, ctx_off, dtype=np.float64):
    """Algorithm 1 lines 7-8: probe tokens take their fresh state, every other token of
    unit u gets reuse_j + w_j * mu_u."""
    out = np.array(reuse, dtype, copy=True)
    for u in range(len(ctx_off) - 1):
        a, e = int(ctx_off[u]), int(ctx_off[u + 1])
        out[a:e] += np.asarray(w[a:e], dtype)[:, None, None] * mu[u][None]
    out[s_idx] = np.asarray(fresh[s_idx], dtype)
    return out


def naive_reuse(model, units, order, query_ids, dtype=np.float64):
    """Direct reuse (Section 3.1): context K/V at every layer are the re-aligned cache;
    only the query rows are computed and they attend to reused KV plus their own."""
    c = model.cfg
    N = sum(units[u]["K"].shape[1] for u in order)
    nq = len(query_ids)
    qpos = np.arange(N, N + nq)
    allpos = np.arange(N + nq)
    h = embed(model, query_ids, dtype)
    Ks, Vs = [], []
    for l in range(c.n_layers):
        kr, vr = reuse_kv(model, units, order, l, dtype)
        q, k, v = layer_qkv(model, l, h, qpos, dtype)
        K = np.concatenate([kr, k])
        V = np.concatenate([vr, v])
        a = attention(q, K, V, qpos, allpos, None, dtype)
        h = layer_out(model, l, h, a, dtype)
        Ks.append(K)
        Vs.append(V)
    return rmsnorm(h, model.final_norm, c.rms_eps, dtype), np.stack(Ks), np.stack(Vs)


def corrected_reuse(model, units, order, ctx_ids, query_ids, refresh_bp, check_layer=2,
                    probes=None, zero_weights=False, dtype=np.float64):
    """Algorithm 1 around a transformer.

    a. layers 1..check_layer-1: every row, as in full recompute (their K/V are fresh);
    b. at the check layer: fresh K/V of every context row from the dense hidden state,
       scores against the re-aligned cache, probe sets and weights (unless `probes` is given);
    c. for every layer from the check layer on, carrying only the probe and query rows:
       fresh q/k/v of those rows; per-unit offsets from the probes; corrected K/V for the
       whole context; the carried rows attend causally over the corrected K/V; W_o, MLP.
    `zero_weights` forces w = 0: selective recompute with the rest left stale."""
    c = model.cfg
    lens = [units[u]["K"].shape[1] for u in order]
    ctx_off = context_offsets(lens)
    N = int(ctx_off[-1])
    nq = len(query_ids)
    T = N + nq
    lc = check_layer - 1                       # 0-based
    h_all, Ks, Vs = full_recompute(model, ctx_ids, query_ids, dtype, n_dense=lc)
    Ks = [np.asarray(x) for x in Ks]
    Vs = [np.asarray(x) for x in Vs]
    allpos = np.arange(T)

    # b. scores at the check layer (fresh K/V of all context rows; no attention needed)
    _, k_chk, v_chk = layer_qkv(model, lc, h_all[:N], allpos[:N], dtype)
    kr, vr = reuse_kv(model, units, order, lc, dtype)
    d_k = divergence_scores(k_chk, kr, dtype)
    d_v = divergence_scores(v_chk, vr, dtype)
    if probes is None:
        probes = select_probes(d_k, d_v, ctx_off, refresh_bp)
    sk, sv, poff = probes["sk_idx"], probes["sv_idx"], probes["probe_off"]
    w_k = np.zeros(N) if zero_weights else probes["w_k"]
    w_v = np.zeros(N) if zero_weights else probes["w_v"]
    rows = np.concatenate([probes["ctx_rows"], np.arange(N, T)]).astype(np.int64)
    n_probe_rows = len(probes["ctx_rows"])

    h = h_all[rows]
    mus = []
    for l in range(lc, c.n_layers):
        q, k, v = layer_qkv(model, l, h, rows, dtype)
        kr, vr = reuse_kv(model, units, order, l, dtype)
        k_f = np.zeros_like(kr)
        v_f = np.zeros_like(vr)
        k_f[rows[:n_probe_rows]] = k[:n_probe_rows]
        v_f[rows[:n_probe_rows]] = v[:n_probe_rows]
        mu_k = probe_offsets(k_f, kr, sk, poff, dtype)
        mu_v = probe_offsets(v_f, vr, sv, poff, dtype)
        K = np.concatenate([apply_correction(k_f, kr, sk, w_k, mu_k, ctx_off, dtype), k[n_probe_rows:]])
        V = np.concatenate([apply_correction(v_f, vr, sv, w_v, mu_v, ctx_off, dtype), v[n_probe_rows:]])
        a = attention(q, K, V, rows, allpos, None, dtype)
        h = layer_out(model, l, h, a, dtype)
        Ks.append(K)
        Vs.append(V)
        mus.append((mu_k, mu_v))
    out = rmsnorm(h[n_probe_rows:], model.final_norm, c.rms_eps, dtype)
    return {"hidden": out, "K": np.stack(Ks), "V": np.stack(Vs), "d_k": d_k, "d_v": d_v,
            "probes": probes, "rows": rows, "mu": mus, "ctx_off": ctx_off}


def rel_l2(a, b):
    """|| a - b ||_2 / || b ||_2 over the whole tensor (b is the reference)."""
    a = np.asarray(a, np.float64).ravel()
    b = np.asarray(b, np.float64).ravel()
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))
