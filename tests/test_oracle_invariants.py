"""Invariants of the oracle's four modes, and the transformer pinned to a composition of
stock torch CPU operators (float64)."""
import numpy as np
import pytest
import torch

import testgen
from oracle import akvs_oracle as orc
from helpers import small_cfg, small_workload, oracle_model, make_inputs

DT = np.float64


@pytest.fixture(scope="module")
def setup():
    w = small_workload()
    model = oracle_model(w.model, std_scale=8.0)     # large enough that residuals exceed 1
    lens, ctx, qry, units_ids = make_inputs(w)
    units = orc.encode_units(model, units_ids)
    return w, model, lens, ctx, qry, units_ids, units


# ----------------------------------------------------------------- P1: transformer vs stock torch ops

def _torch_forward(model, ids):
    """Independent formulation: torch rms_norm, complex-number RoPE, torch SDPA with
    repeat_interleave for GQA, torch silu."""
    c = model.cfg
    F = torch.nn.functional
    t = lambda a: torch.tensor(np.asarray(a, np.float64))
    T = len(ids)
    h = t(model.tok_emb)[torch.tensor(ids, dtype=torch.long)]
    half = c.head_dim // 2
    theta = torch.tensor(c.rope_base, dtype=torch.float64) ** (-torch.arange(half, dtype=torch.float64) * 2 / c.head_dim)
    rot = torch.polar(torch.ones(T, half, dtype=torch.float64), torch.arange(T, dtype=torch.float64)[:, None] * theta[None])

    def rope(x):                                   # x [T][H][hd]
        z = torch.complex(x[..., :half], x[..., half:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    Ks, Vs = [], []
    for lw in model.layers:
        x = F.rms_norm(h, (c.d_model,), t(lw["attn_norm"]), c.rms_eps)
        q = rope((x @ t(lw["wq"]).T).view(T, c.n_q_heads, c.head_dim))
        k = rope((x @ t(lw["wk"]).T).view(T, c.n_kv_heads, c.head_dim))
        v = (x @ t(lw["wv"]).T).view(T, c.n_kv_heads, c.head_dim)
        g = c.n_q_heads // c.n_kv_heads
        a = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.repeat_interleave(g, 1).transpose(0, 1)[None],
                                           v.repeat_interleave(g, 1).transpose(0, 1)[None], is_causal=True)[0]
        h = h + a.transpose(0, 1).reshape(T, -1) @ t(lw["wo"]).T
        x = F.rms_norm(h, (c.d_model,), t(lw["mlp_norm"]), c.rms_eps)
        h = h + (F.silu(x @ t(lw["w_gate"]).T) * (x @ t(lw["w_up"]).T)) @ t(lw["w_down"]).T
        Ks.append(k.numpy())
        Vs.append(v.numpy())
    out = F.rms_norm(h, (c.d_model,), t(model.final_norm), c.rms_eps)
    return out.numpy(), np.stack(Ks), np.stack(Vs)


def test_full_recompute_matches_stock_torch_ops_on_config1():
    w = testgen.workload("c1")
    model = oracle_model(w.model)
    lens, ctx, qry, _ = make_inputs(w)
    out, K, V = orc.full_recompute(model, ctx, qry)
    tout, tK, tV = _torch_forward(model, np.concatenate([ctx, qry]))
    assert orc.rel_l2(out, tout[-len(qry):]) < 1e-11
    assert orc.rel_l2(K, tK) < 1e-11 and orc.rel_l2(V, tV) < 1e-11


def test_fp32_variant_agrees_with_fp64(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    a = orc.full_recompute(model, ctx, qry, np.float64)
    b = orc.full_recompute(model, ctx, qry, np.float32)
    assert b[0].dtype == np.float32
    for x, y in zip(a, b):
        assert orc.rel_l2(y, x) < 2e-5


# ----------------------------------------------------------------- I1: 100 % refresh == full recompute

@pytest.mark.parametrize("check_layer", [1, 2, 3])
def test_full_refresh_equals_full_recompute(setup, check_layer):
    w, model, lens, ctx, qry, units_ids, units = setup
    full = orc.full_recompute(model, ctx, qry)
    r = orc.corrected_reuse(model, units, range(len(units)), ctx, qry, 10000, check_layer)
    assert len(r["rows"]) == len(ctx) + len(qry)
    assert orc.rel_l2(r["hidden"], full[0]) < 1e-12
    assert orc.rel_l2(r["K"], full[1]) < 1e-12 and orc.rel_l2(r["V"], full[2]) < 1e-12


# ----------------------------------------------------------------- I2: the first unit has zero residual

def test_first_unit_has_zero_residual(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    full = orc.full_recompute(model, ctx, qry)
    n0 = int(lens[0])
    for l in range(model.cfg.n_layers):
        kr, vr = orc.reuse_kv(model, units, range(len(units)), l)
        assert np.abs(full[1][l][:n0] - kr[:n0]).max() < 1e-12
        assert np.abs(full[2][l][:n0] - vr[:n0]).max() < 1e-12
        # ... and later units do not (cross-unit attention changes them) beyond layer 1
        if l >= 1:
            assert np.abs(full[2][l][n0:len(ctx)] - vr[n0:]).max() > 1e-3
    r = orc.corrected_reuse(model, units, range(len(units)), ctx, qry, 2500, 2)
    assert r["d_k"][:n0].max() < 1e-11 and r["probes"]["w_k"][:n0].max() < 1e-11


def test_first_layer_residual_is_zero_for_every_unit(setup):
    """Layer-1 K/V depend on token and position only, so after re-alignment they match."""
    w, model, lens, ctx, qry, units_ids, units = setup
    full = orc.full_recompute(model, ctx, qry)
    kr, vr = orc.reuse_kv(model, units, range(len(units)), 0)
    assert np.abs(full[1][0][:len(ctx)] - kr).max() < 1e-11
    assert np.abs(full[2][0][:len(ctx)] - vr).max() < 1e-12


# ----------------------------------------------------------------- I3: 0 % refresh == naive reuse

def test_zero_refresh_equals_naive_reuse(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    naive = orc.naive_reuse(model, units, range(len(units)), qry)
    r = orc.corrected_reuse(model, units, range(len(units)), ctx, qry, 0, 1)
    assert len(r["rows"]) == len(qry)
    assert orc.rel_l2(r["hidden"], naive[0]) < 1e-12
    assert orc.rel_l2(r["K"], naive[1]) < 1e-12 and orc.rel_l2(r["V"], naive[2]) < 1e-12


def test_zero_weights_leave_non_probes_stale(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    r = orc.corrected_reuse(model, units, range(len(units)), ctx, qry, 2500, 2, zero_weights=True)
    N = len(ctx)
    for l in range(1, model.cfg.n_layers):
        kr, vr = orc.reuse_kv(model, units, range(len(units)), l)
        non = np.setdiff1d(np.arange(N), r["probes"]["sk_idx"])
        assert np.array_equal(r["K"][l][non], kr[non])
        pk = r["probes"]["sk_idx"]
        assert np.abs(r["K"][l][pk] - kr[pk]).max() > 1e-6


# ----------------------------------------------------------------- I4: exact constant offsets are recovered

@pytest.mark.parametrize("check_layer", [1, 2])
def test_constant_offset_cache_recovers_full_recompute(setup, check_layer):
    w, model, lens, ctx, qry, units_ids, units = setup
    c = model.cfg
    full = orc.full_recompute(model, ctx, qry)
    off = orc.context_offsets(lens)
    g = np.random.default_rng(3)
    fake = []
    for u in range(len(lens)):
        a, e = off[u], off[u + 1]
        K, V = [], []
        for l in range(c.n_layers):
            ck = g.standard_normal((c.n_kv_heads, c.head_dim)) * 2      # ||c|| >> 1 -> w = 1
            cv = g.standard_normal((c.n_kv_heads, c.head_dim)) * 2
            K.append(orc.rope_rotate(full[1][l][a:e] - ck[None], np.full(e - a, -a), c.rope_base))
            V.append(full[2][l][a:e] - cv[None])
        fake.append({"K": np.stack(K), "V": np.stack(V)})
    r = orc.corrected_reuse(model, fake, range(len(fake)), ctx, qry, 2500, check_layer)
    assert r["probes"]["w_k"].min() == 1.0 and r["probes"]["w_v"].min() == 1.0
    assert orc.rel_l2(r["hidden"], full[0]) < 1e-10
    assert orc.rel_l2(r["K"], full[1]) < 1e-10 and orc.rel_l2(r["V"], full[2]) < 1e-10
    # naive reuse of the same cache is far off, so the test has teeth
    naive = orc.naive_reuse(model, fake, range(len(fake)), qry)
    assert orc.rel_l2(naive[1], full[1]) > 0.1


# ----------------------------------------------------------------- I5: re-alignment == encoding at the offset

def test_rerotation_equals_encoding_at_offset(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    c = model.cfg
    ids = units_ids[1]
    n, o = len(ids), 37
    pos = np.arange(o, o + n)
    h = orc.embed(model, ids)
    for l in range(c.n_layers):
        h, k, v = orc.dense_layer(model, l, h, pos)
        assert np.abs(k - orc.rope_rotate(units[1]["K"][l], np.full(n, o), c.rope_base)).max() < 1e-11
        assert np.abs(v - units[1]["V"][l]).max() < 1e-11


# ----------------------------------------------------------------- retrieval order, probes given, quantised cache

def test_retrieval_order_is_respected(setup):
    w, model, lens, ctx, qry, units_ids, units = setup
    order = [2, 0, 1]
    ctx2 = np.concatenate([units_ids[u] for u in order])
    full = orc.full_recompute(model, ctx2, qry)
    r = orc.corrected_reuse(model, units, order, ctx2, qry, 10000, 2)
    assert orc.rel_l2(r["hidden"], full[0]) < 1e-12
    r = orc.corrected_reuse(model, units, order, ctx2, qry, 2500, 2)
    n_first = len(units_ids[2])
    assert r["d_k"][:n_first].max() < 1e-11                      # whichever unit comes first is exact
    assert list(r["ctx_off"]) == [0, n_first, n_first + len(units_ids[0]), len(ctx2)]


def test_corrected_beats_naive_on_constant_plus_noise_cache(setup):
    """Residual model r = mu + xi (Section 3.4): with a dominant shared offset the
    corrected K is closer to fresh than the reused K."""
    w, model, lens, ctx, qry, units_ids, units = setup
    c = model.cfg
    full = orc.full_recompute(model, ctx, qry)
    off = orc.context_offsets(lens)
    g = np.random.default_rng(5)
    fake = []
    for u in range(len(lens)):
        a, e = off[u], off[u + 1]
        K = [orc.rope_rotate(full[1][l][a:e] - 2.0 + 0.05 * g.standard_normal(full[1][l][a:e].shape),
                             np.full(e - a, -a), c.rope_base) for l in range(c.n_layers)]
        V = [full[2][l][a:e] + 1.5 + 0.05 * g.standard_normal(full[2][l][a:e].shape) for l in range(c.n_layers)]
        fake.append({"K": np.stack(K), "V": np.stack(V)})
    r = orc.corrected_reuse(model, fake, range(len(fake)), ctx, qry, 2500, 1)
    naive = orc.naive_reuse(model, fake, range(len(fake)), qry)
    assert orc.rel_l2(r["K"], full[1]) < 0.2 * orc.rel_l2(naive[1], full[1])
    assert orc.rel_l2(r["V"], full[2]) < 0.2 * orc.rel_l2(naive[2], full[2])
    assert orc.rel_l2(r["hidden"], full[0]) < orc.rel_l2(naive[0], full[0])


@pytest.mark.parametrize("bits", [4, 2])
def test_quantised_cache_path(setup, bits):
    w, model, lens, ctx, qry, units_ids, units = setup
    cfg = small_cfg(hd=64, d_model=128, n_q=2, n_kv=1)
    wl = small_workload(cfg)
    model = oracle_model(cfg, std_scale=4.0)
    lens, ctx, qry, units_ids = make_inputs(wl)
    plain = orc.encode_units(model, units_ids)
    quant = orc.encode_units(model, units_ids, kv_bits=bits)
    for p, q in zip(plain, quant):
        assert q["K_codes"].max() <= (1 << bits) - 1
        step = q["K_scale"].astype(np.float64).max()
        assert np.abs(p["K"] - q["K"]).max() <= step * 0.51 + 1e-3
    # at 100 % refresh the cache content does not matter
    full = orc.full_recompute(model, ctx, qry)
    r = orc.corrected_reuse(model, quant, range(len(quant)), ctx, qry, 10000, 2)
    assert orc.rel_l2(r["hidden"], full[0]) < 1e-12
    # check layer 1 with a quantised cache: scores are the quantisation error, non-zero
    r = orc.corrected_reuse(model, quant, range(len(quant)), ctx, qry, 2500, 1)
    assert r["d_k"].min() > 0


def test_threads_over_heads_change_nothing():
    """ATTENTION_WORKERS only spreads the heads of one attention call over threads."""
    g = np.random.default_rng(5)
    q, k, v = g.standard_normal((9, 6, 8)), g.standard_normal((23, 2, 8)), g.standard_normal((23, 2, 8))
    qpos = np.sort(g.choice(23, 9, replace=False))
    a = orc.attention(q, k, v, qpos, np.arange(23))
    orc.ATTENTION_WORKERS = 4
    try:
        b = orc.attention(q, k, v, qpos, np.arange(23))
    finally:
        orc.ATTENTION_WORKERS = 1
    assert np.array_equal(a, b)
