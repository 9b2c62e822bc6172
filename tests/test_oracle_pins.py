"""Pins of the CPU oracle against things other than itself: closed forms, brute force,
library routines, and the inequalities/identities the paper proves."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import akvs_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(7)


# ----------------------------------------------------------------- budget b = ceil(r n)  (Section 3.3)

def test_budget_golden_file():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "probe_budget.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) >= 10
    for n, bp, b in rows:
        assert orc.probe_budget(int(n), int(bp)) == int(b), (n, bp, b)


def test_budget_exact_rational():
    for n in list(range(0, 400, 7)) + [320, 384, 256, 1, 2, 3]:
        for bp in (0, 1, 500, 1000, 1500, 2000, 2500, 3000, 3333, 9999, 10000):
            want = min(n, math.ceil(Fraction(bp, 10000) * n))
            assert orc.probe_budget(n, bp) == want
    # the float pitfall the integer form avoids: 0.1 * 320 is not 32 in binary64 products
    assert orc.probe_budget(320, 1000) == 32


# ----------------------------------------------------------------- top-b (Section 3.3; brute force)

def _brute_top_b(scores, b):
    keyed = sorted(range(len(scores)), key=lambda i: (-(float(scores[i]) + 0.0), i))
    return sorted(keyed[:b])


@pytest.mark.parametrize("n,b", [(1, 1), (5, 0), (17, 5), (64, 16), (100, 100), (33, 32)])
def test_top_b_brute_force_random_and_tied(n, b):
    for trial in range(20):
        s = rng.random(n)
        if trial % 2:
            s = np.round(s * 4) / 4          # heavy ties
        if trial % 5 == 0:
            s[:] = 0.0
            s[::3] = -0.0                     # signed zeros are one value
        assert list(orc.top_b(s, b)) == _brute_top_b(s, b)


def test_top_b_rejects_nan():
    with pytest.raises(ValueError):
        orc.top_b(np.array([0.1, np.nan]), 1)


def test_select_probes_structure():
    off = np.array([0, 10, 10, 35, 64])
    dk, dv = rng.random(64) * 2, rng.random(64) * 2
    p = orc.select_probes(dk, dv, off, 2500)
    bs = [3, 0, 7, 8]
    assert list(np.diff(p["probe_off"])) == bs
    for u in range(4):
        a, e = off[u], off[u + 1]
        S = p["sk_idx"][p["probe_off"][u]:p["probe_off"][u + 1]]
        assert list(S) == [a + i for i in _brute_top_b(dk[a:e], bs[u])]
        S = p["sv_idx"][p["probe_off"][u]:p["probe_off"][u + 1]]
        assert list(S) == [a + i for i in _brute_top_b(dv[a:e], bs[u])]
    assert np.array_equal(p["w_k"], np.where(dk < 1, dk, 1.0))
    assert list(p["ctx_rows"]) == sorted(set(p["sk_idx"]) | set(p["sv_idx"]))


# ----------------------------------------------------------------- scores (Section 3.3)

def test_divergence_score_closed_form():
    fresh = np.zeros((3, 2, 4))
    reuse = np.zeros((3, 2, 4))
    fresh[0, 0, 0], fresh[0, 1, 3] = 3.0, 4.0           # norm over BOTH heads: 5
    reuse[1] = 1.0                                      # sqrt(8)
    d = orc.divergence_scores(fresh, reuse)
    assert d[0] == 5.0 and abs(d[1] - math.sqrt(8)) < 1e-15 and d[2] == 0.0


# ----------------------------------------------------------------- mean estimation (closed form)

def test_probe_offset_is_arithmetic_mean_small_integers():
    N, H, D = 12, 2, 4
    j = np.arange(N, dtype=np.float64)
    fresh = np.zeros((N, H, D))
    reuse = np.zeros((N, H, D))
    fresh[:] = (3 * j)[:, None, None] + np.arange(D)[None, None, :]
    reuse[:] = j[:, None, None]
    # residual_j = 2 j + dim
    s_idx = np.array([1, 4, 7, 5, 8, 11])
    poff = np.array([0, 3, 3, 6])                       # unit 1 has no probes
    for dt in (np.float64, np.float32):
        mu = orc.probe_offsets(fresh, reuse, s_idx, poff, dt)
        assert np.array_equal(mu[0, 0], 2 * (1 + 4 + 7) // 3 + np.arange(D))
        assert np.array_equal(mu[1], np.zeros((H, D)))
        assert np.array_equal(mu[2, 1], 2 * (5 + 8 + 11) // 3 + np.arange(D))


def test_correction_closed_form_and_equivariance():
    N, H, D = 10, 1, 3
    ctx_off = np.array([0, 4, 10])
    reuse = rng.standard_normal((N, H, D))
    fresh = rng.standard_normal((N, H, D))
    w = rng.random(N)
    mu = rng.standard_normal((2, H, D))
    S = np.array([1, 6, 9])
    out = orc.apply_correction(fresh, reuse, S, w, mu, ctx_off)
    for jj in range(N):
        u = 0 if jj < 4 else 1
        want = fresh[jj] if jj in S else reuse[jj] + w[jj] * mu[u]
        assert np.allclose(out[jj], want, rtol=0, atol=1e-15)
    # add a constant c to unit 1's cache with probes, weights and FRESH values fixed: the
    # offset moves by -c, so non-probes move by (1 - w_j) c and probes do not move
    c = rng.standard_normal((H, D))
    poff = np.array([0, 1, 3])
    reuse2 = reuse.copy()
    reuse2[4:] += c
    mu_a = orc.probe_offsets(fresh, reuse, S, poff)
    mu_b = orc.probe_offsets(fresh, reuse2, S, poff)
    assert np.allclose(mu_b[1], mu_a[1] - c)
    a = orc.apply_correction(fresh, reuse, S, w, mu_a, ctx_off)
    b = orc.apply_correction(fresh, reuse2, S, w, mu_b, ctx_off)
    for jj in range(4, N):
        want = 0 if jj in S else (1 - w[jj]) * c
        assert np.allclose(b[jj] - a[jj], want, atol=1e-14)
    assert np.array_equal(a[:4], b[:4])


def test_prop2_residual_identity():
    """Proposition 2 set-up: residuals r_i = mu + xi_i, correction with w = 1 applied to
    every token gives k* - k_corr = xi_i - (mu_hat - mu)."""
    n, D = 40, 8
    mu = rng.standard_normal(D)
    xi = 0.1 * rng.standard_normal((n, 1, D))
    reuse = rng.standard_normal((n, 1, D))
    fresh = reuse + mu[None, None, :] + xi
    S = np.sort(rng.choice(n, 7, replace=False))
    mu_hat = orc.probe_offsets(fresh, reuse, S, np.array([0, 7]))
    corr = orc.apply_correction(fresh, reuse, np.zeros(0, np.int64), np.ones(n), mu_hat, np.array([0, n]))
    e = mu_hat[0, 0] - mu
    assert np.allclose(fresh - corr, xi - e[None, None, :], atol=1e-13)
    assert np.allclose(e, xi[S].mean(axis=0)[0], atol=1e-13)


def test_probe_mean_error_scales_as_inverse_sqrt_b():
    """Appendix C.2: with Gaussian fluctuations and probes drawn with replacement the
    probe-mean error decays like b^(-1/2)."""
    g = np.random.default_rng(11)
    n, D = 512, 16
    reuse = np.zeros((n, 1, D))
    fresh = g.standard_normal((n, 1, D)) + 3.0
    rbar = fresh.mean(axis=0)[0]
    bs = [4, 16, 64, 256]
    errs = []
    for b in bs:
        e = []
        for _ in range(200):
            S = g.integers(0, n, b)
            mu = orc.probe_offsets(fresh, reuse, S, np.array([0, b]))[0, 0]
            e.append(np.linalg.norm(mu - rbar))
        errs.append(np.mean(e))
    slope = np.polyfit(np.log(bs), np.log(errs), 1)[0]
    assert abs(slope + 0.5) < 0.1, slope


# ----------------------------------------------------------------- attention

def _brute_attention(q, k, v, qpos, kpos, klo=None):
    R, nq, hd = q.shape
    g = nq // k.shape[1]
    out = np.zeros_like(q)
    for r in range(R):
        for h in range(nq):
            js = [j for j in range(len(k)) if kpos[j] <= qpos[r] and (klo is None or kpos[j] >= klo[r])]
            z = [sum(q[r, h, i] * k[j, h // g, i] for i in range(hd)) / math.sqrt(hd) for j in js]
            m = max(z)
            e = [math.exp(t - m) for t in z]
            s = sum(e)
            for i in range(hd):
                out[r, h, i] = sum(e[t] / s * v[j, h // g, i] for t, j in enumerate(js))
    return out


def test_attention_brute_force_gqa_sparse_rows():
    T, nq, nkv, hd = 23, 4, 2, 8
    k = rng.standard_normal((T, nkv, hd))
    v = rng.standard_normal((T, nkv, hd))
    rows = np.array([0, 3, 4, 11, 22])
    q = rng.standard_normal((len(rows), nq, hd))
    a = orc.attention(q, k, v, rows, np.arange(T))
    assert np.allclose(a, _brute_attention(q, k, v, rows, np.arange(T)), atol=1e-12)
    lo = np.array([0, 2, 2, 9, 20])
    a = orc.attention(q, k, v, rows, np.arange(T), lo)
    assert np.allclose(a, _brute_attention(q, k, v, rows, np.arange(T), lo), atol=1e-12)


def test_attention_gqa_equals_mha_with_replicated_kv():
    T, nq, nkv, hd = 16, 6, 2, 4
    q = rng.standard_normal((T, nq, hd))
    k = rng.standard_normal((T, nkv, hd))
    v = rng.standard_normal((T, nkv, hd))
    a = orc.attention(q, k, v, np.arange(T), np.arange(T))
    b = orc.attention(q, np.repeat(k, 3, axis=1), np.repeat(v, 3, axis=1), np.arange(T), np.arange(T))
    assert np.allclose(a, b, atol=1e-14)


def test_lemma1_attention_perturbation_bound():
    """Lemma 1: ||y - y*|| <= C ||q|| Vmax / sqrt(d) * max||dk|| + max||dv|| holds for any
    perturbation; the proof's constant is C = 1/2, the statement prints C = 1."""
    for trial in range(50):
        n, d = int(rng.integers(2, 40)), int(rng.choice([4, 16, 64]))
        q = rng.standard_normal((1, 1, d)) * rng.uniform(0.1, 3)
        k = rng.standard_normal((n, 1, d))
        v = rng.standard_normal((n, 1, d))
        dk = rng.standard_normal((n, 1, d)) * rng.uniform(0, 2)
        dv = rng.standard_normal((n, 1, d)) * rng.uniform(0, 2)
        pos = np.zeros(n, int)
        y0 = orc.attention(q, k, v, [0], pos)[0, 0]
        y1 = orc.attention(q, k + dk, v + dv, [0], pos)[0, 0]
        vmax = np.linalg.norm(v, axis=-1).max()
        mk = np.linalg.norm(dk, axis=-1).max()
        mv = np.linalg.norm(dv, axis=-1).max()
        lhs = np.linalg.norm(y1 - y0)
        tight = vmax * np.linalg.norm(q) / (2 * math.sqrt(d)) * mk + mv
        assert lhs <= tight * (1 + 1e-12)


# ----------------------------------------------------------------- RoPE

def test_rope_is_complex_rotation_and_relative():
    n, H, hd, base = 9, 2, 8, 1e4
    x = rng.standard_normal((n, H, hd))
    pos = np.array([0, 1, 2, 5, 17, 100, 1000, 4095, 12000])
    y = orc.rope_rotate(x, pos, base)
    theta = base ** (-2.0 * np.arange(hd // 2) / hd)
    z = (x[..., :hd // 2] + 1j * x[..., hd // 2:]) * np.exp(1j * pos[:, None, None] * theta[None, None, :])
    assert np.allclose(y[..., :hd // 2], z.real, atol=1e-12) and np.allclose(y[..., hd // 2:], z.imag, atol=1e-12)
    assert np.array_equal(orc.rope_rotate(x, np.zeros(n), base), x)          # Rot(0) = I exactly
    # composition: Rot(a) Rot(b) = Rot(a + b); inverse: Rot(-a) Rot(a) = I
    a = orc.rope_rotate(orc.rope_rotate(x, pos, base), np.full(n, 33), base)
    assert np.allclose(a, orc.rope_rotate(x, pos + 33, base), atol=1e-11)
    assert np.allclose(orc.rope_rotate(y, -pos, base), x, atol=1e-11)
    # the inner product depends on the position difference only
    q = rng.standard_normal((1, 1, hd))
    kk = rng.standard_normal((1, 1, hd))
    d1 = (orc.rope_rotate(q, [50], base) * orc.rope_rotate(kk, [43], base)).sum()
    d2 = (orc.rope_rotate(q, [7], base) * orc.rope_rotate(kk, [0], base)).sum()
    assert abs(d1 - d2) < 1e-12


# ----------------------------------------------------------------- quantiser

@pytest.mark.parametrize("bits", [2, 4])
def test_quantiser_error_bound_and_exact_cases(bits):
    levels = (1 << bits) - 1
    x = (rng.standard_normal((5, 3, 128)) * 2).astype(np.float32)
    codes, s16, m16 = orc.quantize_groups(x, bits)
    assert codes.max() <= levels and codes.shape == x.shape and s16.shape == (5, 3, 2)
    y = orc.dequantize_groups(codes, s16, m16)
    s = s16.astype(np.float64).repeat(64, axis=-1).reshape(x.shape)
    # half a step, plus what rounding scale and minimum to float16 can add over the range
    slack = levels * np.abs(s) * 2.0 ** -11 + np.abs(m16.astype(np.float64)).repeat(64, -1).reshape(x.shape) * 2.0 ** -11
    assert np.all(np.abs(y.astype(np.float64) - x) <= s / 2 + slack + 1e-6)
    # a constant group is reproduced exactly when the constant is a float16
    c = np.full((1, 1, 64), 0.375, np.float32)
    cc, cs, cm = orc.quantize_groups(c, bits)
    assert cs[0, 0, 0] == 0 and np.all(cc == 0) and np.array_equal(orc.dequantize_groups(cc, cs, cm), c)
    # values on a float16-exact grid round-trip exactly
    grid = (0.5 + 0.25 * (np.arange(64) % (levels + 1))).astype(np.float32).reshape(1, 1, 64)
    gc, gs, gm = orc.quantize_groups(grid, bits)
    assert np.array_equal(gc[0, 0], np.arange(64) % (levels + 1))
    assert np.array_equal(orc.dequantize_groups(gc, gs, gm), grid)


def test_quantiser_round_half_even_and_packing():
    # min 0, max 3 with 2 bits: scale 1; 0.5 -> 0, 1.5 -> 2, 2.5 -> 2
    x = np.zeros((1, 64), np.float32)
    x[0, :5] = [0.0, 3.0, 0.5, 1.5, 2.5]
    codes, s16, m16 = orc.quantize_groups(x, 2)
    assert list(codes[0, :5]) == [0, 3, 0, 2, 2]
    packed = orc.pack_codes(codes, 2)
    assert packed.shape == (1, 16) and packed[0, 0] == (0 | 3 << 2 | 0 << 4 | 2 << 6) and packed[0, 1] == 2
    c4 = (np.arange(64) % 16).astype(np.uint8).reshape(1, 64)
    p4 = orc.pack_codes(c4, 4)
    assert p4.shape == (1, 32) and p4[0, 0] == (0 | 1 << 4) and p4[0, 7] == (14 | 15 << 4)


# ----------------------------------------------------------------------------- FP8 (E4M3) cache

def test_e4m3_every_code_round_trips():
    """All 254 finite bit patterns decode to a value that encodes back to the same pattern
    (brute force over the whole format); the decoded table has the format's landmarks."""
    codes = np.array([c for c in range(256) if c & 0x7f != 0x7f], np.uint8)
    vals = orc.e4m3_decode(codes)
    assert np.array_equal(orc.e4m3_encode(vals), codes)
    assert vals.max() == 448.0 and vals.min() == -448.0
    pos = np.sort(vals[vals > 0])
    assert pos[0] == 2.0 ** -9 and pos[7] == 2.0 ** -6          # smallest subnormal, smallest normal
    assert orc.e4m3_decode(np.uint8(0x38)) == 1.0 and orc.e4m3_decode(np.uint8(0x40)) == 2.0


def test_e4m3_rounding_rules():
    """Ties go to the even mantissa, everything else to the nearest value, magnitudes above
    448 saturate (hand-computed cases: between 1 and 2 the grid step is 1/8)."""
    enc = lambda x: float(orc.e4m3_decode(orc.e4m3_encode(np.float32(x))))
    assert enc(1.0625) == 1.0            # tie between 1.0 (mantissa 0) and 1.125 (mantissa 1)
    assert enc(1.1875) == 1.25           # tie between 1.125 (1) and 1.25 (2)
    assert enc(1.07) == 1.125 and enc(1.05) == 1.0
    assert enc(1.96) == 2.0              # rounds up into the next binade
    assert enc(447.0) == 448.0 and enc(1.0e6) == 448.0 and enc(-3.0e4) == -448.0
    assert enc(2.0 ** -10) == 0.0        # tie between 0 and the smallest subnormal 2^-9: even is 0
    assert enc(3 * 2.0 ** -10) == 2.0 ** -8   # tie between 1 and 2 subnormal steps: even is 2
    assert enc(0.0) == 0.0 and orc.e4m3_encode(np.float32(-0.0)) == 0x80


def test_e4m3_matches_the_library_cast_and_is_monotone():
    """Against torch's CPU float8_e4m3fn conversion (an independent implementation) on random
    values inside the finite range, plus monotonicity and idempotence."""
    import torch
    g = np.random.default_rng(5)
    x = np.concatenate([g.normal(0, 3, 20000), g.normal(0, 0.01, 5000), g.uniform(-448, 448, 5000)]).astype(np.float32)
    ours = orc.e4m3_decode(orc.e4m3_encode(x))
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(ours, lib)
    xs = np.sort(x)
    assert np.all(np.diff(orc.e4m3_decode(orc.e4m3_encode(xs))) >= 0)
    assert np.array_equal(orc.e4m3_encode(ours), orc.e4m3_encode(x))
    assert np.all(np.abs(ours - x) <= np.maximum(np.abs(x) / 16, 2.0 ** -10))   # half a step of 3 mantissa bits


# ----------------------------------------------------------------------------- residual diagnostics

def test_residual_stats_closed_forms():
    """(i) subtracting the exact mean leaves total - n |mean|^2 (the variance identity);
    (ii) a residual that IS a per-unit constant is removed entirely; (iii) no correction
    leaves everything; (iv) the selection weights form a weighted mean (hand-computed)."""
    g = np.random.default_rng(3)
    off = np.array([0, 5, 5, 12])                            # the middle unit is empty
    fresh, reuse = g.standard_normal((12, 2, 4)), g.standard_normal((12, 2, 4))
    mean, total, rem0 = orc.residual_stats(fresh, reuse, off)
    assert np.allclose(rem0, total) and total[1] == 0 and np.all(mean[1] == 0)
    _, _, rem = orc.residual_stats(fresh, reuse, off, mu=mean)
    n = np.diff(off)
    assert np.allclose(rem, total - n * (mean ** 2).sum(axis=1))
    const = np.repeat(g.standard_normal((3, 8)), n, axis=0).reshape(12, 2, 4)
    m2, t2, _ = orc.residual_stats(reuse + const, reuse, off)
    _, _, r2 = orc.residual_stats(reuse + const, reuse, off, mu=m2)
    assert np.allclose(r2, 0, atol=1e-20) and np.allclose(t2, n * (m2 ** 2).sum(axis=1))
    # weighted mean by hand: unit 0, weights 2,0,1,0,0 -> (2 r0 + r2) / 3
    sel = np.zeros(12)
    sel[[0, 2]] = [2, 1]
    m3, _, _ = orc.residual_stats(fresh, reuse, off, sel=sel)
    r = (fresh - reuse).reshape(12, 8)
    assert np.allclose(m3[0], (2 * r[0] + r[2]) / 3) and np.all(m3[2] == 0)
    # per-token weights scale the subtracted vector
    w = g.random(12)
    _, _, r4 = orc.residual_stats(fresh, reuse, off, mu=mean, w=w)
    assert np.isclose(r4[2], sum(((r[i] - w[i] * mean[2]) ** 2).sum() for i in range(5, 12)))
