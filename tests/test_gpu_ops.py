"""Per-kernel parity of the CUDA library against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import akvs_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def akvs():
    import paper_2607_21604_b200 as a
    return a


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype) if dtype is not None else t


def n64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


EPS = {torch.float32: 2.0 ** -23, torch.bfloat16: 2.0 ** -8, torch.float16: 2.0 ** -11}   # one rounding
H16 = [torch.bfloat16, torch.float16]


# ----------------------------------------------------------------------------- linear layers

@pytest.mark.parametrize("M,N,K", [(1, 128, 64), (77, 256, 200), (128, 128, 64), (130, 384, 1024), (1357, 1024, 4096),
                                   (300, 11008, 2048), (200, 384, 200), (257, 640, 72)])
@pytest.mark.parametrize("algo", [0, 1, 2, 3])      # by shape, CUDA cores, single CTAs, CTA pairs
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_linear_16bit(akvs, M, N, K, algo, dtype):
    g = np.random.default_rng(M * 7 + N)
    x = dev(g.standard_normal((M, K)).astype(np.float32), dtype)
    w = dev((g.standard_normal((N, K)) * 0.05).astype(np.float32), dtype)
    y = akvs.op_linear(x, w, algo)
    torch.cuda.synchronize()
    ref = n64(x) @ n64(w).T
    ulp = EPS[dtype]                                 # only the output rounding remains
    assert orc.rel_l2(n64(y), ref) < 2 * ulp
    assert np.abs(n64(y) - ref).max() <= ulp * np.abs(ref).max() + 1e-5


@pytest.mark.parametrize("M,N,K", [(300, 256, 4096), (958, 2048, 11008), (130, 384, 2120), (77, 128, 136)])
@pytest.mark.parametrize("algo", [0, 2, 3])         # by shape, single CTAs, CTA pairs
@pytest.mark.parametrize("splits", [0, 1, 2, 3, 4])  # split-K: by the cost model, or forced
@pytest.mark.parametrize("dtype", H16)
def test_linear_residual_split_k(akvs, M, N, K, algo, splits, dtype):
    """h += x W^T with the k range cut into work items that add into h at the L2: every split
    count gives the plain sum (float accumulation; the ragged last 64-wide slab and a last split
    shorter than the others included)."""
    g = np.random.default_rng(M + N + K)
    x = dev(g.standard_normal((M, K)).astype(np.float32), dtype)
    w = dev((g.standard_normal((N, K)) * 0.05).astype(np.float32), dtype)
    h0 = g.standard_normal((M, N)).astype(np.float32)
    h = dev(h0)
    slabs = (K + 63) // 64
    if splits > 1 and (slabs + splits - 1) // splits * (splits - 1) >= slabs:
        with pytest.raises(akvs.AkvsError):
            akvs.op_linear_residual(x, w, h, algo, splits)
        return
    akvs.op_linear_residual(x, w, h, algo, splits)
    again = dev(h0)
    akvs.op_linear_residual(x, w, again, algo, splits)
    torch.cuda.synchronize()
    assert torch.equal(h, again)                     # partial sums arrive in a fixed order
    ref = h0.astype(np.float64) + n64(x) @ n64(w).T
    assert np.abs(n64(h) - ref).max() <= 1e-5 * np.abs(ref).max() * max(1.0, np.sqrt(K / 1024))


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (65, 130, 33), (200, 688, 256)])
def test_linear_f32(akvs, M, N, K):
    g = np.random.default_rng(M)
    x = dev(g.standard_normal((M, K)).astype(np.float32))
    w = dev(g.standard_normal((N, K)).astype(np.float32))
    y = akvs.op_linear(x, w)
    torch.cuda.synchronize()
    assert orc.rel_l2(n64(y), n64(x) @ n64(w).T) < 1e-6


@pytest.mark.parametrize("M,N,K", [(1, 1, 1), (65, 130, 33), (200, 688, 256)])
def test_linear_residual_f32(akvs, M, N, K):
    g = np.random.default_rng(M + 1)
    x = dev(g.standard_normal((M, K)).astype(np.float32))
    w = dev(g.standard_normal((N, K)).astype(np.float32))
    h0 = g.standard_normal((M, N)).astype(np.float32)
    h = akvs.op_linear_residual(x, w, dev(h0))
    torch.cuda.synchronize()
    assert orc.rel_l2(n64(h), h0.astype(np.float64) + n64(x) @ n64(w).T) < 1e-6
    with pytest.raises(akvs.AkvsError):
        akvs.op_linear_residual(x, w, dev(h0), 0, 2)     # no split-K on the CUDA-core kernel


@pytest.mark.parametrize("algo", [2, 3])
@pytest.mark.parametrize("dtype", H16)
def test_linear_16bit_full_size_sampled(akvs, dtype, algo):
    """Config-3 MLP shape on single CTAs and on CTA pairs (the last pair's second CTA holds no
    row: M = 10 x 256 + 26); the oracle checks sampled outputs one by one."""
    g = torch.Generator(device="cuda").manual_seed(5)
    M, N, K = 2586, 4096, 14336
    x = torch.randn((M, K), generator=g, device="cuda").to(dtype)
    w = (torch.randn((N, K), generator=g, device="cuda") * 0.02).to(dtype)
    y = akvs.op_linear(x, w, algo)
    torch.cuda.synchronize()
    rs = np.random.default_rng(0)
    rows = np.concatenate([[0, 127, 128, 255, 256, 2559, 2560, M - 1], rs.integers(0, M, 60)])
    cols = np.concatenate([[0, 255, 256, N - 1], rs.integers(0, N, 60)])
    xr, wc = n64(x[rows]), n64(w[cols])
    ref = xr @ wc.T
    got = n64(y[rows][:, cols])
    assert np.abs(got - ref).max() <= EPS[dtype] * np.abs(ref).max() + 1e-4


# ----------------------------------------------------------------------------- RoPE

@pytest.mark.parametrize("dtype,hd", [(torch.float32, 64), (torch.float16, 128), (torch.bfloat16, 128),
                                      (torch.float32, 128)])
def test_rope(akvs, dtype, hd):
    g = np.random.default_rng(1)
    n, H = 37, 3
    x = g.standard_normal((n, H, hd)).astype(np.float32)
    pos = np.concatenate([[0, 1, 12415], g.integers(0, 12416, n - 3)]).astype(np.int32)
    xt = dev(x, dtype)
    ref = orc.rope_rotate(n64(xt), pos, 1e4)
    akvs.op_rope(xt, dev(pos), 1e4)
    torch.cuda.synchronize()
    assert orc.rel_l2(n64(xt), ref) < max(1e-6, EPS[dtype])


# ----------------------------------------------------------------------------- attention

@pytest.mark.parametrize("dtype,hd,nq,nkv", [(torch.float32, 64, 4, 2), (torch.float16, 128, 8, 2),
                                             (torch.bfloat16, 128, 4, 1), (torch.float16, 128, 5, 1),
                                             (torch.bfloat16, 64, 2, 2)])
@pytest.mark.parametrize("algo", [0, 1])
def test_attention_sparse_rows_and_block_diagonal(akvs, dtype, hd, nq, nkv, algo):
    g = np.random.default_rng(2)
    T = 300
    k = dev(g.standard_normal((T, nkv, hd)).astype(np.float32), dtype)
    v = dev(g.standard_normal((T, nkv, hd)).astype(np.float32), dtype)
    rows = np.sort(g.choice(T, 45, replace=False)).astype(np.int32)
    rows[0] = 0
    q = dev(g.standard_normal((len(rows), nq, hd)).astype(np.float32), dtype)
    tol = max(1e-5, 4 * EPS[dtype])
    out = akvs.op_attention(q, k, v, dev(np.zeros_like(rows)), dev(rows), algo)
    torch.cuda.synchronize()
    ref = orc.attention(n64(q), n64(k), n64(v), rows, np.arange(T))
    assert orc.rel_l2(n64(out), ref) < tol
    # block-diagonal causal (isolated units): lower bounds are the unit starts
    starts = np.array([0, 0, 40, 40, 40, 131, 131, 299], np.int32)
    r2 = np.array([0, 39, 40, 77, 130, 131, 298, 299], np.int32)
    q2 = dev(g.standard_normal((len(r2), nq, hd)).astype(np.float32), dtype)
    out = akvs.op_attention(q2, k, v, dev(starts), dev(r2), algo)
    torch.cuda.synchronize()
    ref = orc.attention(n64(q2), n64(k), n64(v), r2, np.arange(T), starts)
    assert orc.rel_l2(n64(out), ref) < tol


@pytest.mark.parametrize("dtype", H16)
@pytest.mark.parametrize("nq,nkv", [(4, 1), (16, 2), (5, 1), (2, 2)])
def test_attention_tensor_core_many_tiles(akvs, dtype, nq, nkv):
    """Several 128-key tiles, ragged ends, sparse sorted rows with duplicates-free positions,
    then the dense causal case (every position is a row)."""
    g = np.random.default_rng(nq * 10 + nkv)
    T, hd = 1100, 128
    k = dev(g.standard_normal((T, nkv, hd)).astype(np.float32), dtype)
    v = dev(g.standard_normal((T, nkv, hd)).astype(np.float32), dtype)
    rows = np.sort(g.choice(T, 203, replace=False)).astype(np.int32)
    rows[-1] = T - 1
    q = dev((g.standard_normal((len(rows), nq, hd)) * 1.5).astype(np.float32), dtype)
    out = akvs.op_attention(q, k, v, dev(np.zeros_like(rows)), dev(rows), 0)
    torch.cuda.synchronize()
    ref = orc.attention(n64(q), n64(k), n64(v), rows, np.arange(T))
    per_row = np.linalg.norm((n64(out) - ref).reshape(len(rows), -1), axis=1) / np.linalg.norm(ref.reshape(len(rows), -1), axis=1)
    assert per_row.max() < 8 * EPS[dtype], (per_row.argmax(), per_row.max())
    allr = np.arange(T, dtype=np.int32)
    qa = dev(g.standard_normal((T, nq, hd)).astype(np.float32), dtype)
    out = akvs.op_attention(qa, k, v, dev(np.zeros_like(allr)), dev(allr), 0)
    torch.cuda.synchronize()
    ref = orc.attention(n64(qa), n64(k), n64(v), allr, allr)
    per_row = np.linalg.norm((n64(out) - ref).reshape(T, -1), axis=1) / np.linalg.norm(ref.reshape(T, -1), axis=1)
    assert per_row.max() < 8 * EPS[dtype], (per_row.argmax(), per_row.max())
    # the CUDA-core kernel agrees with it too
    out1 = akvs.op_attention(qa, k, v, dev(np.zeros_like(allr)), dev(allr), 1)
    torch.cuda.synchronize()
    assert orc.rel_l2(n64(out), n64(out1)) < 4 * EPS[dtype]


@pytest.mark.parametrize("dtype", H16)
@pytest.mark.parametrize("shape", ["rising", "falling", "spiky"])
def test_attention_tensor_core_moving_maximum(akvs, dtype, shape):
    """Scores whose maximum moves by far more than 2^8 between key tiles: the shared reference
    maximum is raised again and again (the output accumulator is rescaled in tensor memory), stays
    put while later tiles fall far below it, or jumps on single keys."""
    g = np.random.default_rng(17)
    T, hd, nq, nkv = 1500, 128, 8, 2
    kk = g.standard_normal((T, nkv, hd)).astype(np.float32)
    ramp = np.linspace(0.05, 6.0, T, dtype=np.float32)
    if shape == "rising":
        kk *= ramp[:, None, None]
    elif shape == "falling":
        kk *= ramp[::-1, None, None]
    else:
        kk *= 0.2
        kk[g.choice(T, 25, replace=False)] *= 40.0
    k, v = dev(kk, dtype), dev(g.standard_normal((T, nkv, hd)).astype(np.float32), dtype)
    rows = np.sort(g.choice(T, 150, replace=False)).astype(np.int32)
    rows[-1] = T - 1
    q = dev((g.standard_normal((len(rows), nq, hd)) * 2.0).astype(np.float32), dtype)
    out = akvs.op_attention(q, k, v, dev(np.zeros_like(rows)), dev(rows), 0)
    torch.cuda.synchronize()
    ref = orc.attention(n64(q), n64(k), n64(v), rows, np.arange(T))
    per_row = np.linalg.norm((n64(out) - ref).reshape(len(rows), -1), axis=1) / np.linalg.norm(ref.reshape(len(rows), -1), axis=1)
    assert per_row.max() < 8 * EPS[dtype], (per_row.argmax(), per_row.max())
    assert torch.isfinite(out.float()).all()


# ----------------------------------------------------------------------------- selection (bit-exact)

def _check_select(akvs, dk, dv, off, nq, bp):
    p = akvs.op_select(dev(dk), dev(dv), off, nq, bp)
    ref = orc.select_probes(dk.astype(np.float64), dv.astype(np.float64), off, bp)
    nP = int(ref["probe_off"][-1])
    assert np.array_equal(p.probe_off.cpu().numpy()[:len(off)], ref["probe_off"])
    assert np.array_equal(p.sk_idx.cpu().numpy()[:nP], ref["sk_idx"])
    assert np.array_equal(p.sv_idx.cpu().numpy()[:nP], ref["sv_idx"])
    rows = np.concatenate([ref["ctx_rows"], np.arange(off[-1], off[-1] + nq)])
    assert p.n_probe_rows == len(ref["ctx_rows"]) and p.n_rows == len(rows) and p.n_ctx == off[-1]
    assert np.array_equal(p.rows.cpu().numpy()[:len(rows)], rows)
    assert np.array_equal(p.w_k.cpu().numpy()[:off[-1]], np.minimum(dk, 1).astype(np.float32))
    assert np.array_equal(p.w_v.cpu().numpy()[:off[-1]], np.minimum(dv, 1).astype(np.float32))


@pytest.mark.parametrize("bp", [0, 1000, 1500, 2500, 10000])
def test_select_bit_exact(akvs, bp):
    g = np.random.default_rng(bp + 1)
    lens = np.concatenate([g.integers(128, 385, 30), [1, 0, 2, 1500, 2500]])
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    N = int(off[-1])
    dk = (g.random(N) * 3).astype(np.float32)
    dv = (g.random(N) * 3).astype(np.float32)
    _check_select(akvs, dk, dv, off, 17, bp)
    # heavy ties, zeros and negative zeros
    dk = (np.round(g.random(N) * 4) / 4).astype(np.float32)
    dv = np.zeros(N, np.float32)
    dv[::3] = -0.0
    _check_select(akvs, dk, dv, off, 0, bp)


def test_select_nan_is_reported(akvs):
    dk = np.ones(64, np.float32)
    dk[5] = np.nan
    with pytest.raises(akvs.AkvsError) as e:
        akvs.op_select(dev(dk), dev(np.ones(64, np.float32)), np.array([0, 64]), 4, 2500)
    assert e.value.code == -7


# ----------------------------------------------------------------------------- quantiser (bit-exact)

@pytest.mark.parametrize("bits", [2, 4])
@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
def test_quantize_bit_exact(akvs, bits, dtype):
    g = np.random.default_rng(bits)
    x = g.standard_normal((203, 2, 128)).astype(np.float32) * 3
    x[0, 0, :64] = 0.375                                   # constant group
    x[1, 0, :64] = np.arange(64) % 4 * 0.25                # values on the grid
    xt = dev(x, dtype)
    codes, meta = akvs.op_quantize(xt, bits)
    torch.cuda.synchronize()
    rc, rs, rm = orc.quantize_groups(xt.float().cpu().numpy(), bits)
    assert np.array_equal(codes.cpu().numpy(), orc.pack_codes(rc, bits))
    m = meta.cpu().numpy()
    assert np.array_equal(m[..., 0].view(np.uint16), rs.view(np.uint16))
    assert np.array_equal(m[..., 1].view(np.uint16), rm.view(np.uint16))


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
def test_fp8_cast_bit_exact(akvs, dtype):
    """FP8 (E4M3) cache bytes equal the oracle's cast of the same stored values: random data,
    ties, subnormals, saturation, signed zero."""
    g = np.random.default_rng(8)
    x = g.standard_normal((77, 2, 128)).astype(np.float32) * 3
    x[0, 0, :16] = [1.0625, 1.1875, 1.07, 1.96, 447.0, 6e4, -3e4, 2.0 ** -10, 3 * 2.0 ** -10, 0.0, -0.0, 2.0 ** -9,
                    -2.0 ** -6, 448.0, 0.0009, -0.0021]
    x[1] *= 0.004                                          # subnormal range of the format
    x[2] *= 100                                            # saturating range
    xt = dev(x, dtype)
    codes, meta = akvs.op_quantize(xt, 8)
    torch.cuda.synchronize()
    assert meta is None
    assert np.array_equal(codes.cpu().numpy(), orc.e4m3_encode(xt.float().cpu().numpy()))


# ----------------------------------------------------------------------------- offsets + correction

def _correct_case(akvs, dtype_t, kv_format, N_units, len_lo, len_hi, nkv, hd, nq, bp, seed=0):
    g = np.random.default_rng(seed)
    lens = g.integers(len_lo, len_hi + 1, N_units)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    N = int(off[-1])
    T = N + nq
    # a store that holds the units in another order than the request uses them
    perm = g.permutation(N_units)
    store_off = np.concatenate([[0], np.cumsum(lens[perm])])
    slot_of = np.empty(N_units, np.int64)
    slot_of[perm] = np.arange(N_units)
    src = np.concatenate([store_off[slot_of[u]] + np.arange(lens[u]) for u in range(N_units)]).astype(np.int32)
    ck = g.standard_normal((N, nkv, hd)).astype(np.float32)
    cv = g.standard_normal((N, nkv, hd)).astype(np.float32)
    dk = (g.random(N) * 2).astype(np.float32)
    dv = (g.random(N) * 2).astype(np.float32)
    probes = akvs.op_select(dev(dk), dev(dv), off, nq, bp)
    ref_p = orc.select_probes(dk.astype(np.float64), dv.astype(np.float64), off, bp)
    R = probes.n_rows
    fk = g.standard_normal((R, nkv, hd)).astype(np.float32)
    fv = g.standard_normal((R, nkv, hd)).astype(np.float32)
    dt = {torch.float32: akvs.F32, torch.bfloat16: akvs.BF16, torch.float16: akvs.F16}[dtype_t]
    fk_t, fv_t = dev(fk, dtype_t), dev(fv, dtype_t)
    if kv_format == 0:
        ck_t, cv_t = dev(ck, dtype_t), dev(cv, dtype_t)
        ck_ref, cv_ref = n64(ck_t), n64(cv_t)
        km = vm = None
    elif kv_format == 8:
        kc, vc = orc.e4m3_encode(ck), orc.e4m3_encode(cv)
        ck_t, cv_t = dev(kc), dev(vc)
        km = vm = None
        ck_ref, cv_ref = orc.e4m3_decode(kc), orc.e4m3_decode(vc)
    else:
        kc, ks, kmn = orc.quantize_groups(ck, kv_format)
        vc, vs, vmn = orc.quantize_groups(cv, kv_format)
        ck_t, cv_t = dev(orc.pack_codes(kc, kv_format)), dev(orc.pack_codes(vc, kv_format))
        km, vm = dev(np.stack([ks, kmn], -1)), dev(np.stack([vs, vmn], -1))
        ck_ref = orc.dequantize_groups(kc, ks, kmn).astype(np.float64)
        cv_ref = orc.dequantize_groups(vc, vs, vmn).astype(np.float64)
    # the GPU reads store rows through src; lay the store out accordingly
    inv = np.empty(N, np.int64)
    inv[src] = np.arange(N)
    st_k, st_v = ck_t[dev(inv)].contiguous(), cv_t[dev(inv)].contiguous()
    st_km = km[dev(inv)].contiguous() if km is not None else None
    st_vm = vm[dev(inv)].contiguous() if vm is not None else None
    out_k, out_v, mu_k, mu_v = akvs.op_correct_layer(dt, kv_format, st_k, st_v, st_km, st_vm, dev(src), fk_t, fv_t,
                                                     probes, N_units, nq, nkv, hd, 1e4)
    torch.cuda.synchronize()
    # oracle: reuse = re-aligned cache; fresh indexed by global position
    P = len(ref_p["ctx_rows"])
    kr = np.concatenate([orc.rope_rotate(ck_ref[off[u]:off[u + 1]], np.full(lens[u], off[u]), 1e4)
                         for u in range(N_units)]) if N else ck_ref
    k_f = np.zeros((N, nkv, hd))
    v_f = np.zeros((N, nkv, hd))
    k_f[ref_p["ctx_rows"]] = n64(fk_t)[:P]
    v_f[ref_p["ctx_rows"]] = n64(fv_t)[:P]
    rmu_k = orc.probe_offsets(k_f, kr, ref_p["sk_idx"], ref_p["probe_off"])
    rmu_v = orc.probe_offsets(v_f, cv_ref, ref_p["sv_idx"], ref_p["probe_off"])
    rk = np.concatenate([orc.apply_correction(k_f, kr, ref_p["sk_idx"], ref_p["w_k"], rmu_k, off), n64(fk_t)[P:]])
    rv = np.concatenate([orc.apply_correction(v_f, cv_ref, ref_p["sv_idx"], ref_p["w_v"], rmu_v, off), n64(fv_t)[P:]])
    tol = max(2e-6, EPS[dtype_t])
    assert orc.rel_l2(n64(mu_k).reshape(rmu_k.shape), rmu_k) < 2e-6 * (1 if dtype_t == torch.float32 else 10)
    assert orc.rel_l2(n64(mu_v).reshape(rmu_v.shape), rmu_v) < 2e-6 * (1 if dtype_t == torch.float32 else 10)
    assert orc.rel_l2(n64(out_k), rk) < tol and orc.rel_l2(n64(out_v), rv) < tol
    # probe rows and query rows are copies: exact
    pk = ref_p["sk_idx"]
    assert np.array_equal(n64(out_k)[pk], k_f[pk])
    assert np.array_equal(n64(out_k)[N:], n64(fk_t)[P:])
    return N


@pytest.mark.parametrize("dtype_t,kv_format,hd", [(torch.float32, 0, 64), (torch.float16, 0, 128),
                                                  (torch.bfloat16, 0, 128), (torch.bfloat16, 4, 64),
                                                  (torch.float16, 4, 128), (torch.float16, 2, 128),
                                                  (torch.float32, 4, 64), (torch.float32, 2, 128),
                                                  (torch.float16, 8, 128), (torch.bfloat16, 8, 64),
                                                  (torch.float32, 8, 64)])
def test_correct_layer_small_ragged(akvs, dtype_t, kv_format, hd):
    _correct_case(akvs, dtype_t, kv_format, 5, 3, 41, 2, hd, 7, 2500)
    _correct_case(akvs, dtype_t, kv_format, 3, 1, 2, 1, hd, 0, 0, seed=1)         # no probes, no query
    _correct_case(akvs, dtype_t, kv_format, 2, 20, 30, 2, hd, 3, 10000, seed=2)   # everything is a probe


@pytest.mark.parametrize("dtype_t,kv_format,hd,nkv", [(torch.float16, 0, 128, 20), (torch.float32, 0, 128, 9),
                                                      (torch.bfloat16, 4, 64, 35), (torch.float16, 8, 128, 17),
                                                      (torch.float16, 2, 128, 3)])
def test_correct_layer_many_kv_heads(akvs, dtype_t, kv_format, hd, nkv):
    """More kv heads than one CTA row of the correction kernel covers (16 heads of 128 in a 16-bit
    type): the heads are split over blockIdx.y and the last group is short; odd head counts."""
    _correct_case(akvs, dtype_t, kv_format, 4, 5, 23, nkv, hd, 5, 3000, seed=5)


@pytest.mark.parametrize("kv_format", [0, 4, 2, 8])
def test_correct_layer_full_size(akvs, kv_format):
    """One layer at the 8B-class shapes (8 kv heads x 128, ~8k / ~12k context tokens)."""
    if kv_format == 0:
        N = _correct_case(akvs, torch.float16, 0, 32, 128, 384, 8, 128, 128, 1500, seed=3)
    else:
        N = _correct_case(akvs, torch.float16, kv_format, 48, 256, 256, 8, 128, 128, 2000, seed=4)
    assert N > 6000


# ----------------------------------------------------------------------------- residual diagnostics

@pytest.mark.parametrize("dtype_t,kv_format,nkv,hd", [(torch.float32, 0, 2, 64), (torch.float16, 0, 8, 128),
                                                      (torch.float16, 4, 2, 128), (torch.bfloat16, 8, 2, 64)])
def test_residual_stats_op(akvs, dtype_t, kv_format, nkv, hd):
    """Unit means under selection weights and total / remaining residual energy against the oracle:
    exact mean (sel = 1), a with-replacement sample (multiplicities), weighted correction."""
    g = np.random.default_rng(11)
    lens = np.array([37, 0, 5, 64, 1])
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    N, M = int(off[-1]), len(lens)
    src = g.permutation(N).astype(np.int32)                 # store rows in another order
    ck = g.standard_normal((N, nkv, hd)).astype(np.float32)
    cv = g.standard_normal((N, nkv, hd)).astype(np.float32)
    dt = {torch.float32: akvs.F32, torch.bfloat16: akvs.BF16, torch.float16: akvs.F16}[dtype_t]
    km = vm = None
    if kv_format == 0:
        ck_t, cv_t = dev(ck, dtype_t), dev(cv, dtype_t)
        ck_ref, cv_ref = n64(ck_t), n64(cv_t)
    elif kv_format == 8:
        kc, vc = orc.e4m3_encode(ck), orc.e4m3_encode(cv)
        ck_t, cv_t = dev(kc), dev(vc)
        ck_ref, cv_ref = orc.e4m3_decode(kc), orc.e4m3_decode(vc)
    else:
        kc, ks, kmn = orc.quantize_groups(ck, kv_format)
        vc, vs, vmn = orc.quantize_groups(cv, kv_format)
        ck_t, cv_t = dev(orc.pack_codes(kc, kv_format)), dev(orc.pack_codes(vc, kv_format))
        km, vm = dev(np.stack([ks, kmn], -1)), dev(np.stack([vs, vmn], -1))
        ck_ref = orc.dequantize_groups(kc, ks, kmn).astype(np.float64)
        cv_ref = orc.dequantize_groups(vc, vs, vmn).astype(np.float64)
    inv = np.empty(N, np.int64)
    inv[src] = np.arange(N)
    st = lambda t: t[dev(inv)].contiguous() if t is not None else None
    # fresh = reuse + a unit offset + noise, so that the mean explains part of the energy
    kr = np.concatenate([orc.rope_rotate(ck_ref[off[u]:off[u + 1]], np.full(lens[u], off[u]), 1e4) for u in range(M)])
    shift = np.repeat(g.standard_normal((M, nkv, hd)), lens, axis=0)
    fk_t = dev((kr + shift + 0.5 * g.standard_normal(kr.shape)).astype(np.float32), dtype_t)
    fv_t = dev((cv_ref + 0.7 * shift + 0.5 * g.standard_normal(kr.shape)).astype(np.float32), dtype_t)
    fk, fv = n64(fk_t), n64(fv_t)
    sel = np.bincount(np.concatenate([off[u] + g.integers(0, lens[u], max(1, lens[u] // 8))
                                      for u in range(M) if lens[u] > 0]), minlength=N).astype(np.float32)
    w = g.random(N).astype(np.float32)
    args = (dt, kv_format, st(ck_t), st(cv_t), st(km), st(vm), dev(src), fk_t, fv_t, off, nkv, hd, 1e4)
    tol = 2e-5

    def check(got, ref_k, ref_v):
        mk, mv, en = got
        en = n64(en)
        assert np.allclose(n64(mk), ref_k[0], rtol=tol, atol=tol) and np.allclose(n64(mv), ref_v[0], rtol=tol, atol=tol)
        assert np.allclose(en[:, 0], ref_k[1], rtol=tol) and np.allclose(en[:, 1], ref_k[2], rtol=tol, atol=1e-6)
        assert np.allclose(en[:, 2], ref_v[1], rtol=tol) and np.allclose(en[:, 3], ref_v[2], rtol=tol, atol=1e-6)

    exact = akvs.op_residual_stats(*args)
    check(exact, orc.residual_stats(fk, kr, off), orc.residual_stats(fv, cv_ref, off))
    # subtract the exact mean the op just returned; means from a sample with replacement
    mu_k, mu_v = n64(exact[0]), n64(exact[1])
    got = akvs.op_residual_stats(*args, sel_k=dev(sel), sel_v=dev(sel), mu_k=exact[0], mu_v=exact[1])
    check(got, orc.residual_stats(fk, kr, off, sel=sel, mu=mu_k), orc.residual_stats(fv, cv_ref, off, sel=sel, mu=mu_v))
    assert np.all(n64(got[2])[:, 1] <= n64(got[2])[:, 0] + 1e-6)          # the exact mean never adds energy
    # per-token weights on the subtracted vector (the method's w = min(d, 1))
    got = akvs.op_residual_stats(*args, mu_k=exact[0], mu_v=exact[1], w_k=dev(w), w_v=dev(w))
    check(got, orc.residual_stats(fk, kr, off, mu=mu_k, w=w), orc.residual_stats(fv, cv_ref, off, mu=mu_v, w=w))
