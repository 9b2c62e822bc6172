"""End-to-end parity of the four modes against the oracle, through the C ABI.

Tolerances are the benchmark spec's: max relative L2 error 2e-3 for the float model, 1e-2 for
bf16 models, over the final hidden states and over every layer's K and V.  Probe indices
are compared bit-exactly: (i) the selection function on identical scores (test_gpu_ops),
(ii) end to end on the float configuration where the score gap at the cut is resolvable.
The prefill itself is always run with the oracle's probe sets on both sides."""
import ctypes as C

import numpy as np
import pytest
import torch

import testgen
from oracle import akvs_oracle as orc
from gpu_helpers import Case, t2n, max_layer_err, both_16bit

pytestmark = pytest.mark.gpu

def small16(dtype):
    return testgen.Workload("small16-" + dtype, testgen.ModelCfg("small16", 3, 256, 4, 2, 128, 768, 512, dtype),
                            5, 40, 90, 24, (2500,))


# weight scale per 16-bit type: at x4 the softmax is sharp enough that bf16 activation rounding
# alone (about 1.4e-2 after three layers) breaks the 1e-2 bound; float16 stays near 2e-3
SMALL16 = [("bf16", 1.0), ("f16", 4.0)]
F32_HD128 = testgen.Workload(
    "f32-hd128", testgen.ModelCfg("f32-hd128", 3, 128, 2, 1, 128, 200, 300, "f32"), 4, 5, 37, 9, (2500,))


def _check_encode(case, tol):
    case.encode()
    units = case.oracle_units()
    k = np.concatenate([u["K"] for u in units], axis=1)
    v = np.concatenate([u["V"] for u in units], axis=1)
    if case.kv_format == 0:
        assert max_layer_err(t2n(case.store.k), k) < tol and max_layer_err(t2n(case.store.v), v) < tol
    return units


def _run_all_modes(case, bp, check_layer, units):
    tol = case.tol
    o_units = list(case.order)
    # full recompute
    full = orc.full_recompute(case.omodel, case.ctx, case.qry)
    hid, k, v = case.gpu_prefill(case.akvs.MODE_FULL)
    assert orc.rel_l2(hid, full[0]) < tol and max_layer_err(k, full[1]) < tol and max_layer_err(v, full[2]) < tol
    # both sides read the same cache from here on
    case.load_oracle_cache(units)
    naive = orc.naive_reuse(case.omodel, units, o_units, case.qry)
    hid, k, v = case.gpu_prefill(case.akvs.MODE_NAIVE)
    assert orc.rel_l2(hid, naive[0]) < tol and max_layer_err(k, naive[1]) < tol and max_layer_err(v, naive[2]) < tol
    # corrected reuse with the oracle's probes
    ref = orc.corrected_reuse(case.omodel, units, o_units, case.ctx, case.qry, bp, check_layer)
    probes, ctx, ws = case.gpu_select(bp, check_layer)
    n_first = int(ref["ctx_off"][1])
    far = slice(n_first, case.N)            # the first unit's scores are ~0 on both sides: compare the rest
    if check_layer > 1 or case.kv_format != 0:
        assert orc.rel_l2(t2n(probes.d_k)[far], ref["d_k"][far]) < tol
        assert orc.rel_l2(t2n(probes.d_v)[far], ref["d_v"][far]) < tol
    assert np.array_equal(probes.ctx_off.cpu().numpy()[:case.M + 1], ref["ctx_off"])
    assert np.array_equal(probes.probe_off.cpu().numpy()[:case.M + 1], ref["probes"]["probe_off"])
    case.set_probes(probes, ref["probes"])
    hid, k, v = case.gpu_prefill(case.akvs.MODE_CORRECTED, ws, probes, ctx, check_layer)
    case.akvs.free(ctx)
    assert orc.rel_l2(hid, ref["hidden"]) < tol
    assert max_layer_err(k, ref["K"]) < tol and max_layer_err(v, ref["V"]) < tol
    return ref, full


def test_config1_float_all_modes():
    case = Case(testgen.workload("c1"))
    units = _check_encode(case, case.tol)
    _run_all_modes(case, 2500, 2, units)


def test_config1_indices_end_to_end():
    """GPU-selected probes equal the oracle's wherever the score gap at the cut is resolvable."""
    case = Case(testgen.workload("c1"), std_scale=4.0)
    units = case.oracle_units()
    case.load_oracle_cache(units)
    ref = orc.corrected_reuse(case.omodel, units, case.order, case.ctx, case.qry, 2500, 2)
    probes, ctx, ws = case.gpu_select(2500, 2)
    case.akvs.free(ctx)
    poff = ref["probes"]["probe_off"]
    sk, sv = probes.sk_idx.cpu().numpy(), probes.sv_idx.cpu().numpy()
    checked = 0
    for u in range(1, case.M):                       # unit 0 has zero residual: all ties at rounding level
        a, e = int(ref["ctx_off"][u]), int(ref["ctx_off"][u + 1])
        for d, got, want in ((ref["d_k"], sk, ref["probes"]["sk_idx"]), (ref["d_v"], sv, ref["probes"]["sv_idx"])):
            s = np.sort(d[a:e])[::-1]
            b = poff[u + 1] - poff[u]
            gap = (s[b - 1] - s[b]) / s[b - 1]
            print(f"unit {u}: relative gap at the cut {gap:.2e}")
            if gap > 1e-4:
                assert np.array_equal(got[poff[u]:poff[u + 1]], want[poff[u]:poff[u + 1]])
                checked += 1
    assert checked >= 3


@pytest.mark.parametrize("check_layer", [1, 2, 3])
def test_float_hd128_check_layers_and_order(check_layer):
    case = Case(F32_HD128, std_scale=6.0, order=[2, 0, 3, 1])
    units = _check_encode(case, case.tol)
    _run_all_modes(case, 2500, check_layer, units)


@pytest.mark.parametrize("dtype,scale", SMALL16)
def test_small16_all_modes(dtype, scale):
    case = Case(small16(dtype), std_scale=scale)
    units = _check_encode(case, case.tol)
    _run_all_modes(case, 2500, 2, units)


def test_small16_bf16_storage_at_weight_scale_4_tracks_float16_by_the_roundoff_ratio():
    """The case bfloat16 storage does NOT pass at 1e-2 (sharp softmax at 4x weight scale): instead
    of leaving it out, both storage types run on identical inputs (bf16-valued weights and cache)
    and the bfloat16 error is held to the first-order bound 12 x the float16 error of the same
    tensor (unit roundoff 2^-8 against 2^-11 = 8x, times 1.5 for the spread of the rounding noise)
    and to 5e-2 absolutely; float16 meets the benchmark spec's 1e-2."""
    w = small16("f16")
    errs = {}
    ref = None
    for dtype in ("f16", "bf16"):
        case = Case(w, std_scale=4.0, gpu_dtype=dtype)
        if ref is None:
            units = [{"K": both_16bit(u["K"]), "V": both_16bit(u["V"])} for u in case.oracle_units()]
            ref = orc.corrected_reuse(case.omodel, units, list(case.order), case.ctx, case.qry, 2500, 2)
        case.load_oracle_cache(units)
        probes, ctx, ws = case.gpu_select(2500, 2)
        case.set_probes(probes, ref["probes"])
        hid, k, v = case.gpu_prefill(case.akvs.MODE_CORRECTED, ws, probes, ctx, 2)
        case.akvs.free(ctx)
        errs[dtype] = (orc.rel_l2(hid, ref["hidden"]), max_layer_err(k, ref["K"]), max_layer_err(v, ref["V"]))
    print("rel L2 (hidden, K, V): f16", errs["f16"], "bf16", errs["bf16"],
          "ratio", [b / a for a, b in zip(errs["f16"], errs["bf16"])])
    assert max(errs["f16"]) < 1e-2
    assert max(errs["bf16"]) < 5e-2
    for a, b in zip(errs["f16"], errs["bf16"]):
        assert b < 12.0 * max(a, 2e-4)


@pytest.mark.parametrize("dtype,scale", SMALL16)
def test_small16_all_modes_linear_layers_on_cta_pairs(dtype, scale):
    """The same with every tensor-core linear layer of more than 128 rows forced onto the
    CTA-pair kernel (fused RoPE, residual and SwiGLU epilogues), which the shapes of this small
    model would not pick by themselves."""
    case = Case(small16(dtype), std_scale=scale)
    case.akvs.lib.akvs_debug_set_linear_algo(2 << 2)
    try:
        units = _check_encode(case, case.tol)
        _run_all_modes(case, 2500, 2, units)
    finally:
        case.akvs.lib.akvs_debug_set_linear_algo(0)


def wide16(dtype):
    return testgen.Workload("wide16-" + dtype, testgen.ModelCfg("wide16", 4, 512, 4, 2, 128, 896, 512, dtype),
                            5, 40, 90, 24, (2500,))


@pytest.mark.parametrize("dtype,scale", SMALL16)
@pytest.mark.parametrize("switches", [0, 2 << 2, (2 << 2) | (2 << 4), 3 << 4])
def test_wide16_all_modes_tilings_and_split_k(dtype, scale, switches):
    """A four-layer model of width 512 (d_ff 896 = 14 slabs of 64): every mode against the oracle
    with the linear layers by shape, on CTA pairs, and with the residual layers' k range forced
    into 2 (on pairs) and 3 ordered partial sums."""
    case = Case(wide16(dtype), std_scale=scale)
    case.akvs.lib.akvs_debug_set_linear_algo(switches)
    try:
        units = _check_encode(case, case.tol)
        _run_all_modes(case, 2500, 2, units)
    finally:
        case.akvs.lib.akvs_debug_set_linear_algo(0)


@pytest.mark.parametrize("kv_format", [4, 2])
@pytest.mark.parametrize("dtype,scale", SMALL16)
def test_small16_quantised_cache(kv_format, dtype, scale):
    case = Case(small16(dtype), std_scale=scale, kv_format=kv_format)
    case.encode()
    units = case.oracle_units()
    # the GPU's own codes decode to values within one quantisation step of the oracle's cache
    # (its inputs are bf16, so codes may differ by one where a value sits on a rounding edge)
    a = case.akvs
    step = max(float(u["K_scale"].astype(np.float64).max()) for u in units)
    kq = np.concatenate([u["K"] for u in units], axis=1)
    codes = case.store.k.cpu().numpy()
    meta = case.store.k_meta.cpu().numpy()
    per = 8 // kv_format
    un = np.stack([(codes >> (kv_format * i)) & ((1 << kv_format) - 1) for i in range(per)], -1).reshape(kq.shape)
    deq = orc.dequantize_groups(un.astype(np.uint8), meta[..., 0], meta[..., 1])
    assert np.abs(deq - kq).max() <= 1.1 * step + 0.05
    _run_all_modes(case, 2500, 2, units)
    _run_all_modes(case, 2000, 1, units)           # check layer 1: scores are the quantisation error


@pytest.mark.parametrize("dtype,scale", SMALL16)
def test_small16_fp8_cache(dtype, scale):
    """FP8 (E4M3) cache: the library's own bytes sit within one format step of the oracle's
    (its K/V are 16-bit), then all modes with the oracle's bytes on both sides."""
    case = Case(small16(dtype), std_scale=scale, kv_format=8)
    case.encode()
    units = case.oracle_units()
    kq = np.concatenate([u["K"] for u in units], axis=1)
    got = orc.e4m3_decode(case.store.k.cpu().numpy())
    assert np.all(np.abs(got - kq) <= np.maximum(np.abs(kq) / 8, 2.0 ** -9) + 0.02 * np.abs(kq).max())
    _run_all_modes(case, 2500, 2, units)
    if dtype == "f16":
        # check layer 1: the scores ARE the FP8 rounding error (a few percent of |v|), which bf16
        # storage of the fresh rows (0.4 % of |v|) cannot resolve to 1e-2; float16 can
        _run_all_modes(case, 2000, 1, units)


def test_invariants_on_gpu():
    """100 % refresh equals full recompute; 0 % refresh equals naive reuse (GPU vs GPU)."""
    case = Case(small16("f16"), std_scale=4.0)
    case.encode()
    a = case.akvs
    full = case.gpu_prefill(a.MODE_FULL)
    probes, ctx, ws = case.gpu_select(10000, 2)
    assert probes.n_probe_rows == case.N
    corr = case.gpu_prefill(a.MODE_CORRECTED, ws, probes, ctx, 2)
    a.free(ctx)
    for x, y in zip(corr, full):
        assert orc.rel_l2(x, y) < 1e-6
    naive = case.gpu_prefill(a.MODE_NAIVE)
    probes, ctx, ws = case.gpu_select(0, 1)
    assert probes.n_probe_rows == 0 and probes.n_rows == case.nq
    corr = case.gpu_prefill(a.MODE_CORRECTED, ws, probes, ctx, 1)
    a.free(ctx)
    for x, y in zip(corr, naive):
        assert orc.rel_l2(x, y) < 1e-6


def test_first_unit_scores_are_zero_on_gpu():
    case = Case(testgen.workload("c1"), std_scale=4.0)
    case.encode()
    probes, ctx, ws = case.gpu_select(2500, 2)
    case.akvs.free(ctx)
    n0 = int(case.lens[case.order[0]])
    d = t2n(probes.d_k)
    assert d[:n0].max() < 1e-3 * d[n0:case.N].mean()


def test_argument_validation():
    case = Case(testgen.workload("c1"))
    a = case.akvs
    ws = case.workspace(2)
    probes = a.Probes(case.N, case.M, case.nq)
    ctx = C.c_void_p()
    with pytest.raises(a.AkvsError) as e:
        a.select_probes(case.gmodel, case.store, case.req, 10001, 2, probes, ctx, ws)
    assert e.value.code == -1
    with pytest.raises(a.AkvsError) as e:
        a.select_probes(case.gmodel, case.store, case.req, 2500, 3, probes, ctx, ws)     # only 2 layers
    assert e.value.code == -1
    small = a.alloc_workspace(1024)
    with pytest.raises(a.AkvsError) as e:
        a.select_probes(case.gmodel, case.store, case.req, 2500, 2, probes, ctx, small)
    assert e.value.code == -3
    hid, k, v = a.alloc_outputs(case.gmodel, case.N, case.nq)
    with pytest.raises(a.AkvsError) as e:                                              # corrected mode without ctx
        a.prefill_corrected(case.gmodel, case.store, case.req, probes, a.MODE_CORRECTED, hid, k, v, None, ws)
    assert e.value.code == -1
    bad = a.Request([0, 1, 99], case.qry)
    with pytest.raises(a.AkvsError) as e:
        a.prefill_corrected(case.gmodel, case.store, bad, None, a.MODE_NAIVE, hid, k, v, None, ws)
    assert e.value.code == -1


def test_empty_edges():
    """No query tokens; a request of one unit; zero-length unit in the store."""
    w = testgen.Workload("edge", F32_HD128.model, 3, 4, 9, 6, (2500,))
    case = Case(w, std_scale=6.0, order=[1])
    units = _check_encode(case, case.tol)
    _run_all_modes(case, 5000, 2, units)


def test_cache_streamed_in_behind_layer_events():
    """An offloaded cache copied in on a side stream, one event per layer: the library waits for
    each layer's event before it reads that layer, so the result equals the resident-cache run."""
    case = Case(small16("f16"), std_scale=4.0)
    case.encode()
    a = case.akvs
    probes, ctx, ws = case.gpu_select(2500, 2)
    want = case.gpu_prefill(a.MODE_CORRECTED, ws, probes, ctx, 2)
    a.free(ctx)
    h_k, h_v = case.store.k.cpu().pin_memory(), case.store.v.cpu().pin_memory()
    case.store.k.zero_()
    case.store.v.zero_()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    L = case.cfg.n_layers
    events = [torch.cuda.Event() for _ in range(L)]
    with torch.cuda.stream(side):
        torch.cuda._sleep(20_000_000)                      # the copies start late on purpose
        for l in range(L):
            case.store.k[l].copy_(h_k[l], non_blocking=True)
            case.store.v[l].copy_(h_v[l], non_blocking=True)
            events[l].record(side)
    case.store.set_layer_events(events)
    probes, ctx, ws = case.gpu_select(2500, 2)
    got = case.gpu_prefill(a.MODE_CORRECTED, ws, probes, ctx, 2)
    a.free(ctx)
    case.store.set_layer_events(None)
    for x, y in zip(got, want):
        assert np.array_equal(x, y)


def test_corrected_prefill_replays_from_a_cuda_graph():
    """The corrected prefill enqueues only stream work: captured once, its replay writes the same
    bits as the eager call."""
    case = Case(small16("f16"), std_scale=4.0)
    a = case.akvs
    case.encode()
    probes, ctx, ws = case.gpu_select(2500, 2)
    hid, k, v = a.alloc_outputs(case.gmodel, case.N, case.nq)
    run = lambda: a.prefill_corrected(case.gmodel, case.store, case.req, probes, a.MODE_CORRECTED, hid, k, v, ctx, ws)
    run()                                             # eager: also the warm-up the header asks for
    torch.cuda.synchronize()
    want = (hid.clone(), k.clone(), v.clone())
    for t in (hid, k, v):
        t.zero_()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            run()
    torch.cuda.synchronize()
    assert float(hid.abs().max()) == 0.0              # capture records, it does not run
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert a.check(ws) == 0
    assert torch.equal(hid, want[0]) and torch.equal(k, want[1]) and torch.equal(v, want[2])
    a.free(ctx)
