"""Parity on benchmark configurations 2-5 at full model width.

The oracle is plain numpy, so each configuration runs at reduced depth and context (sizes
the oracle finishes in tens of seconds) plus, for the 3B-class model, at its FULL depth of
36 layers on a short context.  Full-size behaviour (the launch configuration the benchmark
times) is covered by per-kernel checks on sampled outputs and by invariants that hold at
any size.  The 16-bit configurations hold their bf16-valued weights in float16 containers:
rounding activations to bf16 between kernels alone exceeds the 1e-2 bound after about a dozen
layers, float16 storage stays near 2e-3."""
import ctypes as C

import numpy as np
import pytest
import torch

import testgen
from oracle import akvs_oracle as orc
from gpu_helpers import Case, t2n, max_layer_err
from test_gpu_pipeline import _check_encode, _run_all_modes

pytestmark = pytest.mark.gpu


def _reduced(name, n_layers, n_units, n_query=None):
    w = testgen.workload(name)
    return testgen.reduced(w, n_layers=n_layers, n_units=n_units, n_query=n_query, dtype="f16")


@pytest.mark.parametrize("name,n_layers,n_units", [("c2", 3, 4), ("c3", 3, 4), ("c4", 3, 3)])
def test_config_width_reduced_depth(name, n_layers, n_units):
    w = _reduced(name, n_layers, n_units)
    case = Case(w)
    units = _check_encode(case, case.tol)
    _run_all_modes(case, w.refresh_bp[0], 2, units)


def _run_corrected_only(case, bp, check_layer, units):
    ref = orc.corrected_reuse(case.omodel, units, list(case.order), case.ctx, case.qry, bp, check_layer)
    probes, ctx, ws = case.gpu_select(bp, check_layer)
    assert np.array_equal(probes.probe_off.cpu().numpy()[:case.M + 1], ref["probes"]["probe_off"])
    case.set_probes(probes, ref["probes"])
    hid, k, v = case.gpu_prefill(case.akvs.MODE_CORRECTED, ws, probes, ctx, check_layer)
    case.akvs.free(ctx)
    assert orc.rel_l2(hid, ref["hidden"]) < case.tol
    assert max_layer_err(k, ref["K"]) < case.tol and max_layer_err(v, ref["V"]) < case.tol


@pytest.mark.parametrize("name,n_layers,n_units,ratios", [("c2", 3, 4, (2000, 3000)), ("c4", 2, 2, (3000,))])
def test_config_other_refresh_ratios(name, n_layers, n_units, ratios):
    """Configurations 2 and 4 are specified at 10, 20 and 30 % refresh: the higher ratios on the
    corrected path (the first ratio runs in test_config_width_reduced_depth)."""
    w = _reduced(name, n_layers, n_units)
    case = Case(w)
    case.encode()
    units = case.oracle_units()
    case.load_oracle_cache(units)
    for bp in ratios:
        _run_corrected_only(case, bp, 2, units)


@pytest.mark.parametrize("name", ["c5q4", "c5q2", "c5fp8"])
def test_config5_quantised_cache(name):
    w = _reduced(name, 3, 4)
    fmt = {"c5q4": 4, "c5q2": 2, "c5fp8": 8}[name]
    case = Case(w, kv_format=fmt)
    case.encode()
    units = case.oracle_units()
    _run_all_modes(case, w.refresh_bp[0], 2, units)


def test_config2_full_depth_short_context():
    """All 36 layers of the 3B-class model: the error stays inside 1e-2 at full depth."""
    w = testgen.reduced(testgen.workload("c2"), n_units=2, len_lo=90, len_hi=130, n_query=32, dtype="f16")
    case = Case(w)
    units = _check_encode(case, case.tol)
    _run_all_modes(case, 2000, 2, units)


def test_attention_full_size_sampled_rows():
    """Config-3 launch shape of one selective layer: 32 q / 8 kv heads, ~2.3k sparse rows over
    ~8.7k keys; the oracle recomputes sampled rows one by one."""
    import paper_2607_21604_b200 as akvs
    g = np.random.default_rng(9)
    T, nq, nkv, hd = 8721, 32, 8, 128
    dev = lambda a: torch.from_numpy(a).cuda()
    k = (torch.randn((T, nkv, hd), device="cuda") * 1.3).half()
    v = torch.randn((T, nkv, hd), device="cuda").half()
    rows = np.sort(g.choice(T - 128, 2150, replace=False)).astype(np.int32)
    rows = np.concatenate([rows, np.arange(T - 128, T, dtype=np.int32)])
    q = (torch.randn((len(rows), nq, hd), device="cuda") * 1.3).half()
    out = akvs.op_attention(q, k, v, dev(np.zeros_like(rows)), dev(rows), 0)
    torch.cuda.synchronize()
    pick = np.concatenate([[0, 1, 31, 32, len(rows) - 1], g.integers(0, len(rows), 20)])
    kn, vn = t2n(k), t2n(v)
    for r in pick:
        ref = orc.attention(t2n(q[r:r + 1]), kn[:rows[r] + 1], vn[:rows[r] + 1], [rows[r]], np.arange(rows[r] + 1))
        assert orc.rel_l2(t2n(out[r:r + 1]), ref) < 2e-3, r


def test_config3_full_size_invariants():
    """The benchmark's configuration (32 layers, ~8.7k tokens): 0 % refresh equals naive reuse,
    the corrected path differs from it, its K/V equal the naive K/V wherever no correction
    applies (first unit: zero residual), and the probe arrays are well formed."""
    w = testgen.reduced(testgen.workload("c3"), dtype="f16")
    m = w.model
    import paper_2607_21604_b200 as akvs
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(16) as ex:
        layers = list(ex.map(lambda l: testgen.layer_weights(m, 1234, l), range(m.n_layers)))
    gmodel = akvs.Model.from_numpy(m, testgen.embedding(m, 1234), layers)
    del layers
    lens = testgen.unit_lengths(w, 1236)
    ctx_ids, qry = testgen.token_ids(w, 1235, lens)
    store = akvs.UnitStore(gmodel, lens, ctx_ids)
    req = akvs.Request(list(range(w.n_units)), qry)
    N, nq, M = int(lens.sum()), w.n_query, w.n_units
    ws = akvs.alloc_workspace(akvs.workspace_bytes(gmodel, N, nq, M, 2))
    akvs.encode_units(gmodel, store, ws)
    assert akvs.check(ws) == 0

    def run(mode, bp=0, check_layer=1):
        hid, k, v = akvs.alloc_outputs(gmodel, N, nq)
        probes, ctx = None, None
        if mode == akvs.MODE_CORRECTED:
            probes, ctx = akvs.Probes(N, M, nq), C.c_void_p()
            akvs.select_probes(gmodel, store, req, bp, check_layer, probes, ctx, ws)
        akvs.prefill_corrected(gmodel, store, req, probes, mode, hid, k, v, ctx, ws)
        assert akvs.check(ws) == 0
        if ctx is not None:
            akvs.free(ctx)
        return hid, k, v, probes

    naive = run(akvs.MODE_NAIVE)
    zero = run(akvs.MODE_CORRECTED, 0, 1)
    for a, b in zip(zero[:3], naive[:3]):
        assert torch.equal(a, b)
    corr = run(akvs.MODE_CORRECTED, 1500, 2)
    p = corr[3]
    off = np.concatenate([[0], np.cumsum(lens)])
    b = [(int(n) * 1500 + 9999) // 10000 for n in lens]
    assert np.array_equal(p.probe_off.cpu().numpy()[:M + 1], np.concatenate([[0], np.cumsum(b)]))
    sk = p.sk_idx.cpu().numpy()[:sum(b)]
    rows = p.rows.cpu().numpy()[:p.n_rows]
    assert np.all(np.diff(rows) > 0) and rows[-1] == N + nq - 1 and p.n_rows == p.n_probe_rows + nq
    o = 0
    for u in range(M):
        s = sk[o:o + b[u]]
        assert np.all(np.diff(s) > 0) and s[0] >= off[u] and s[-1] < off[u + 1]
        o += b[u]
    assert max(b) <= p.n_probe_rows <= 2 * sum(b)
    n0 = int(lens[0])
    d = p.d_k.cpu().numpy()
    assert d[:n0].max() < 1e-2 * d[n0:N].mean()                  # first unit: zero residual
    # layers past the check layer: first-unit non-probe K equals the re-aligned cache (= naive K)
    assert orc.rel_l2(t2n(corr[1][5, :n0]), t2n(naive[1][5, :n0])) < 2e-3
    assert orc.rel_l2(t2n(corr[1][5, n0:N]), t2n(naive[1][5, n0:N])) > 1e-2
    assert torch.isfinite(corr[0]).all() and float(corr[0].abs().max()) > 0
