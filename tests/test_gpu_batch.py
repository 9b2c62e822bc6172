"""Batched requests that share the model (the batch sizes of the throughput study, Section 4.4):
one call runs the linear layers over the rows of all requests while every request keeps its
own positions, attention ranges, offsets and corrections.  Each request of a batch must match
the oracle run on that request ALONE, in all three modes, within the usual tolerances."""
import ctypes as C

import numpy as np
import pytest
import torch

import testgen
from oracle import akvs_oracle as orc
from gpu_helpers import Case, t2n, max_layer_err
from test_gpu_pipeline import small16, F32_HD128

pytestmark = pytest.mark.gpu


def _split(total, parts):
    """Cuts range(total) into len(parts) consecutive pieces proportional to `parts`."""
    cuts = np.floor(np.cumsum(parts) / np.sum(parts) * total).astype(int)
    cuts[-1] = total
    return np.concatenate([[0], cuts])


class BatchCase:
    def __init__(self, case, orders, q_parts, check_layer):
        self.c, self.orders = case, [list(o) for o in orders]
        a = case.akvs
        qo = _split(len(case.qry), q_parts)
        self.qrys = [case.qry[qo[i]:qo[i + 1]] for i in range(len(orders))]
        self.ctxs = [np.concatenate([case.units_ids[u] for u in o]) if len(o) else np.zeros(0, np.int32)
                     for o in self.orders]
        self.cs = np.concatenate([[0], np.cumsum([len(x) for x in self.ctxs])]).astype(int)
        self.qs = qo
        self.N, self.nq, self.M = int(self.cs[-1]), int(qo[-1]), sum(len(o) for o in self.orders)
        self.req = a.Request.batch(list(zip(self.orders, self.qrys)))
        self.ws = a.alloc_workspace(a.workspace_bytes(case.gmodel, max(self.N, case.store.n_tokens), self.nq,
                                                      max(self.M, case.store.n_units), check_layer))

    def prefill(self, mode, probes=None, ctx=None):
        a, c = self.c.akvs, self.c
        hid, k, v = a.alloc_outputs(c.gmodel, self.N, self.nq)
        a.prefill_corrected(c.gmodel, c.store, self.req, probes, mode, hid, k, v, ctx, self.ws)
        assert a.check(self.ws) == 0
        return t2n(hid), t2n(k), t2n(v)

    def request_view(self, b, hid, k, v):
        """Rows of request b in the merged outputs, in the single-request order (context, query)."""
        cs, ce, qs, qe = self.cs[b], self.cs[b + 1], self.qs[b], self.qs[b + 1]
        rows = np.concatenate([np.arange(cs, ce), self.N + np.arange(qs, qe)]).astype(int)
        return hid[qs:qe], k[:, rows], v[:, rows]

    def check(self, got, refs, tol):
        for b, ref in enumerate(refs):
            hid, k, v = self.request_view(b, *got)
            assert orc.rel_l2(hid, ref[0]) < tol, b
            assert max_layer_err(k, ref[1]) < tol and max_layer_err(v, ref[2]) < tol, b


def _run(case, orders, q_parts, bp, check_layer):
    bc = BatchCase(case, orders, q_parts, check_layer)
    a, tol = case.akvs, case.tol
    case.encode()
    units = case.oracle_units()
    full = [orc.full_recompute(case.omodel, bc.ctxs[b], bc.qrys[b]) for b in range(len(orders))]
    bc.check(bc.prefill(a.MODE_FULL), full, tol)
    case.load_oracle_cache(units)
    # a request without units has nothing to reuse: every mode is the query computed alone
    naive = [orc.naive_reuse(case.omodel, units, bc.orders[b], bc.qrys[b]) if bc.orders[b] else full[b]
             for b in range(len(orders))]
    bc.check(bc.prefill(a.MODE_NAIVE), naive, tol)

    z = np.zeros(0, np.int64)
    empty = lambda f: {"hidden": f[0], "K": f[1], "V": f[2], "ctx_off": np.zeros(1, np.int64), "d_k": np.zeros(0),
                       "d_v": np.zeros(0), "probes": {"probe_off": np.zeros(1, np.int64), "sk_idx": z, "sv_idx": z,
                                                      "w_k": np.zeros(0), "w_v": np.zeros(0), "ctx_rows": z}}
    refs = [orc.corrected_reuse(case.omodel, units, bc.orders[b], bc.ctxs[b], bc.qrys[b], bp, check_layer)
            if bc.orders[b] else empty(full[b]) for b in range(len(orders))]
    probes, ctx = a.Probes(bc.N, bc.M, bc.nq), C.c_void_p()
    a.select_probes(case.gmodel, case.store, bc.req, bp, check_layer, probes, ctx, bc.ws)
    # merged bookkeeping equals the per-request bookkeeping, shifted
    ctx_off = np.concatenate([[0]] + [bc.cs[b] + r["ctx_off"][1:] for b, r in enumerate(refs)]).astype(np.int64)
    poff = np.concatenate([[0], np.cumsum(np.concatenate([np.diff(r["probes"]["probe_off"]) for r in refs]))])
    assert np.array_equal(probes.ctx_off.cpu().numpy()[:bc.M + 1], ctx_off)
    assert np.array_equal(probes.probe_off.cpu().numpy()[:bc.M + 1], poff)
    d_k = np.concatenate([r["d_k"] for r in refs])
    mask = np.ones(bc.N, bool)
    for b, r in enumerate(refs):                      # a request's first unit has ~zero scores on both sides
        if len(r["ctx_off"]) > 1:
            mask[bc.cs[b]:bc.cs[b] + int(r["ctx_off"][1])] = False
    if check_layer > 1 and mask.any():
        assert orc.rel_l2(t2n(probes.d_k)[:bc.N][mask], d_k[mask]) < tol
    # the oracle's probe sets, merged, on the GPU side
    dev = probes.sk_idx.device
    put = lambda dst, x, dt: dst[:len(x)].copy_(torch.from_numpy(np.asarray(x).astype(dt)).to(dev))
    put(probes.sk_idx, np.concatenate([bc.cs[b] + r["probes"]["sk_idx"] for b, r in enumerate(refs)]), np.int32)
    put(probes.sv_idx, np.concatenate([bc.cs[b] + r["probes"]["sv_idx"] for b, r in enumerate(refs)]), np.int32)
    put(probes.w_k, np.concatenate([r["probes"]["w_k"] for r in refs]), np.float32)
    put(probes.w_v, np.concatenate([r["probes"]["w_v"] for r in refs]), np.float32)
    ctx_rows = np.concatenate([bc.cs[b] + r["probes"]["ctx_rows"] for b, r in enumerate(refs)])
    rows = np.concatenate([ctx_rows, bc.N + np.arange(bc.nq)])
    put(probes.rows, rows, np.int32)
    put(probes.probe_off, poff, np.int32)
    probes.desc.n_probe_rows, probes.desc.n_rows = len(ctx_rows), len(rows)
    got = bc.prefill(a.MODE_CORRECTED, probes, ctx)
    a.free(ctx)
    bc.check(got, [(r["hidden"], r["K"], r["V"]) for r in refs], tol)
    return bc, got


def test_batch_float_simt_paths():
    """Float model (CUDA-core attention, head_dim 64): three requests of different shapes."""
    case = Case(testgen.workload("c1"))
    M = len(case.lens)
    _run(case, [list(range(M)), [M - 1, 0], [1]], [3, 1, 2], 2500, 2)


def test_batch_float_hd128():
    case = Case(F32_HD128)
    _run(case, [[2, 0, 3], [1, 3, 0, 2]], [1, 1], 2500, 2)


@pytest.mark.parametrize("check_layer", [1, 2])
def test_batch_f16_tensor_core_paths(check_layer):
    """float16 model with head_dim 128: tcgen05 linear layers over the merged rows and the
    tensor-core attention with two visible ranges per query row."""
    case = Case(small16("f16"), std_scale=4.0)
    _run(case, [[0, 1, 2, 3, 4], [3, 1], [4, 0, 2], [2]], [2, 1, 3, 1], 2500, check_layer)


@pytest.mark.parametrize("kv_format", [4, 8])
def test_batch_quantised_caches(kv_format):
    """Batched requests over a 4-bit group-quantised and an FP8 cache (dequantisation fused into
    the scores / offsets / correction reads of every request)."""
    case = Case(small16("f16"), std_scale=4.0, kv_format=kv_format)
    _run(case, [[4, 3, 2, 1, 0], [0, 2], [1, 4, 3]], [1, 2, 1], 2500, 2)


def test_batch_bf16_storage():
    case = Case(small16("bf16"), std_scale=1.0)
    _run(case, [[0, 1, 2], [4, 3]], [1, 1], 2500, 2)


def test_batch_request_without_context():
    """A request with no units (query only) inside a batch: its rows see only its own query."""
    case = Case(small16("f16"), std_scale=4.0)
    _run(case, [[1, 0], [], [2, 4]], [1, 1, 1], 2500, 2)


def test_batch_of_one_equals_single_request():
    """n_requests = 1 takes the single-request path: identical bits."""
    case = Case(small16("f16"), std_scale=4.0)
    a = case.akvs
    case.encode()
    single = case.gpu_prefill(a.MODE_NAIVE)
    req1 = a.Request.batch([(case.order, case.qry)])
    hid, k, v = a.alloc_outputs(case.gmodel, case.N, case.nq)
    ws = case.workspace()
    a.prefill_corrected(case.gmodel, case.store, req1, None, a.MODE_NAIVE, hid, k, v, None, ws)
    assert a.check(ws) == 0
    assert np.array_equal(t2n(hid), single[0]) and np.array_equal(t2n(k), single[1])


def test_batch_argument_validation():
    case = Case(testgen.workload("c1"))
    a = case.akvs
    ws = case.workspace()
    hid, k, v = a.alloc_outputs(case.gmodel, case.N, case.nq)
    bad = a.Request(case.order, case.qry, unit_off=[0, 2, case.M - 1], query_off=[0, 1, case.nq])   # last != n_units
    with pytest.raises(a.AkvsError):
        a.prefill_corrected(case.gmodel, case.store, bad, None, a.MODE_FULL, hid, k, v, None, ws)
    bad = a.Request(case.order, case.qry, unit_off=[0, 3, 2, case.M], query_off=[0, 1, 2, case.nq])  # not monotone
    with pytest.raises(a.AkvsError):
        a.prefill_corrected(case.gmodel, case.store, bad, None, a.MODE_FULL, hid, k, v, None, ws)
