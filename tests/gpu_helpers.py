"""Plumbing shared by the GPU parity tests: the same seeded inputs go to the oracle (numpy,
float64) and to the CUDA library (through the C ABI binding)."""
import ctypes as C
import dataclasses

import numpy as np
import torch

import testgen
from oracle import akvs_oracle as orc
from helpers import oracle_model, make_inputs

TOL = {"f32": 2e-3, "bf16": 1e-2, "f16": 1e-2}          # max relative L2 error per tensor (the benchmark spec)


def t2n(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def both_16bit(x):
    """Values representable in bfloat16 AND in float16: round to bf16, then to float16 (which
    only touches magnitudes under 2^-17 and keeps them bf16-representable).  Inputs rounded this
    way can be given unchanged to a model in either 16-bit storage type."""
    r = testgen.bf16_round(np.asarray(x, np.float32))
    return r.astype(np.float16).astype(np.float64)


class Case:
    """A workload instantiated on both sides."""

    def __init__(self, w, std_scale=1.0, kv_format=0, order=None, omodel=None, gpu_dtype=None):
        """`omodel`: an oracle model built elsewhere (shared between cases); `gpu_dtype`: storage
        type of the library's model when it differs from the workload's (the weight VALUES must
        then be representable in both, which holds for bf16 values rounded to float16)."""
        import paper_2607_21604_b200 as akvs
        self.akvs = akvs
        self.w, self.cfg = w, w.model
        self.omodel = oracle_model(w.model, std_scale=std_scale) if omodel is None else omodel
        self.lens, self.ctx_store, self.qry, self.units_ids = make_inputs(w)
        self.order = list(range(len(self.lens))) if order is None else list(order)
        self.ctx = np.concatenate([self.units_ids[u] for u in self.order]) if len(self.order) else np.zeros(0, np.int32)
        self.N, self.nq, self.M = len(self.ctx), len(self.qry), len(self.order)
        gcfg = w.model if gpu_dtype is None else dataclasses.replace(w.model, dtype=gpu_dtype)
        self.gmodel = akvs.Model.from_numpy(gcfg, self.omodel.tok_emb, self.omodel.layers)
        self.kv_format = kv_format
        self.store = akvs.UnitStore(self.gmodel, self.lens, self.ctx_store, kv_format)
        self.req = akvs.Request(self.order, self.qry)
        self.tol = TOL[gcfg.dtype]

    def workspace(self, check_layer=1, n_ctx=None):
        n_ctx = max(self.N, self.store.n_tokens) if n_ctx is None else n_ctx
        nb = self.akvs.workspace_bytes(self.gmodel, n_ctx, self.nq, max(self.M, self.store.n_units), check_layer)
        return self.akvs.alloc_workspace(nb)

    def encode(self):
        ws = self.workspace()
        self.akvs.encode_units(self.gmodel, self.store, ws)
        assert self.akvs.check(ws) == 0
        return ws

    def oracle_units(self):
        bits = self.kv_format
        return orc.encode_units(self.omodel, self.units_ids, kv_bits=bits)

    def load_oracle_cache(self, units):
        """Gives both sides the same cache: the oracle's values in the store's format.  A
        16-bit store rounds them; the rounded values are written back into `units` so that
        the oracle reads exactly what the library reads (the cache is an input of the prefill)."""
        k = np.concatenate([u["K"] for u in units], axis=1)
        v = np.concatenate([u["V"] for u in units], axis=1)
        if self.kv_format == 0:
            self.store.k.copy_(torch.from_numpy(k).to(self.store.k.dtype))
            self.store.v.copy_(torch.from_numpy(v).to(self.store.v.dtype))
            ks, vs = t2n(self.store.k), t2n(self.store.v)
            o = 0
            for u in units:
                n = u["K"].shape[1]
                u["K"], u["V"] = ks[:, o:o + n], vs[:, o:o + n]
                o += n
        elif self.kv_format == 8:
            for name, dst in (("K", self.store.k), ("V", self.store.v)):
                dst.copy_(torch.from_numpy(np.concatenate([u[name + "_codes"] for u in units], axis=1)))
        else:
            for name, dst, dmeta in (("K", self.store.k, self.store.k_meta), ("V", self.store.v, self.store.v_meta)):
                codes = np.concatenate([u[name + "_codes"] for u in units], axis=1)
                dst.copy_(torch.from_numpy(orc.pack_codes(codes, self.kv_format)))
                s = np.concatenate([u[name + "_scale"] for u in units], axis=1)
                m = np.concatenate([u[name + "_min"] for u in units], axis=1)
                dmeta.copy_(torch.from_numpy(np.stack([s, m], axis=-1)))

    def gpu_prefill(self, mode, ws=None, probes=None, ctx=None, check_layer=1):
        a = self.akvs
        ws = self.workspace(check_layer) if ws is None else ws
        hid, k, v = a.alloc_outputs(self.gmodel, self.N, self.nq)
        a.prefill_corrected(self.gmodel, self.store, self.req, probes, mode, hid, k, v, ctx, ws)
        assert a.check(ws) == 0
        return t2n(hid), t2n(k), t2n(v)

    def gpu_select(self, refresh_bp, check_layer, ws=None):
        a = self.akvs
        ws = self.workspace(check_layer) if ws is None else ws
        probes = a.Probes(self.N, self.M, self.nq)
        ctx = C.c_void_p()
        a.select_probes(self.gmodel, self.store, self.req, refresh_bp, check_layer, probes, ctx, ws)
        return probes, ctx, ws

    def set_probes(self, probes, op):
        """Overwrites the GPU probe arrays with the oracle's selection `op`."""
        dev = probes.sk_idx.device
        nP = len(op["sk_idx"])
        probes.sk_idx[:nP] = torch.from_numpy(op["sk_idx"].astype(np.int32)).to(dev)
        probes.sv_idx[:nP] = torch.from_numpy(op["sv_idx"].astype(np.int32)).to(dev)
        probes.w_k[:self.N] = torch.from_numpy(np.asarray(op["w_k"], np.float32)).to(dev)
        probes.w_v[:self.N] = torch.from_numpy(np.asarray(op["w_v"], np.float32)).to(dev)
        rows = np.concatenate([op["ctx_rows"], np.arange(self.N, self.N + self.nq)]).astype(np.int32)
        probes.rows[:len(rows)] = torch.from_numpy(rows).to(dev)
        probes.probe_off[:self.M + 1] = torch.from_numpy(op["probe_off"].astype(np.int32)).to(dev)
        probes.desc.n_probe_rows = len(op["ctx_rows"])
        probes.desc.n_rows = len(rows)


def max_layer_err(a, b):
    """max over layers of the relative L2 error of [L][T][...] tensors."""
    return max(orc.rel_l2(a[l], b[l]) for l in range(len(b)))
