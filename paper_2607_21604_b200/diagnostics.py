"""Mean-explained residual energy per layer on a synthetic context (the appendix that validates
the residual model r_i = mu + xi_i of Section 3.4): how much of a unit's residual energy
sum_i |fresh_i - reuse_i|^2 a single correction vector removes, for three vectors

    E1  the exact unit mean                                     (oracle)
    E2  the mean of b probes drawn uniformly with replacement   (the estimator of Propositions 2-3)
    E3w the mean of the top-b divergence probes, added with w = min(d, 1)  (the practical rule)

with b = ceil(r n).  Residuals come from the same build's full recompute; every reduction runs
in akvs_op_residual_stats.  With random-init weights the numbers describe this synthetic model,
not a trained one.

    python -m paper_2607_21604_b200.diagnostics --workload c2 --layers 8 --units 8 --ratio 1000"""
import argparse
import ctypes as C

import numpy as np
import torch

import testgen
from . import binding as akvs

SEED_W, SEED_IDS, SEED_LEN, SEED_PROBE = 1234, 1235, 1236, 1237


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--units", type=int, default=0)
    ap.add_argument("--ratio", type=int, default=1000, help="probe budget in basis points")
    ap.add_argument("--check-layer", type=int, default=2)
    args = ap.parse_args()
    w = testgen.workload(args.workload)
    if w.model.dtype != "f32":
        w = testgen.reduced(w, dtype="f16")
    w = testgen.reduced(w, n_layers=args.layers or None, n_units=args.units or None)
    m = w.model
    gmodel = akvs.Model.from_layer_fn(m, testgen.embedding(m, SEED_W), lambda l: testgen.layer_weights(m, SEED_W, l),
                                      n_threads=12)
    lens = testgen.unit_lengths(w, SEED_LEN)
    ctx_ids, qry_ids = testgen.token_ids(w, SEED_IDS, lens)
    kvf = {"native": akvs.KV_NATIVE, "q4": akvs.KV_Q4, "q2": akvs.KV_Q2, "fp8": akvs.KV_FP8}[w.kv_format]
    store = akvs.UnitStore(gmodel, lens, ctx_ids, kvf)
    N, nq, M = int(lens.sum()), w.n_query, w.n_units
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    ws = akvs.alloc_workspace(akvs.workspace_bytes(gmodel, N, nq, M, args.check_layer))
    akvs.encode_units(gmodel, store, ws)
    req = akvs.Request(list(range(M)), qry_ids)
    hid, k_full, v_full = akvs.alloc_outputs(gmodel, N, nq)
    akvs.prefill_corrected(gmodel, store, req, None, akvs.MODE_FULL, hid, k_full, v_full, None, ws)
    probes, ctx = akvs.Probes(N, M, nq), C.c_void_p()
    akvs.select_probes(gmodel, store, req, args.ratio, args.check_layer, probes, ctx, ws)
    assert akvs.check(ws) == 0
    akvs.free(ctx)
    dev_ = hid.device
    # the three selections as per-token weights of the mean
    poff = probes.probe_off[:M + 1].cpu().numpy()
    n_probe = int(poff[-1])
    top_k = torch.zeros(N, dtype=torch.float32, device=dev_)
    top_v = torch.zeros_like(top_k)
    top_k[probes.sk_idx[:n_probe].long()] = 1.0
    top_v[probes.sv_idx[:n_probe].long()] = 1.0
    g = np.random.default_rng(SEED_PROBE)
    rnd = np.zeros(N, np.float32)
    for u in range(M):
        b = int(poff[u + 1] - poff[u])
        if b:
            np.add.at(rnd, off[u] + g.integers(0, lens[u], b), 1.0)
    rnd = torch.from_numpy(rnd).to(dev_)
    src = torch.arange(N, dtype=torch.int32, device=dev_)
    dt = {"f32": akvs.F32, "bf16": akvs.BF16, "f16": akvs.F16}[m.dtype]
    print(f"# {w.name}: {m.name}-class decoder, {m.n_layers} layers, {M} units ({N} tokens), probe budget "
          f"{args.ratio / 100:g} % per unit, cache {w.kv_format}; mean-explained residual energy, all units pooled")
    print("| layer | K: exact mean | K: random probes | K: top-b, weighted | V: exact mean | V: random probes | "
          "V: top-b, weighted |")
    print("|---|---|---|---|---|---|---|")
    for l in range(args.check_layer - 1, m.n_layers):
        km = store.k_meta[l] if store.k_meta is not None else None
        vm = store.v_meta[l] if store.v_meta is not None else None
        base = (dt, kvf, store.k[l], store.v[l], km, vm, src, k_full[l][:N].contiguous(), v_full[l][:N].contiguous(),
                off, m.n_kv_heads, m.head_dim, m.rope_base)

        def explained(sel_k, sel_v, w_k=None, w_v=None):
            mk, mv, _ = akvs.op_residual_stats(*base, sel_k=sel_k, sel_v=sel_v)
            _, _, en = akvs.op_residual_stats(*base, mu_k=mk, mu_v=mv, w_k=w_k, w_v=w_v)
            en = en.double().sum(dim=0).cpu().numpy()
            return 1.0 - en[1] / en[0], 1.0 - en[3] / en[2]

        e1 = explained(None, None)
        e2 = explained(rnd, rnd)
        e3 = explained(top_k, top_v, probes.w_k[:N].contiguous(), probes.w_v[:N].contiguous())
        print(f"| {l + 1} | {e1[0]:.3f} | {e2[0]:.3f} | {e3[0]:.3f} | {e1[1]:.3f} | {e2[1]:.3f} | {e3[1]:.3f} |", flush=True)


if __name__ == "__main__":
    main()
