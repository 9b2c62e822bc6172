"""Refresh-ratio, context-length and batch sweep of the corrected prefill on synthetic contexts:
the shape of the throughput study (Section 4.4: speedup over no reuse against refresh ratio,
tokens per request and batch size) with the relative L2 error of the query hidden state
against the same build's full recompute as the quality proxy (random-init weights: the error
columns show trends, not answer quality).

    python -m paper_2607_21604_b200.sweep --workload c2 --ratios 100,500,1000,2000,3000,5000,7500 \
        --units 8,16,32,64 --batch 1,4,16

Prints one markdown table row per (tokens per request, batch, refresh ratio):
time of select + corrected prefill, full recompute and naive reuse; speedup over full
recompute; error of naive reuse, of selective recompute without the offset (weights forced
to 0) and of the corrected reuse.  Everything runs through the library's public calls."""
import argparse
import ctypes as C

import numpy as np
import torch

import testgen
from . import binding as akvs

SEED_W, SEED_IDS, SEED_LEN = 1234, 1235, 1236


def rel_l2(a, b):
    return float(torch.linalg.vector_norm((a - b).double()) / torch.linalg.vector_norm(b.double()))


def timed(fn, steps=3, warmup=1):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / steps


def run(w0, ratios, unit_counts=None, batches=(1,), check_layer=2, emit=print, std_scale=1.0):
    """Sweeps one workload; prints a markdown table through `emit` and returns its rows as dicts
    (tok_per_req, batch, refresh_bp, rows, corrected_ms, full_ms, naive_ms, err_naive,
    err_no_offset, err_corrected).  `std_scale` multiplies the seeded weights (tests)."""
    m = w0.model
    unit_counts = list(unit_counts) if unit_counts else [w0.n_units]

    def layer(l):
        lw = testgen.layer_weights(m, SEED_W, l)
        return {k: (v * np.float32(std_scale) if k.startswith("w") else v) for k, v in lw.items()} if std_scale != 1.0 else lw

    gmodel = akvs.Model.from_layer_fn(m, testgen.embedding(m, SEED_W) * np.float32(std_scale), layer, n_threads=12)
    kvf = {"native": akvs.KV_NATIVE, "q4": akvs.KV_Q4, "q2": akvs.KV_Q2, "fp8": akvs.KV_FP8}[w0.kv_format]
    emit(f"# {w0.name}: {m.name}-class decoder L{m.n_layers} d{m.d_model}, units {w0.len_lo}-{w0.len_hi} tokens, "
         f"{w0.n_query} query tokens, check layer {check_layer}, cache {w0.kv_format}")
    emit("| tok/req | batch | refresh | rows recomputed | corrected ms | full ms | naive ms | speedup vs full | "
         "err naive | err no offset | err corrected |")
    emit("|---|---|---|---|---|---|---|---|---|---|---|")
    rows_out = []
    for n_units in unit_counts:
        w = testgen.reduced(w0, n_units=n_units)
        lens = testgen.unit_lengths(w, SEED_LEN)
        ctx_ids, qry_ids = testgen.token_ids(w, SEED_IDS, lens)
        store = akvs.UnitStore(gmodel, lens, ctx_ids, kvf)
        N1, nq1, M1 = int(lens.sum()), w.n_query, n_units
        ws0 = akvs.alloc_workspace(akvs.workspace_bytes(gmodel, N1, 0, M1, 1))
        akvs.encode_units(gmodel, store, ws0)
        assert akvs.check(ws0) == 0
        del ws0
        for B in batches:
            order = list(range(M1))
            if B == 1:
                req = akvs.Request(order, qry_ids)
            else:
                req = akvs.Request.batch([([(u + 5 * b) % M1 for u in order], np.roll(qry_ids, 7 * b))
                                          for b in range(B)])
            N, nq, M = N1 * B, nq1 * B, M1 * B
            ws = akvs.alloc_workspace(akvs.workspace_bytes(gmodel, N, nq, M, check_layer))
            hid, k, v = akvs.alloc_outputs(gmodel, N, nq)
            probes, ctx = akvs.Probes(N, M, nq), C.c_void_p()

            def full():
                akvs.prefill_corrected(gmodel, store, req, None, akvs.MODE_FULL, hid, k, v, None, ws)

            def naive():
                akvs.prefill_corrected(gmodel, store, req, None, akvs.MODE_NAIVE, hid, k, v, None, ws)

            full_ms = timed(full)
            h_full = hid.clone()
            naive_ms = timed(naive)
            e_naive = rel_l2(hid, h_full)
            for bp in ratios:
                def corrected():
                    akvs.select_probes(gmodel, store, req, bp, check_layer, probes, ctx, ws)
                    akvs.prefill_corrected(gmodel, store, req, probes, akvs.MODE_CORRECTED, hid, k, v, ctx, ws)

                ms = timed(corrected)
                e_corr = rel_l2(hid, h_full)
                # the same probe rows recomputed, the rest left stale: weights forced to zero
                probes.w_k.zero_()
                probes.w_v.zero_()
                akvs.prefill_corrected(gmodel, store, req, probes, akvs.MODE_CORRECTED, hid, k, v, ctx, ws)
                e_sel = rel_l2(hid, h_full)
                assert akvs.check(ws) == 0
                emit(f"| {N1} | {B} | {bp / 100:g} % | {probes.n_rows} / {N + nq} | {ms:.2f} | {full_ms:.2f} | "
                     f"{naive_ms:.2f} | {full_ms / ms:.2f}x | {e_naive:.3e} | {e_sel:.3e} | {e_corr:.3e} |")
                rows_out.append({"tok_per_req": N1, "batch": B, "refresh_bp": bp, "rows": probes.n_rows,
                                 "corrected_ms": ms, "full_ms": full_ms, "naive_ms": naive_ms, "err_naive": e_naive,
                                 "err_no_offset": e_sel, "err_corrected": e_corr})
            akvs.free(ctx)
            del ws, hid, k, v, probes
            torch.cuda.empty_cache()
    return rows_out


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--ratios", default="100,500,1000,2000,3000,5000,7500", help="refresh ratios in basis points")
    ap.add_argument("--units", default="", help="units per request (default: the workload's)")
    ap.add_argument("--batch", default="1", help="requests per call")
    ap.add_argument("--check-layer", type=int, default=2)
    ap.add_argument("--layers", type=int, default=0)
    args = ap.parse_args(argv)
    w0 = testgen.workload(args.workload)
    if w0.model.dtype != "f32":
        w0 = testgen.reduced(w0, dtype="f16")
    if args.layers:
        w0 = testgen.reduced(w0, n_layers=args.layers)
    ratios = [int(x) for x in args.ratios.split(",")]
    unit_counts = [int(x) for x in args.units.split(",")] if args.units else None
    batches = [int(x) for x in args.batch.split(",")]
    return run(w0, ratios, unit_counts, batches, args.check_layer, emit=lambda s: print(s, flush=True))


if __name__ == "__main__":
    main()
