"""Parity at the configurations as they are specified: full depth, full context, both 16-bit
storage types.

* config 2 (3B-class): all 36 layers, all 20 units (5219 context + 64 query tokens), 10 % refresh -
  the configuration whose ~1000 recomputed rows make the residual linear layers split their k
  range into ordered partial sums;
* config 3 (the benchmarked one): all 32 layers, all 32 units (8593 context + 128 query tokens),
  15 % refresh, check layer 2;
* config 5 with the 4-bit cache: all 32 layers, the first 16 of its 48 units (4096 context
  tokens: the cut keeps the oracle's run near a minute; width, depth and refresh are the
  configuration's);
* config 4 (32B-class): its first 8 of 64 layers, the first 12 of its 30 units (4608 tokens).

The oracle runs here, on the host cores, once per configuration (numpy: encode every unit alone
in its float32 variant, then Algorithm 1 in float64); its result serves both storage types.  For that the two sides
share inputs that are representable in float16 AND bfloat16: the configurations' bf16-valued
weights, and a unit cache whose values are the oracle's encoding rounded to bf16 (the
configurations say "bf16"; a float16 container holds such values exactly).  Each test prints
the error of every layer's K and V and of the query hidden state.

What is asserted
* float16 storage: every tensor within the benchmark spec's 1e-2.
* bfloat16 storage: the same rounding points with unit roundoff 2^-8 instead of 2^-11, so to
  first order every error is 8x the float16 one.  Asserted: each tensor's error is at most
  BF16_RATIO_CAP = 12 times the float16 error of the same tensor (8 x 1.5 for the spread between two
  realisations of the rounding noise) and under BF16_ABS_CAP = 5e-2 absolutely.  Whether it
  also meets 1e-2 is printed, not asserted: past about a dozen random-init layers it does not.
* the library's own probe selection at full size: the selection function is bit-exact on
  the library's scores, and the sets it picks overlap the oracle's almost everywhere (scores
  differ by 16-bit rounding, so ties at the cut may fall differently).
"""
import dataclasses
import functools
import os
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import testgen
from oracle import akvs_oracle as orc
from gpu_helpers import Case, t2n, both_16bit
from helpers import SEED_W, make_inputs

pytestmark = pytest.mark.gpu

BF16_RATIO_CAP = 12.0
BF16_ABS_CAP = 5e-2
CHECK_LAYER = 2

# name -> (workload, layers, units, cache format)
FULL = {
    "c2": ("c2", None, None, 0),
    "c3": ("c3", None, None, 0),
    "c5q4": ("c5q4", None, 16, 4),
    "c4": ("c4", 8, 12, 0),
}


def _workload(name):
    base, n_layers, n_units, _ = FULL[name]
    # "f16" weight values: the configuration's bf16 values, representable in both 16-bit types
    return testgen.reduced(testgen.workload(base), n_layers=n_layers, n_units=n_units, dtype="f16")


@functools.lru_cache(maxsize=1)
def _golden(name):
    """Oracle side of one configuration: model, encoded units (cache rounded as above, or its
    4-bit codes), corrected reuse.  Cached for the two storage types; one entry at a time."""
    t0 = time.time()
    orc.ATTENTION_WORKERS = max(1, min(16, len(os.sched_getaffinity(0))))     # heads in parallel: same arithmetic
    w = _workload(name)
    m = w.model
    with ThreadPoolExecutor(16) as ex:
        layers = list(ex.map(lambda l: testgen.layer_weights(m, SEED_W, l), range(m.n_layers)))
    omodel = orc.Model(m, testgen.embedding(m, SEED_W), layers)
    lens, ctx_store, qry, units_ids = make_inputs(w)
    fmt = FULL[name][3]
    t1 = time.time()
    # the isolated encoding in the oracle's single-precision variant (it agrees with the float64 one
    # to ~1e-5, far inside both the 16-bit rounding the cache gets below and the 1e-2 bound of the
    # encoder check) - it is the larger half of the oracle's work; Algorithm 1 itself runs in float64
    units = orc.encode_units(omodel, units_ids, kv_bits=fmt, dtype=np.float32)
    fresh_units = None
    if fmt == 0:
        # keep the unrounded encoding for the check of the library's own encoder
        fresh_units = [{"K": u["K"], "V": u["V"]} for u in units]
        units = [{"K": both_16bit(u["K"]), "V": both_16bit(u["V"])} for u in units]
    t2 = time.time()
    ctx = np.concatenate(units_ids)
    ref = orc.corrected_reuse(omodel, units, list(range(len(units))), ctx, qry, w.refresh_bp[0], CHECK_LAYER)
    t3 = time.time()
    print(f"\n[{name}] oracle: weights {t1 - t0:.0f} s, encode_units {t2 - t1:.0f} s, corrected_reuse {t3 - t2:.0f} s; "
          f"L={m.n_layers} N={len(ctx)} n_q={len(qry)} rows={len(ref['rows'])}")
    return w, omodel, units, fresh_units, ref


_F16_ERR = {}       # (name, tensor) -> per-layer float16 errors, for the bf16 ratio bound


def _curve(label, errs):
    print(f"  {label}: " + " ".join(f"{e:.2e}" for e in errs))


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("name", ["c2", "c3", "c5q4", "c4"])
def test_full_depth_corrected_prefill(name, dtype):
    w, omodel, units, fresh_units, ref = _golden(name)
    fmt = FULL[name][3]
    case = Case(w, kv_format=fmt, omodel=omodel, gpu_dtype=dtype)
    L = w.model.n_layers

    # ---- the library's own encoder against the oracle's (unrounded) encoding, every layer
    case.encode()
    if fmt == 0:
        gk, gv = t2n(case.store.k), t2n(case.store.v)
        ok = np.concatenate([u["K"] for u in fresh_units], axis=1)
        ov = np.concatenate([u["V"] for u in fresh_units], axis=1)
        enc_k = [orc.rel_l2(gk[l], ok[l]) for l in range(L)]
        enc_v = [orc.rel_l2(gv[l], ov[l]) for l in range(L)]
        del gk, gv, ok, ov
    else:
        enc_k = enc_v = []

    # ---- both sides read the same cache from here on
    case.load_oracle_cache(units)

    # ---- the library's selection at full size
    probes, ctx, ws = case.gpu_select(w.refresh_bp[0], CHECK_LAYER)
    poff = ref["probes"]["probe_off"]
    assert np.array_equal(probes.ctx_off.cpu().numpy()[:case.M + 1], ref["ctx_off"])
    assert np.array_equal(probes.probe_off.cpu().numpy()[:case.M + 1], poff)
    d_k, d_v = t2n(probes.d_k)[:case.N], t2n(probes.d_v)[:case.N]
    n0 = int(ref["ctx_off"][1])                      # first unit: zero residual on both sides
    score_err = (orc.rel_l2(d_k[n0:], ref["d_k"][n0:]), orc.rel_l2(d_v[n0:], ref["d_v"][n0:]))
    again = orc.select_probes(d_k.astype(np.float32), d_v.astype(np.float32), ref["ctx_off"], w.refresh_bp[0])
    nP = int(poff[-1])
    g_sk, g_sv = probes.sk_idx.cpu().numpy()[:nP], probes.sv_idx.cpu().numpy()[:nP]
    assert np.array_equal(g_sk, again["sk_idx"]) and np.array_equal(g_sv, again["sv_idx"])   # bit-exact on its scores
    assert np.array_equal(probes.rows.cpu().numpy()[:probes.n_probe_rows], again["ctx_rows"])
    far = lambda s: s[s >= n0]
    overlap = (len(np.intersect1d(far(g_sk), far(ref["probes"]["sk_idx"]))) / max(1, len(far(ref["probes"]["sk_idx"]))),
               len(np.intersect1d(far(g_sv), far(ref["probes"]["sv_idx"]))) / max(1, len(far(ref["probes"]["sv_idx"]))))

    # ---- corrected prefill with the oracle's probe sets
    case.set_probes(probes, ref["probes"])
    hid, k, v = case.gpu_prefill(case.akvs.MODE_CORRECTED, ws, probes, ctx, CHECK_LAYER)
    case.akvs.free(ctx)
    e_h = orc.rel_l2(hid, ref["hidden"])
    e_k = [orc.rel_l2(k[l], ref["K"][l]) for l in range(L)]
    e_v = [orc.rel_l2(v[l], ref["V"][l]) for l in range(L)]
    del k, v

    print(f"\n[{name} {dtype}] N={case.N} n_q={case.nq} L={L} rows={len(ref['rows'])} cache format {fmt}")
    print(f"  scores d_K, d_V: {score_err[0]:.2e} {score_err[1]:.2e}; own probe sets vs oracle's: "
          f"{overlap[0]:.4f} {overlap[1]:.4f} of S^K, S^V shared")
    if enc_k:
        _curve("encode_units K per layer", enc_k)
        _curve("encode_units V per layer", enc_v)
    _curve("corrected K per layer", e_k)
    _curve("corrected V per layer", e_v)
    print(f"  query hidden: {e_h:.2e}; max K {max(e_k):.2e}; max V {max(e_v):.2e}; "
          f"within 1e-2: {max([e_h] + e_k + e_v) < 1e-2}")

    tensors = {"hidden": [e_h], "K": e_k, "V": e_v, "enc_K": enc_k, "enc_V": enc_v,
               "scores": list(score_err)}
    if dtype == "f16":
        for t, errs in tensors.items():
            _F16_ERR[(name, t)] = errs
            assert all(e < case.tol for e in errs), (t, max(errs))
        assert min(overlap) > 0.97
    else:
        for t, errs in tensors.items():
            assert all(e < BF16_ABS_CAP for e in errs), (t, max(errs))
            base = _F16_ERR.get((name, t))
            if base:                                   # the float16 run of this configuration came first
                # floor: where the float16 error is at float-accumulation level, 16-bit rounding is not
                # what it measures
                ratios = [e / max(b, 2e-4) for e, b in zip(errs, base)]
                print(f"  bf16 / f16 error ratio, {t}: max {max(ratios):.1f}, median {float(np.median(ratios)):.1f}")
                assert max(ratios) < BF16_RATIO_CAP, (t, max(ratios))
        assert min(overlap) > 0.90
