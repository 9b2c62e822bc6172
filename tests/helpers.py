"""Shared test plumbing: build oracle models and workloads from the seeded generators."""
import dataclasses

import numpy as np

import testgen
from oracle import akvs_oracle as orc

SEED_W, SEED_IDS, SEED_LEN = 1234, 1235, 1236


def small_cfg(n_layers=3, d_model=64, n_q=4, n_kv=2, hd=16, d_ff=96, vocab=128, dtype="f32"):
    return testgen.ModelCfg("small", n_layers, d_model, n_q, n_kv, hd, d_ff, vocab, dtype)


def small_workload(cfg=None, n_units=3, len_lo=9, len_hi=17, n_query=5, bp=(2500,)):
    return testgen.Workload("small", cfg or small_cfg(), n_units, len_lo, len_hi, n_query, bp)


def oracle_model(m, seed=SEED_W, std_scale=1.0):
    layers = [testgen.layer_weights(m, seed, l) for l in range(m.n_layers)]
    emb = testgen.embedding(m, seed)
    if std_scale != 1.0:
        s = np.float32(std_scale)
        emb = emb * s
        for lw in layers:
            for k in lw:
                if k.startswith("w"):
                    lw[k] = lw[k] * s
    return orc.Model(m, emb, layers)


def make_inputs(w, seed_ids=SEED_IDS, seed_len=SEED_LEN):
    lens = testgen.unit_lengths(w, seed_len)
    ctx, qry = testgen.token_ids(w, seed_ids, lens)
    off = np.zeros(len(lens) + 1, np.int64)
    off[1:] = np.cumsum(lens)
    units = [ctx[off[i]:off[i + 1]] for i in range(len(lens))]
    return lens, ctx, qry, units
