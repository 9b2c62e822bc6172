"""Counter-based seeded generators for the five synthetic workloads.

Every tensor is drawn from its own Philox stream keyed by (seed, tensor id), so one
layer's weights can be produced without producing any other layer's: the 32B-class
configuration never has to be resident on the host in full.

Weights: i.i.d. N(0, 0.02^2); stored [out_features][in_features]; rounded to bf16
(round-to-nearest-even) for the 16-bit configurations so that both consumers see the
same representable values ("f16" additionally rounds the bf16 values to float16, which
changes only magnitudes below 2^-17).  RMSNorm gains are 1.  Token ids are uniform on [0, vocab).
Unit lengths are uniform on the closed interval the configuration names.
"""
from __future__ import annotations

import dataclasses
import numpy as np

WEIGHT_STD = 0.02


@dataclasses.dataclass(frozen=True)
class ModelCfg:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str            # "f32" | "bf16" | "f16" (bf16-valued weights in float16 containers)
    rope_base: float = 1.0e4
    rms_eps: float = 1.0e-6

    @property
    def dq(self):
        return self.n_q_heads * self.head_dim

    @property
    def dkv(self):
        return self.n_kv_heads * self.head_dim


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    model: ModelCfg
    n_units: int
    len_lo: int
    len_hi: int           # inclusive
    n_query: int
    refresh_bp: tuple     # refresh ratios in basis points
    kv_format: str = "native"   # "native" | "q4" | "q2"


_M1 = ModelCfg("tiny", 2, 256, 4, 2, 64, 688, 4096, "f32")
_M2 = ModelCfg("3b", 36, 2048, 16, 2, 128, 11008, 32000, "bf16")
_M3 = ModelCfg("8b", 32, 4096, 32, 8, 128, 14336, 32000, "bf16")
_M4 = ModelCfg("32b", 64, 5120, 40, 8, 128, 27648, 32000, "bf16")

CONFIGS = {
    "c1": Workload("c1", _M1, 4, 64, 64, 32, (2500,)),
    "c2": Workload("c2", _M2, 20, 192, 320, 64, (1000, 2000, 3000)),
    "c3": Workload("c3", _M3, 32, 128, 384, 128, (1500,)),
    "c4": Workload("c4", _M4, 30, 384, 384, 128, (1000, 2000, 3000)),
    "c5q4": Workload("c5q4", _M3, 48, 256, 256, 128, (2000,), "q4"),
    "c5q2": Workload("c5q2", _M3, 48, 256, 256, 128, (2000,), "q2"),
    "c5fp8": Workload("c5fp8", _M3, 48, 256, 256, 128, (2000,), "fp8"),     # extra: configuration 5 with the FP8 cache
}


def workload(name: str) -> Workload:
    return CONFIGS[name]


def model_cfg(name: str) -> ModelCfg:
    return CONFIGS[name].model


def reduced(w: Workload, n_layers=None, n_units=None, len_lo=None, len_hi=None,
            n_query=None, dtype=None) -> Workload:
    """The same workload with fewer layers / units (full width), for fast parity runs."""
    m = w.model
    m2 = dataclasses.replace(m, n_layers=n_layers or m.n_layers, dtype=dtype or m.dtype)
    return dataclasses.replace(w, model=m2, n_units=n_units or w.n_units,
                               len_lo=len_lo or w.len_lo, len_hi=len_hi or w.len_hi,
                               n_query=n_query or w.n_query)


# ----------------------------------------------------------------------------- storage rounding

def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 values rounded to the nearest bf16-representable value, returned as fp32."""
    u = np.array(x, dtype=np.float32, copy=True).view(np.uint32)
    bias = u >> np.uint32(16)
    bias &= np.uint32(1)
    bias += np.uint32(0x7FFF)
    u += bias
    u &= np.uint32(0xFFFF0000)
    return u.view(np.float32)


# ----------------------------------------------------------------------------- streams

_TENSOR_IDS = {"tok_emb": 1, "wq": 2, "wk": 3, "wv": 4, "wo": 5, "w_gate": 6, "w_up": 7,
               "w_down": 8, "ids": 9, "lengths": 10, "query": 11}


def _rng(seed: int, what: str, index: int = 0) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | (_TENSOR_IDS[what] << 32) | (int(index) << 40)
    return np.random.Generator(np.random.Philox(key=key))


def _normal(seed, what, index, shape, dtype):
    w = _rng(seed, what, index).standard_normal(size=shape, dtype=np.float32)
    w *= np.float32(WEIGHT_STD)
    if dtype == "f32":
        return w
    w = bf16_round(w)                       # the configurations' weights are bf16 values
    if dtype == "f16":                      # held in float16 containers: exact for |w| >= 2^-17
        w = w.astype(np.float16).astype(np.float32)
    return w


def embedding(m: ModelCfg, seed: int) -> np.ndarray:
    """[vocab][d_model] fp32 values (bf16-representable when m.dtype == 'bf16')."""
    return _normal(seed, "tok_emb", 0, (m.vocab, m.d_model), m.dtype)


def layer_weights(m: ModelCfg, seed: int, layer: int) -> dict:
    """One decoder layer: projections stored [out][in]; norm gains all ones."""
    return {
        "attn_norm": np.ones(m.d_model, np.float32),
        "wq": _normal(seed, "wq", layer, (m.dq, m.d_model), m.dtype),
        "wk": _normal(seed, "wk", layer, (m.dkv, m.d_model), m.dtype),
        "wv": _normal(seed, "wv", layer, (m.dkv, m.d_model), m.dtype),
        "wo": _normal(seed, "wo", layer, (m.d_model, m.dq), m.dtype),
        "mlp_norm": np.ones(m.d_model, np.float32),
        "w_gate": _normal(seed, "w_gate", layer, (m.d_ff, m.d_model), m.dtype),
        "w_up": _normal(seed, "w_up", layer, (m.d_ff, m.d_model), m.dtype),
        "w_down": _normal(seed, "w_down", layer, (m.d_model, m.d_ff), m.dtype),
    }


def unit_lengths(w: Workload, seed: int) -> np.ndarray:
    return _rng(seed, "lengths").integers(w.len_lo, w.len_hi + 1, size=w.n_units).astype(np.int32)


def token_ids(w: Workload, seed: int, lengths: np.ndarray):
    """(context ids [sum lengths], query ids [n_query]), uniform on [0, vocab)."""
    ctx = _rng(seed, "ids").integers(0, w.model.vocab, size=int(lengths.sum())).astype(np.int32)
    qry = _rng(seed, "query").integers(0, w.model.vocab, size=w.n_query).astype(np.int32)
    return ctx, qry
