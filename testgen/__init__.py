"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests.

This package only draws numbers (weights, token ids, unit lengths) and rounds them to
the storage type.  It contains none of the method's arithmetic.
"""
from .gen import (CONFIGS, ModelCfg, Workload, model_cfg, workload, layer_weights,
                  embedding, unit_lengths, token_ids, bf16_round, to_bf16_bits,
                  from_bf16_bits, reduced)

__all__ = ["CONFIGS", "ModelCfg", "Workload", "model_cfg", "workload", "layer_weights",
           "embedding", "unit_lengths", "token_ids", "bf16_round", "to_bf16_bits",
           "from_bf16_bits", "reduced"]
