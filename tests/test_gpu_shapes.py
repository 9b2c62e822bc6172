"""A sweep of small models with awkward shapes through all modes against the oracle: GQA
group sizes that do not divide 128 (partly filled M tiles), one kv head, units of a single
token, one query token, refresh ratios at both ends, every check layer, permuted retrieval
orders.  Each case is seeded; the tensor-core paths (head_dim 128, float16) and the CUDA-core
paths (float, head_dim 64) both run."""
import numpy as np
import pytest

import testgen
from gpu_helpers import Case
from test_gpu_pipeline import _check_encode, _run_all_modes

pytestmark = pytest.mark.gpu

# (n_layers, d_model, n_q, n_kv, head_dim, d_ff, dtype, n_units, len_lo, len_hi, n_query, bp, check_layer, scale)
CASES = [
    (3, 256, 10, 2, 128, 512, "f16", 4, 1, 40, 1, 2500, 2, 4.0),     # g = 5, a single query token, 1-token units possible
    (2, 384, 6, 2, 128, 384, "f16", 3, 100, 140, 9, 500, 1, 4.0),    # g = 3, several key tiles, check layer 1, 5 %
    (3, 128, 2, 1, 128, 256, "f16", 6, 5, 60, 33, 10000, 3, 4.0),    # one kv head, every token a probe, last check layer
    (2, 256, 16, 2, 128, 512, "f16", 2, 130, 260, 17, 0, 2, 4.0),    # g = 8, no probes at all
    (3, 512, 4, 4, 128, 640, "f16", 5, 1, 3, 2, 5000, 2, 4.0),       # MHA (g = 1), tiny units
    (2, 256, 8, 2, 128, 512, "bf16", 4, 20, 50, 12, 3000, 2, 1.0),   # bf16 storage
    (2, 192, 6, 3, 64, 400, "f32", 4, 1, 30, 7, 2500, 2, 1.0),       # float, head_dim 64, g = 2
    (3, 256, 4, 1, 64, 304, "f32", 3, 17, 45, 1, 7500, 1, 1.0),      # float, one kv head, 75 %
]


@pytest.mark.parametrize("i", range(len(CASES)))
def test_awkward_shapes_all_modes(i):
    L, d, nq, nkv, hd, ff, dtype, n_units, lo, hi, n_query, bp, check_layer, scale = CASES[i]
    w = testgen.Workload(f"shape{i}", testgen.ModelCfg(f"shape{i}", L, d, nq, nkv, hd, ff, 300, dtype),
                         n_units, lo, hi, n_query, (bp,))
    order = list(np.random.default_rng(100 + i).permutation(n_units))
    case = Case(w, std_scale=scale, order=order)
    case.encode()
    units = case.oracle_units()
    _run_all_modes(case, bp, check_layer, units)
