"""The C-ABI library builds for sm_100a, loads without a GPU, exports every function the
header declares, and its host-side validation works (no kernels are launched here)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    import importlib.util
    spec = importlib.util.spec_from_file_location("akvs_build", os.path.join(ROOT, "paper_2607_21604_b200", "build.py"))
    build = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(build)                  # by path: importing the package needs the library built
    return C.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "akvs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(akvs_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported(lib):
    names = _declared()
    assert {"akvs_encode_units", "akvs_select_probes", "akvs_prefill_corrected", "akvs_free",
            "akvs_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_exports(lib):
    import paper_2607_21604_b200.binding as b
    assert sorted(b.EXPORTS) == _declared()


def _fake_model(b, L=2, d=256, nq=4, nkv=2, hd=64, f=688, vocab=4096, dtype=0):
    m = b.ModelDesc()
    m.n_layers, m.d_model, m.n_q_heads, m.n_kv_heads, m.head_dim, m.d_ff, m.vocab, m.dtype = L, d, nq, nkv, hd, f, vocab, dtype
    m.rope_base, m.rms_eps = 1e4, 1e-6
    m.tok_emb = m.final_norm = 0x1000                    # never dereferenced by the size query
    arr = (C.c_void_p * L)(*([0x1000] * L))
    for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"):
        setattr(m, n, C.cast(arr, C.POINTER(C.c_void_p)))
    m._keep = arr
    return m


def test_workspace_bytes_host_logic(lib):
    import paper_2607_21604_b200.binding as b
    m = _fake_model(b)
    out = C.c_int64(0)
    assert lib.akvs_workspace_bytes(C.byref(m), 256, 32, 4, 2, C.byref(out)) == 0
    base = out.value
    assert base > 288 * 256 * 4 * 2 and base % 256 == 0
    for args in ((512, 32, 4, 2), (256, 64, 4, 2), (256, 32, 8, 2)):
        assert lib.akvs_workspace_bytes(C.byref(m), *args, C.byref(out)) == 0 and out.value >= base
    assert lib.akvs_workspace_bytes(C.byref(m), 256, 32, 4, 1, C.byref(out)) == 0 and out.value < base
    assert lib.akvs_workspace_bytes(C.byref(m), 256, 32, 4, 3, C.byref(out)) == -1      # check layer > n_layers
    assert lib.akvs_workspace_bytes(C.byref(m), -1, 32, 4, 2, C.byref(out)) == -1
    assert lib.akvs_workspace_bytes(None, 256, 32, 4, 2, C.byref(out)) == -1
    m2 = _fake_model(b, hd=48)
    assert lib.akvs_workspace_bytes(C.byref(m2), 256, 32, 4, 1, C.byref(out)) == -4     # unsupported head_dim
    m3 = _fake_model(b, nq=5)
    assert lib.akvs_workspace_bytes(C.byref(m3), 256, 32, 4, 1, C.byref(out)) == -2     # 5 q heads over 2 kv heads
    lib.akvs_op_scratch_bytes.restype = C.c_int64
    assert lib.akvs_op_scratch_bytes(8192, 128, 32, 128) > 8192 * 18


def test_free_accepts_null(lib):
    lib.akvs_free.restype = None
    lib.akvs_free(None)
