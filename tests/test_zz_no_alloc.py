"""akvs_op_select_static -- probe selection for callers that cannot allocate device memory
(fixed memory pools, allocation-free request paths): the scratch lives in an array inside
the library.  It must give exactly what akvs_op_select gives, call after call, although
every call reuses the same array and finds the previous call's contents in it.

Collected last on purpose: a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _same(akvs, dk, dv, off, nq, bp):
    ref = akvs.op_select(_dev(dk), _dev(dv), off, nq, bp)          # caller-provided scratch
    got = akvs.op_select_static(_dev(dk), _dev(dv), off, nq, bp)   # the library's own array
    torch.cuda.synchronize()
    N, M = int(off[-1]), len(off) - 1
    assert (got.n_ctx, got.n_probe_rows, got.n_rows) == (ref.n_ctx, ref.n_probe_rows, ref.n_rows)
    nP = int(ref.probe_off[M].item())
    for name, n in (("ctx_off", M + 1), ("probe_off", M + 1), ("sk_idx", nP), ("sv_idx", nP), ("rows", ref.n_rows),
                    ("w_k", N), ("w_v", N)):
        assert torch.equal(getattr(got, name)[:n], getattr(ref, name)[:n]), name
    return got


def test_static_select_matches_select_on_two_calls_in_a_row():
    import paper_2607_21604_b200 as akvs
    g = np.random.default_rng(42)
    # first call: a large request that fills most of the array
    lens = g.integers(128, 385, 48)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    N = int(off[-1])
    dk, dv = (g.random(N) * 3).astype(np.float32), (g.random(N) * 3).astype(np.float32)
    a = _same(akvs, dk, dv, off, 128, 2000)
    assert a.n_probe_rows > 0
    # second call right after it: smaller, other scores, heavy ties -- stale keys, flags and
    # counters of the first call are still in the array and must not leak into the result
    lens2 = np.array([5, 0, 64, 1, 300])
    off2 = np.concatenate([[0], np.cumsum(lens2)]).astype(np.int64)
    N2 = int(off2[-1])
    dk2 = (np.round(g.random(N2) * 4) / 4).astype(np.float32)
    dv2 = np.zeros(N2, np.float32)
    b = _same(akvs, dk2, dv2, off2, 0, 2500)
    assert b.n_rows == b.n_probe_rows < a.n_probe_rows
    # and the first request again gives the first answer again
    c = _same(akvs, dk, dv, off, 128, 2000)
    assert torch.equal(c.rows[:c.n_rows], a.rows[:a.n_rows])


def test_static_select_rejects_what_does_not_fit():
    import paper_2607_21604_b200 as akvs
    N = akvs.STATIC_MAX_CTX + 1
    d = torch.ones(N, dtype=torch.float32, device="cuda")
    with pytest.raises(akvs.AkvsError) as e:
        akvs.op_select_static(d, d, np.array([0, N]), 4, 1000)
    assert e.value.code == -8
    M = akvs.STATIC_MAX_UNITS + 1
    off = np.arange(M + 1)
    with pytest.raises(akvs.AkvsError) as e:
        akvs.op_select_static(d, d, off, 4, 1000)
    assert e.value.code == -8
    # exactly at the limit is accepted
    N = akvs.STATIC_MAX_CTX
    dk = torch.rand(N, device="cuda")
    _same(akvs, dk.cpu().numpy(), dk.flip(0).cpu().numpy().copy(), np.array([0, N // 2, N]), 1, 1500)
