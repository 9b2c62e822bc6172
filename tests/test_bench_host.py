"""Host-side logic of the benchmark that needs no GPU: the reference arm on a tiny workload,
rank handling under a multi-process launch, and the max-over-ranks reduction (gloo, 2 ranks)."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _run(args, env_extra=None):
    env = dict(os.environ)
    env.update(env_extra or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, capture_output=True, text=True,
                          env=env, timeout=600)


def test_reference_arm_prints_contract_line_on_tiny_config():
    r = _run(["--impl", "reference", "--workload", "c1", "--steps", "1", "--warmup", "0"])
    assert r.returncode == 0, r.stderr[-2000:]
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert d["higher_is_better"] is True and d["vs_baseline"] is None


def test_reference_arm_runs_on_rank_zero_only():
    r = _run(["--impl", "reference", "--workload", "c1", "--steps", "1", "--warmup", "0"],
             {"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, device="cpu")
    rate = bench.whole_job_rate(1000, world, ms)
    dist.barrier()
    if rank == 0:
        out.put((ms, rate))
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_processes():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29531, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, rate = out.get(timeout=120)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert ms == 20.0                       # the slowest rank decides
    assert rate == pytest.approx(2 * 1000 / 0.020)


def test_oracle_sample_is_the_oracles_corrected_reuse_when_nothing_is_skipped():
    """On the tiny configuration the bounded sample skips no row and no layer, so the steps it
    strings together must reproduce the oracle's corrected reuse."""
    import numpy as np
    import bench
    import testgen
    from oracle import akvs_oracle as orc
    w = testgen.workload("c1")
    smp = bench.OracleSample(w)
    smp.step()
    assert smp.last["rows_sampled"] == smp.last["rows_recomputed"] and smp.last["dense_rows_sampled"] == smp.T
    ctx = np.concatenate([np.asarray(testgen.token_ids(w, bench.SEED_IDS, testgen.unit_lengths(w, bench.SEED_LEN))[0])])
    qry = testgen.token_ids(w, bench.SEED_IDS, testgen.unit_lengths(w, bench.SEED_LEN))[1]
    ref = orc.corrected_reuse(smp.model, smp.units, smp.order, ctx, qry, smp.bp, bench.CHECK_LAYER)
    assert np.allclose(smp.last_hidden, ref["hidden"], rtol=0, atol=1e-12)
    assert smp.last["extrapolated_s"] > 0
