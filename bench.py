#!/usr/bin/env python
"""Benchmark of the corrected selective-recompute prefill (one step = probe selection +
prefill of one request) on seeded synthetic memory-unit contexts.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--impl ours|reference]

Prints ONE JSON line.  `value` is context tokens prefilled per second with the unit cache
already resident in HBM; `e2e` is the same with the unit cache, ids and result crossing
PCIe inside the timed region.  `--impl reference` times the CPU oracle on a bounded sample.
N > 1 runs independent replicas (requests are independent; no data-path collective).
"""
import argparse
import ctypes as C
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import testgen  # noqa: E402

SEED_W, SEED_IDS, SEED_LEN = 1234, 1235, 1236
METRIC = "context tokens/s prefilled (corrected reuse, 15% refresh)"
UNIT = "tokens/s"
CHECK_LAYER = 2
# dram__bytes_read.sum + dram__bytes_write.sum per linear-layer launch (bytes), averaged over
# the four linear-layer launches of one selective layer, from one ncu --set full capture of a
# 3-layer run of this workload (algorithmic: 201 MB per launch)
GEMM_TRAFFIC_PER_LAUNCH = {"c3": 203.6e6}


def peaks():
    try:
        p = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        return {"hbm": p["hbm_gbs"], "tensor": p["bf16_tflops_sustained"], "src": "measured"}
    except Exception:
        return {"hbm": 6650.0, "tensor": 1400.0, "src": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.p, self.index, self.t0 = [], None, index, None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.p = None

    def _read(self):
        for line in self.p.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def mark(self):
        """The timed region starts now (the sampler itself was started earlier: nvidia-smi takes
        a few hundred ms to deliver its first line)."""
        deadline = time.time() + 2.0
        while self.p is not None and not self.rows and time.time() < deadline:
            time.sleep(0.02)
        self.t0 = time.time()

    def stop(self):
        if self.p is not None:
            self.p.terminate()
        t0 = self.t0 or 0.0
        inside = [r for t, r in self.rows if t >= t0]
        self.rows = inside if inside else [r for _, r in self.rows[-2:]]   # a region shorter than one sample period
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({names[i] for r in self.rows if len(r) >= 7 for i in range(4) if r[3 + i] == "Active"})
        busy = sorted(sm)[len(sm) // 2:] if sm else []
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def max_over_ranks(value, world, device="cuda"):
    """Multi-GPU numbers are the slowest rank's: all-reduce MAX over the process group."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(tokens_per_rank, world, ms):
    """Replicas: every rank prefills its own request; the job's rate is the sum over ranks
    divided by the slowest rank's time."""
    return world * tokens_per_rank / (ms * 1e-3)


class OracleSample:
    """The CPU oracle on a bounded sample of the workload, for the reference arm and the
    `cpu_baseline` object.

    The sample keeps the model's full width and the workload's FULL context (every unit, every
    context and query token), so the attention term that grows with the context is in it.  It is
    bounded in depth (the first min(3, L) layers: the dense layer, the check layer and one more
    selective layer) and in rows: the steps of the oracle's corrected reuse are called in its
    order on every `stride`-th row where the cost is per row,
      dense layer:      q/k/v projections of all T rows; attention, W_o, MLP of every sd-th row
      check layer:      k/v of all N context rows, re-aligned cache, scores, top-b selection
      selective layers: re-aligned cache and correction of all N tokens; projections, probe
                        offsets, attention, W_o, MLP of every ss-th probe row and all query rows
    (rows whose dense output was not computed enter the check layer with their embedding: the
    work is the same, the values are not, and nothing here is checked for values).  The time of
    the whole workload is extrapolated from the phases: per-row phases by rows / sampled rows,
    the selective layer by the number of selective layers.  One step = one pass over the sample."""

    def __init__(self, w):
        from oracle import akvs_oracle as orc
        self.orc, self.w = orc, w
        m = w.model
        self.L, self.L_s = m.n_layers, min(3, m.n_layers)
        ms = testgen.reduced(w, n_layers=self.L_s).model
        lens = testgen.unit_lengths(w, SEED_LEN)
        ctx, qry = testgen.token_ids(w, SEED_IDS, lens)
        off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        units_ids = [ctx[off[i]:off[i + 1]] for i in range(len(lens))]
        layers = [testgen.layer_weights(ms, SEED_W, l) for l in range(self.L_s)]
        self.model = orc.Model(ms, testgen.embedding(ms, SEED_W), layers)
        self.units = orc.encode_units(self.model, units_ids)          # precondition ("encoded once"), not timed
        self.order = list(range(len(lens)))
        self.ctx_off = off
        self.N, self.nq = len(ctx), len(qry)
        self.T = self.N + self.nq
        self.h0 = orc.embed(self.model, np.concatenate([ctx, qry]))
        self.bp = w.refresh_bp[0]
        self.sd = max(1, self.T // 256)
        self.rows_target = 256
        self.last = None

    def step(self):
        """One pass over the sample; returns its wall time in seconds and keeps the phase times."""
        orc, model, N, T = self.orc, self.model, self.N, self.T
        now = time.perf_counter
        allpos = np.arange(T)
        lc = CHECK_LAYER - 1
        c0 = now()
        q, k, v = orc.layer_qkv(model, 0, self.h0, allpos)
        c1 = now()
        D = allpos[::self.sd]
        a = orc.attention(q[D], k, v, D, allpos)
        hD = orc.layer_out(model, 0, self.h0[D], a)
        c2 = now()
        h_all = self.h0.copy()
        h_all[D] = hD
        _, k_chk, v_chk = orc.layer_qkv(model, lc, h_all[:N], allpos[:N])
        kr, vr = orc.reuse_kv(model, self.units, self.order, lc)
        d_k = orc.divergence_scores(k_chk, kr)
        d_v = orc.divergence_scores(v_chk, vr)
        probes = orc.select_probes(d_k, d_v, self.ctx_off, self.bp)
        c3 = now()
        rows_full = np.concatenate([probes["ctx_rows"], np.arange(N, T)]).astype(np.int64)
        R, nP = len(rows_full), len(probes["ctx_rows"])
        ss = max(1, -(-R // self.rows_target))
        keep = np.concatenate([np.arange(0, nP, ss), np.arange(nP, R)])     # every ss-th probe row, every query row
        rows = rows_full[keep]
        nPs = int((keep < nP).sum())
        sets = []
        for s_idx in (probes["sk_idx"], probes["sv_idx"]):       # the probe sets restricted to the carried rows
            s = s_idx[np.isin(s_idx, rows[:nPs])]
            sets.append((s, np.searchsorted(s, self.ctx_off)))
        h = h_all[rows]
        fixed, per_row = [], []
        for l in range(lc, self.L_s):
            f0 = now()
            kr, vr = orc.reuse_kv(model, self.units, self.order, l)
            f1 = now()
            q, k, v = orc.layer_qkv(model, l, h, rows)
            k_f, v_f = np.zeros_like(kr), np.zeros_like(vr)
            k_f[rows[:nPs]] = k[:nPs]
            v_f[rows[:nPs]] = v[:nPs]
            mu_k = orc.probe_offsets(k_f, kr, sets[0][0], sets[0][1])
            mu_v = orc.probe_offsets(v_f, vr, sets[1][0], sets[1][1])
            f2 = now()
            K = np.concatenate([orc.apply_correction(k_f, kr, sets[0][0], probes["w_k"], mu_k, self.ctx_off), k[nPs:]])
            V = np.concatenate([orc.apply_correction(v_f, vr, sets[1][0], probes["w_v"], mu_v, self.ctx_off), v[nPs:]])
            f3 = now()
            a = orc.attention(q, K, V, rows, allpos)
            h = orc.layer_out(model, l, h, a)
            f4 = now()
            fixed.append((f1 - f0) + (f3 - f2))
            per_row.append((f2 - f1) + (f4 - f3))
        end = now()
        n_sel = self.L - CHECK_LAYER + 1
        sel_layer = float(np.mean(fixed)) + float(np.mean(per_row)) * R / len(rows)
        dense_layer = (c1 - c0) + (c2 - c1) * T / len(D)
        self.last_hidden = orc.rmsnorm(h[nPs:], model.final_norm, model.cfg.rms_eps)   # for the test that pins the sample
        self.last = {"rows_recomputed": R, "rows_sampled": len(rows), "dense_rows_sampled": len(D),
                     "extrapolated_s": (CHECK_LAYER - 1) * dense_layer + (c3 - c2) + n_sel * sel_layer}
        return end - c0

    def describe(self):
        m, l = self.w.model, self.last
        return (f"oracle (float64 numpy) steps of corrected reuse, full width, full context ({self.N} ctx + {self.nq} "
                f"query tokens), layers 1-{self.L_s} of {m.n_layers}; dense layer: projections of all rows, attention + "
                f"MLP of {l['dense_rows_sampled']} of {self.T} rows; selective layers: correction of all tokens, "
                f"{l['rows_sampled']} of {l['rows_recomputed']} recomputed rows; whole-workload time extrapolated per phase")


def reference_arm(args, w):
    """Times `steps` passes over the oracle sample.  Returns (tokens/s of the whole workload from
    the extrapolated time, measured ms per sample step, extrapolated ms of the whole workload,
    cores, description)."""
    smp = OracleSample(w)
    times, extra = [], []
    for i in range(args.warmup + args.steps):
        t = smp.step()
        if i >= args.warmup:
            times.append(t)
            extra.append(smp.last["extrapolated_s"])
    full_s = float(np.mean(extra))
    return smp.T / full_s, float(np.mean(times)) * 1e3, full_s * 1e3, len(os.sched_getaffinity(0)), smp.describe()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--layers", type=int, default=0, help="debug: fewer layers (invalid as a result)")
    ap.add_argument("--dtype", default="f16", choices=["f16", "bf16"],
                    help="16-bit storage type of weights, cache and activations (weight VALUES are bf16 either way)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-switches", type=int, default=0,
                    help="comparisons: the library's cross-check switch word (bits 2-3: tiling of the linear layers; "
                         "bits 4-6: forced split-K count); recorded in config, 0 for any reported result")
    ap.add_argument("--no-variants", action="store_true", help="skip the pass with the other 16-bit storage type")
    ap.add_argument("--graph", action="store_true",
                    help="replay the corrected prefill from a CUDA graph captured once (selection stays eager)")
    ap.add_argument("--batch", type=int, default=1,
                    help="requests per call that share the model (each retrieves all units in its own order); "
                         "the metric's configuration is 1")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w = testgen.workload(args.workload)
    if w.model.dtype != "f32":
        w = testgen.reduced(w, dtype=args.dtype)
    if args.layers:
        w = testgen.reduced(w, n_layers=args.layers)
    m = w.model
    bp = w.refresh_bp[0]
    metric = METRIC if args.workload == "c3" else f"context tokens/s prefilled (corrected reuse, {bp / 100:g}% refresh)"

    if args.impl == "reference":
        if rank != 0:
            return
        val, ms_step, full_ms, cores, sample = reference_arm(args, w)
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name}: one step = one pass over the sample in cpu_baseline.sample; "
                                   "value = tokens of the whole workload / cpu_baseline.extrapolated_ms"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "sample_ms": ms_step, "extrapolated_ms": full_ms},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    import paper_2607_21604_b200 as akvs
    if args.kernel_switches:
        akvs.lib.akvs_debug_set_linear_algo(int(args.kernel_switches))

    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # ---------------------------------------------------------------- synthetic inputs
    t_setup = time.time()
    cores = len(os.sched_getaffinity(0))
    gmodel = akvs.Model.from_layer_fn(m, testgen.embedding(m, SEED_W), lambda l: testgen.layer_weights(m, SEED_W, l),
                                      n_threads=max(1, min(12, cores // max(1, world))))
    lens = testgen.unit_lengths(w, SEED_LEN)
    ctx_ids, qry_ids = testgen.token_ids(w, SEED_IDS, lens)
    kvf = {"native": akvs.KV_NATIVE, "q4": akvs.KV_Q4, "q2": akvs.KV_Q2, "fp8": akvs.KV_FP8}[w.kv_format]
    order = list(range(w.n_units))
    B = max(1, args.batch)
    N, nq, M = int(lens.sum()) * B, w.n_query * B, w.n_units * B
    T = N + nq
    if B == 1:
        pos_local = np.arange(T, dtype=np.float64)
    else:
        pos_local = np.concatenate([np.tile(np.arange(N // B), B), np.tile(N // B + np.arange(nq // B), B)]).astype(np.float64)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    pk = peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_times = []

    def timed(fn, steps, warmup):
        """Mean time per step over `steps` steps (max over ranks).  An event after every step also
        gives the single-step times of the last call (rank-local), for the median and the best."""
        for _ in range(warmup):
            fn()
        barrier()
        marks = [ev() for _ in range(steps + 1)]
        marks[0].record()
        for i in range(steps):
            fn()
            marks[i + 1].record()
        barrier()
        step_times[:] = [marks[i].elapsed_time(marks[i + 1]) for i in range(steps)]
        return max_over_ranks(marks[0].elapsed_time(marks[-1]), world) / steps

    class Pass:
        """Everything resident for one model (storage type): unit store, request, outputs, workspace."""

    def device_pass(gm):
        """Device-resident timing of one model.  The headline time comes from K plain steps.  The
        per-kernel figures of the roofline object come from K more steps of the same work with CUDA
        events around every linear-layer, attention, correction, norm and offset launch (the events
        sit between kernels, which keeps a kernel from being scheduled while its predecessor drains,
        so that pass is a little slower: its time is reported beside)."""
        ps = Pass()
        ps.gm = gm
        ps.store = akvs.UnitStore(gm, lens, ctx_ids, kvf)
        if B == 1:
            ps.req = akvs.Request(order, qry_ids)
        else:
            # every request retrieves the same units in its own order and asks its own question
            ps.req = akvs.Request.batch([([(u + 5 * b) % (M // B) for u in order], np.roll(qry_ids, 7 * b)) for b in range(B)])
        ps.ws = akvs.alloc_workspace(akvs.workspace_bytes(gm, N, nq, M, CHECK_LAYER))
        e0, e1 = ev(), ev()
        e0.record()
        akvs.encode_units(gm, ps.store, ps.ws)                  # precondition ("encoded once"), timed apart
        e1.record()
        torch.cuda.synchronize()
        assert akvs.check(ps.ws) == 0
        ps.encode_ms = e0.elapsed_time(e1)
        ps.probes = akvs.Probes(N, M, nq)
        ps.hid, ps.out_k, ps.out_v = akvs.alloc_outputs(gm, N, nq)
        ps.ctx = C.c_void_p()
        ps.graph, graph_launches = None, 0

        def step():
            akvs.select_probes(gm, ps.store, ps.req, bp, CHECK_LAYER, ps.probes, ps.ctx, ps.ws)
            if ps.graph is not None:
                ps.graph.replay()
            else:
                akvs.prefill_corrected(gm, ps.store, ps.req, ps.probes, akvs.MODE_CORRECTED, ps.hid, ps.out_k, ps.out_v,
                                       ps.ctx, ps.ws)
        ps.step = step

        sampler = ClockSampler(local)
        sampler.start()
        for _ in range(args.warmup):
            step()
        barrier()
        if args.graph:
            # the probe counts of this request are fixed (same inputs every step), so one capture serves
            side = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            n0 = akvs.launch_count()
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    akvs.prefill_corrected(gm, ps.store, ps.req, ps.probes, akvs.MODE_CORRECTED, ps.hid, ps.out_k,
                                           ps.out_v, ps.ctx, ps.ws)
            torch.cuda.synchronize()
            graph_launches = akvs.launch_count() - n0      # kernels recorded in the graph: replayed every step
            ps.graph = g
            step()
            barrier()
        launches0 = akvs.launch_count()
        sampler.mark()
        ps.ms_step = timed(step, args.steps, 0)
        ps.ms_median, ps.ms_best = float(np.median(step_times)), float(min(step_times))
        ps.launches = akvs.launch_count() - launches0 + graph_launches * args.steps
        # the per-kernel events are recorded at launch time, so this pass launches eagerly even when
        # the timed steps replayed a graph
        g_timed, ps.graph = ps.graph, None
        akvs.prof_enable((1 << 1) | (1 << 2) | (1 << 3) | (1 << 4) | (1 << 5), 8192)
        step()
        barrier()
        akvs.prof_reset()
        ms_step_prof = timed(step, args.steps, 0)
        ps.clocks = sampler.stop()
        recs = akvs.prof_read()
        akvs.prof_enable(0)
        ps.graph = g_timed
        assert akvs.check(ps.ws) == 0
        ps.P = ps.probes.n_probe_rows

        gemm = [r for r in recs if r[2] >> 8 == 1]
        corr = [r for r in recs if r[2] >> 8 == 2]
        attn = [r for r in recs if r[2] >> 8 == 3]
        norm = [r for r in recs if r[2] >> 8 == 4]
        offs = [r for r in recs if r[2] >> 8 == 5]
        g_ms = sum(r[0] for r in gemm)
        g_fl = sum(r[1] for r in gemm)
        by_epi = {}
        by_shape = {}
        for ms_, fl, sub in gemm:
            a_ = by_epi.setdefault(sub & 255, [0.0, 0.0, 0])
            a_[0] += ms_; a_[1] += fl; a_[2] += 1
            a_ = by_shape.setdefault((sub & 255, round(fl / 1e9, 1)), [0.0, 0.0, 0])
            a_[0] += ms_; a_[1] += fl; a_[2] += 1
        # attention flops of one step from the recomputed rows: 4 * dq * sum_r (keys visible to r);
        # the dense first layer sees every row, the selective layers the probe and query rows
        rows = ps.probes.rows[:ps.probes.n_rows].cpu().numpy()
        a_fl = 4.0 * m.dq * ((CHECK_LAYER - 1) * float((pos_local + 1).sum()) +
                             (m.n_layers - CHECK_LAYER + 1) * float((pos_local[rows] + 1).sum()))
        a_ms = sum(r[0] for r in attn) / args.steps
        c_ms = sum(r[0] for r in corr)
        c_by = sum(r[1] for r in corr)
        achieved = g_fl / (g_ms * 1e-3) / 1e12 if g_ms > 0 else 0.0
        hbm_nominal = 8000.0
        c_gbs = c_by / (c_ms * 1e-3) / 1e9 if c_ms > 0 else None
        ps.other = {
            "attention_tc_kernel": {"bound": "tensor", "tflops": a_fl / (a_ms * 1e-3) / 1e12 if a_ms > 0 else None,
                                    "frac": a_fl / (a_ms * 1e-3) / 1e12 / pk["tensor"] if a_ms > 0 else None,
                                    "ms_per_step": a_ms, "launches_per_step": len(attn) / args.steps},
            "correct_kernel": {"bound": "hbm", "gbs": c_gbs,
                               "frac": c_gbs / pk["hbm"] if c_gbs else None,
                               "frac_of_nominal_8tbs": c_gbs / hbm_nominal if c_gbs else None,
                               "how": "one launch between two events, inside the layer loop",
                               "ms_per_step": c_ms / args.steps, "launches_per_step": len(corr) / args.steps,
                               "bytes_per_launch": c_by / max(1, len(corr))},
            "rmsnorm_kernel": {"bound": "hbm", "gbs": sum(r[1] for r in norm) / (sum(r[0] for r in norm) * 1e-3) / 1e9
                               if norm else None, "ms_per_step": sum(r[0] for r in norm) / args.steps,
                               "launches_per_step": len(norm) / args.steps},
            "offsets_kernel": {"bound": "hbm/latency", "ms_per_step": sum(r[0] for r in offs) / args.steps,
                               "launches_per_step": len(offs) / args.steps}}
        ps.roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel + gemm_tc_pair_kernel (all linear layers of the step)",
                       "achieved": achieved, "peak": pk["tensor"], "unit": "TFLOP/s", "frac": achieved / pk["tensor"],
                       "frac_of_nominal_2250": achieved / 2250.0,
                       "peak_source": pk["src"] + " bf16 cuBLAS sustained (f16 and bf16 MMAs run at the same rate)",
                       "traffic": GEMM_TRAFFIC_PER_LAUNCH.get(args.workload) if B == 1 else None, "launches": len(gemm),
                       "share_of_step": g_ms / (ms_step_prof * args.steps), "instrumented_ms_per_step": ms_step_prof,
                       "by_epilogue": {{0: "qkv_store", 1: "residual", 2: "swiglu"}.get(k, str(k)):
                                       {"tflops": v[1] / (v[0] * 1e-3) / 1e12, "ms_per_step": v[0] / args.steps,
                                        "launches": v[2]} for k, v in sorted(by_epi.items())},
                       # one entry per distinct launch shape: epilogue kind, GFLOP per launch, us per launch, TFLOP/s
                       "by_shape": [{"epilogue": {0: "qkv_store", 1: "residual", 2: "swiglu"}.get(k[0], str(k[0])),
                                     "gflop": k[1], "us": 1e3 * v[0] / v[2], "tflops": v[1] / (v[0] * 1e-3) / 1e12,
                                     "launches": v[2]} for k, v in sorted(by_shape.items())]}
        return ps

    ps = device_pass(gmodel)
    setup_s = time.time() - t_setup
    store, req, probes, hid, out_k, out_v, ws, step = ps.store, ps.req, ps.probes, ps.hid, ps.out_k, ps.out_v, ps.ws, ps.step
    ms_step, P = ps.ms_step, ps.P
    R_ = argparse.Namespace(ms_median=ps.ms_median, ms_best=ps.ms_best, clocks=ps.clocks, launches=ps.launches,
                            roofline=ps.roofline, other=ps.other, encode_ms=ps.encode_ms)

    # the correction pass alone, back to back over distinct layers' buffers (no launch ramp between
    # events): the same kernel, inputs and outputs as in the step, one pair of events around all launches
    if B == 1:
        n_rep = m.n_layers - CHECK_LAYER + 1

        def corr_only():
            akvs.debug_correct_repeat(gmodel, store, req, probes, out_k, out_v, ps.ctx, ws)
        b2b_ms = timed(corr_only, 5, 2) / n_rep
        by = R_.other["correct_kernel"]["bytes_per_launch"]
        # calibration: a plain device-to-device copy moving the same number of bytes (half read,
        # half written), timed both ways over buffers cycled beyond the L2
        n_el = int(by // 4)
        srcs = [torch.empty(n_el, dtype=torch.float16, device="cuda").normal_() for _ in range(8)]
        dsts = [torch.empty_like(t) for t in srcs]
        for a_, b_ in zip(srcs, dsts):
            b_.copy_(a_)
        torch.cuda.synchronize()
        singles = []
        for rep in range(3):
            for a_, b_ in zip(srcs, dsts):
                x0, x1 = ev(), ev()
                x0.record(); b_.copy_(a_); x1.record()
                torch.cuda.synchronize()
                singles.append(x0.elapsed_time(x1))
        x0, x1 = ev(), ev()
        x0.record()
        for rep in range(3):
            for a_, b_ in zip(srcs, dsts):
                b_.copy_(a_)
        x1.record()
        torch.cuda.synchronize()
        copy_b2b = x0.elapsed_time(x1) / 24
        del srcs, dsts
        R_.other["correct_kernel"]["copy_of_the_same_bytes"] = {
            "what": "torch device-to-device copy of bytes_per_launch / 2, same two ways of timing",
            "single_launch_us": 1e3 * float(np.median(singles)), "single_launch_frac": by / (float(np.median(singles)) * 1e-3) / 1e9 / pk["hbm"],
            "back_to_back_us": 1e3 * copy_b2b, "back_to_back_frac": by / (copy_b2b * 1e-3) / 1e9 / pk["hbm"]}
        R_.other["correct_kernel"]["back_to_back"] = {
            "how": f"{n_rep} launches in a row over the layers' own cache and output buffers ({n_rep * by / 1e9:.2f} GB, "
                   "beyond the L2), one pair of events around them",
            "us_per_launch": 1e3 * b2b_ms, "gbs": by / (b2b_ms * 1e-3) / 1e9,
            "frac": by / (b2b_ms * 1e-3) / 1e9 / pk["hbm"], "frac_of_nominal_8tbs": by / (b2b_ms * 1e-3) / 1e9 / 8000.0}

    # the same build's full recompute, for context (not the metric)
    def full():
        akvs.prefill_corrected(gmodel, store, req, None, akvs.MODE_FULL, hid, out_k, out_v, None, ws)
    full_ms = timed(full, max(1, args.steps // 2), 1)

    # ---------------------------------------------------------------- end to end through host buffers
    pin = lambda t: t.cpu().pin_memory()
    h_k, h_v = pin(store.k), pin(store.v)
    h_km = pin(store.k_meta) if store.k_meta is not None else None
    h_vm = pin(store.v_meta) if store.v_meta is not None else None
    h_ids, h_q = pin(store.token_ids), pin(req.query_ids)
    h_out = torch.empty(hid.shape, dtype=hid.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (h_k, h_v, h_km, h_vm, h_ids, h_q) if t is not None)
    d2h = h_out.numel() * h_out.element_size()

    # The offloaded cache is streamed in layer by layer on a copy stream; each layer's event is
    # handed to the library, which waits for it right before it first reads that layer, so the
    # PCIe transfer overlaps the prefill.  Everything is still inside the timed region.
    copy_stream = torch.cuda.Stream()
    layer_events = [torch.cuda.Event() for _ in range(m.n_layers)]

    def step_e2e():
        main = torch.cuda.current_stream()
        copy_stream.wait_stream(main)                      # the previous step is done with the cache
        store.token_ids.copy_(h_ids, non_blocking=True)
        req.query_ids.copy_(h_q, non_blocking=True)
        with torch.cuda.stream(copy_stream):
            for l in range(m.n_layers):
                store.k[l].copy_(h_k[l], non_blocking=True)
                store.v[l].copy_(h_v[l], non_blocking=True)
                if h_km is not None:
                    store.k_meta[l].copy_(h_km[l], non_blocking=True)
                    store.v_meta[l].copy_(h_vm[l], non_blocking=True)
                layer_events[l].record(copy_stream)
        store.set_layer_events(layer_events)
        step()
        h_out.copy_(hid, non_blocking=True)
        main.synchronize()
    e2e_ms = timed(step_e2e, args.steps, 1)
    store.set_layer_events(None)
    akvs.free(ps.ctx)
    weight_gb = sum(p.numel() * p.element_size() for l in gmodel.layers for p in l.values()) / 1e9

    # ---------------------------------------------------------------- the other 16-bit storage type
    # The configurations say "bf16"; the headline runs their bf16-valued weights in float16
    # containers (the storage type that meets the 1e-2 parity bound at full depth).  The same
    # step with bfloat16 storage throughout, measured in the same invocation:
    variants = None
    other_dt = {"f16": "bf16", "bf16": "f16"}.get(m.dtype)
    if other_dt and not args.no_variants and weight_gb < 40 and B == 1 and not args.graph:
        del h_k, h_v, h_km, h_vm
        td = torch.bfloat16 if other_dt == "bf16" else torch.float16
        cfg2 = testgen.reduced(w, dtype=other_dt).model
        # bf16 values survive a float16 container (and back) exactly, so the conversion is exact
        layers2 = [{n: (t if "norm" in n else t.to(td)) for n, t in lw.items()} for lw in gmodel.layers]
        gm2 = akvs.Model(cfg2, gmodel.tok_emb.to(td), layers2, gmodel.final_norm, akvs.BF16 if other_dt == "bf16" else akvs.F16)
        del ps, store, probes, hid, out_k, out_v, ws, step, full
        torch.cuda.empty_cache()
        p2 = device_pass(gm2)
        akvs.free(p2.ctx)
        variants = {other_dt: {
            "value": whole_job_rate(T, world, p2.ms_step), "unit": UNIT, "ms_per_step": p2.ms_step,
            "ms_per_step_median": p2.ms_median, "linear_layers_frac": p2.roofline["frac"],
            "linear_layers_tflops": p2.roofline["achieved"],
            "attention_frac": p2.other["attention_tc_kernel"]["frac"],
            "correct_kernel_frac": p2.other["correct_kernel"]["frac"], "clocks": p2.clocks,
            "dtype": f"{other_dt} storage (weights, cache, activations, K/V outputs), f32 accumulate"}}

    if world > 1:
        dist.barrier()                     # every rank is past its last collective before any of them leaves
        dist.destroy_process_group()
    if rank != 0:
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        a2 = argparse.Namespace(steps=1, warmup=0)
        val, sample_ms, full_ms_cpu, ccores, sample = reference_arm(a2, w)
        cpu = {"value": val, "unit": UNIT, "cores": ccores, "kind": "oracle", "sample": sample,
               "sample_ms": sample_ms, "extrapolated_ms": full_ms_cpu}
    out = {
        "metric": metric, "value": whole_job_rate(T, world, ms_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_median": R_.ms_median,
        "ms_per_step_best": R_.ms_best, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": {"f16": "f16 storage (bf16-valued random-init weights), f32 accumulate",
                  "bf16": "bf16 storage, f32 accumulate", "f32": "f32"}[m.dtype],
        "data": "synthetic",
        "config": {"workload": f"{w.name}: {m.name}-class decoder L{m.n_layers} d{m.d_model} {m.n_q_heads}q/{m.n_kv_heads}kv "
                               f"hd{m.head_dim} ff{m.d_ff}; {M // B} units {w.len_lo}-{w.len_hi} tok (N={N // B}) + {nq // B} query"
                               + (f", batch of {B} requests per call" if B > 1 else ""),
                   "batch": B, "cuda_graph": bool(args.graph), "kernel_switches": int(args.kernel_switches),
                   "refresh_bp": bp, "check_layer": CHECK_LAYER, "probe_rows": P, "rows_recomputed": P + nq,
                   "effective_refresh": P / max(1, N), "kv_format": w.kv_format, "parallelism": f"replicas x{world}",
                   "l2": f"inputs larger than L2: each step streams all layer weights ({weight_gb:.1f} GB)",
                   "seeds": [SEED_W, SEED_IDS, SEED_LEN]},
        "clocks": R_.clocks,
        "e2e": {"value": whole_job_rate(T, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "what": "unit cache + ids from pinned host memory each step (streamed per layer on a copy "
                        "stream, the library waits per layer), query hidden state back"},
        "gpu_launches": int(R_.launches),
        "roofline": R_.roofline,
        "other_kernels": R_.other,
        "dtype_variants": variants,
        "cpu_baseline": cpu,
        "context": {"full_recompute_ms": full_ms, "speedup_vs_full_recompute": full_ms / ms_step,
                    "encode_units_ms": R_.encode_ms, "setup_s": setup_s,
                    "paper_speedup_range_other_hw": "2-3.5x over no reuse at r=10-30% (A100/H200)"},
    }
    print(json.dumps(out))


if __name__ == "__main__":
    main()
