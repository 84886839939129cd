#!/usr/bin/env python
"""Benchmark of the multi-tier verify step (tier -> slim pass -> full pass -> accept -> commit).

python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one verify_step call over one batch of seeded synthetic input; the metric is verified draft
tokens per second (B * N tokens pushed through the step, summed over GPUs).  With N > 1 (launched by
torchrun) every rank runs an independent replica: the path has no exchange step, so there is no
collective on the data path; ranks only meet at the timing barrier.

--impl reference times the CPU oracle (plain numpy, as it stands) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC, UNIT = "verify_step_tokens_per_s", "tokens/s"
HBM_NOMINAL_GBS = 8000.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def gemm_traffic(wl):
    """DRAM bytes (read + write) of the step's GEMM launches, from the ncu capture of the GEMM kernel at 7B layer
    shapes whose summary is kept under profiles/: per layer 105.8 + 34.1 + 185.6 + 95.5 MB, head 270.8 MB, captured on
    the 2-layer cut of the 7B workload and scaled by the number of layers (traffic is per launch and the launches
    are the same).  Only known for the 7B layer shapes."""
    if wl.name != "c2_7b":
        return None
    return int((105.8 + 34.1 + 185.6 + 95.5) * 1e6 * wl.shape.n_layers + 270.8e6)


# ---------------------------------------------------------------------------------------------
# CPU baseline: the oracle timed on a bounded sample
# ---------------------------------------------------------------------------------------------
def cpu_cores() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


class _OracleSample:
    """Oracle passes over the first 1 and 2 layers of the workload's model (fp32 arithmetic, all rows
    together), the tier rule and the accept walk.  One step of the full model is extrapolated as
    (L + L_s) * per_layer + 2 * fixed + accept, where per_layer = t(2 layers) - t(1 layer) and fixed =
    t(1 layer) - per_layer (embedding, final norm, output head)."""

    def __init__(self, wl):
        from synth import workloads as W
        from oracle import step
        self.W, self.wl = W, wl
        self.model = W.Model(wl, keep=True)
        for l in range(2):
            self.model.layer(l)
        for k in ("embed", "lm_head", "final_norm"):
            self.model.tensor(-1, k)
        self.si = W.step_inputs(wl)
        self.ctx = {(o, w): W.context_kv(wl, 0, o, w) for o in range(2) for w in range(2)} \
            if not wl.real_prefill and wl.ctx else None
        self.lo, self.hi = W.thresholds(wl)

    def _state(self):
        from oracle import step
        wl = self.wl
        if self.ctx is None:
            st = step.new_state(wl.shape, 2, wl.batch, wl.ctx + wl.rows, np.float32)
            st.lens[:] = 0
        else:
            st = step.new_state(wl.shape, 2, wl.batch, wl.ctx + wl.rows, np.float32, base_len=wl.ctx,
                                base_full=lambda o, w: self.ctx[(o, w)], base_slim=lambda o, w: self.ctx[(o, w)])
        st.pending[:] = self.si.pending
        return st

    def run(self) -> dict:
        from oracle import decoder, step, tiers
        wl, si = self.wl, self.si
        rows = step.block_rows(si.pending, si.draft_tok)
        t = {}
        for nl in (1, 2):
            st = self._state()
            t0 = time.perf_counter()
            logits = decoder.forward(self.model, wl.shape, range(nl), st.full, st.lens, rows, wl.parent, np.float32)
            t[nl] = time.perf_counter() - t0
        t0 = time.perf_counter()
        tier, _ = tiers.tier_rule(si.drafter_logits, si.draft_tok, si.prow, self.lo, self.hi)
        tiers.resolve(si.draft_tok, wl.parent, si.prow, tier, si.drafter_logits, logits, logits,
                      tiers.Params(mode=wl.mode, temperature=wl.temperature, seed=wl.seed))
        t_acc = time.perf_counter() - t0
        per_layer = max(t[2] - t[1], 1e-9)
        fixed = max(t[1] - per_layer, 0.0)
        t_step = (wl.shape.n_layers + wl.n_routed) * per_layer + 2 * fixed + t_acc
        return dict(t_step=t_step, per_layer=per_layer, fixed=fixed, accept=t_acc, measured=t[1] + t[2] + t_acc)


def oracle_sample_text(wl) -> str:
    return (f"oracle fp32 passes over 1 and 2 of the {wl.shape.n_layers} layers (all {wl.batch * wl.rows} rows, ctx "
            f"{wl.ctx}) + tier rule + accept walk; step time extrapolated as (L+L_s)*per_layer + 2*fixed + accept")


def run_reference(args, wl) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    samp = _OracleSample(wl)
    for _ in range(max(0, min(args.warmup, 1))):
        samp.run()
    ts = [samp.run()["t_step"] for _ in range(args.steps)]
    t = float(np.mean(ts))
    value = wl.batch * wl.n_nodes / t
    cores = cpu_cores()
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "batch": wl.batch, "ctx": wl.ctx, "draft_nodes": wl.n_nodes,
                       "routed_layers": wl.n_routed, "mode": wl.mode},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": oracle_sample_text(wl)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------------------------------------
# multi-replica aggregation (one process per GPU; replicas are independent, they meet only here)
# ---------------------------------------------------------------------------------------------
def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest replica's time: the job is done when the last rank is."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(world: int, batch: int, n_nodes: int, ms_per_step: float) -> float:
    """Verified draft tokens per second of the whole job: every replica pushes batch * n_nodes tokens per step."""
    return world * batch * n_nodes / (ms_per_step * 1e-3)


# ---------------------------------------------------------------------------------------------
# GPU arm
# ---------------------------------------------------------------------------------------------
def run_ours(args, wl) -> None:
    import torch
    from synth import workloads as W
    from paper_2606_12243_b200 import binding as vb
    from paper_2606_12243_b200 import roofline as RL
    from paper_2606_12243_b200.engine import Engine

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank is an independent replica with its own seed-shifted inputs (same shapes)
    eng = Engine(wl)
    si = W.step_inputs(wl, step=rank)
    eng.set_inputs(si)
    sl, fl = eng.logits_buffer(), eng.logits_buffer()
    res = vb.alloc_result(wl.batch, wl.n_nodes)
    len0, pend0 = eng.len.clone(), eng.pending.clone()
    stream = torch.cuda.current_stream()

    pkw = dict(conf_source=1, strict_break=1) if args.gate == "slim" else {}

    def one_step(i):
        eng.len.copy_(len0, non_blocking=True)            # bench-only: rewind the cache instead of refilling it
        eng.pending.copy_(pend0, non_blocking=True)
        vb.verify_step(eng.model, eng.cache, eng.draft, eng.params(step=i, **pkw), sl, fl, res)

    for i in range(args.warmup):
        one_step(i)
    barrier()
    assert vb.get_stats(eng.model).device_status == 0

    clocks = ClockSampler(local)
    if rank == 0:
        clocks.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    l0 = vb.launch_count()
    ev0.record(stream)
    for i in range(args.steps):
        one_step(i)
    ev1.record(stream)
    barrier()
    launches = vb.launch_count() - l0
    ms = ev0.elapsed_time(ev1)
    ms = max_over_ranks(ms, dist, "cuda")
    ms_step = ms / args.steps
    value = job_value(world, wl.batch, wl.n_nodes, ms_step)

    # second timed region with per-launch events: attributes time to kernel classes
    vb.set_timing(eng.model, True)
    for i in range(min(args.steps, 3)):
        one_step(i)
    timing = vb.get_timing(eng.model)
    vb.set_timing(eng.model, False)
    n_timed = min(args.steps, 3)

    # end to end: host buffers in, host result out, every step
    pin = lambda t: t.cpu().pin_memory()
    h_tok, h_logits, h_pend = pin(eng.draft_tok), pin(eng.drafter_logits), pin(pend0)
    h_out = torch.empty((wl.batch, wl.n_nodes + 1), dtype=torch.int32).pin_memory()
    h_ne = torch.empty((wl.batch,), dtype=torch.int32).pin_memory()
    h2d = h_tok.numel() * 4 + h_logits.numel() * 4 + h_pend.numel() * 4
    d2h = h_out.numel() * 4 + h_ne.numel() * 4

    def e2e_step(i):
        eng.len.copy_(len0, non_blocking=True)
        eng.draft_tok.copy_(h_tok, non_blocking=True)
        eng.drafter_logits.copy_(h_logits, non_blocking=True)
        eng.pending.copy_(h_pend, non_blocking=True)
        vb.verify_step(eng.model, eng.cache, eng.draft, eng.params(step=i, **pkw), sl, fl, res)
        h_out.copy_(res.out_tok, non_blocking=True)
        h_ne.copy_(res.n_emit, non_blocking=True)
        stream.synchronize()

    e2e_step(0)
    barrier()
    ev0.record(stream)
    for i in range(args.steps):
        e2e_step(i)
    ev1.record(stream)
    barrier()
    ms_e2e = ev0.elapsed_time(ev1)
    clk = clocks.stop() if rank == 0 else None          # sampled over all timed regions of this run
    ms_e2e = max_over_ranks(ms_e2e, dist, "cuda")
    e2e_value = job_value(world, wl.batch, wl.n_nodes, ms_e2e / args.steps)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    sb = RL.step_bytes(wl)
    # verify_step streams every layer's weights once and applies the routed layers to both row streams, so the
    # bytes its GEMM launches move are the "shared" figure; the two-separate-passes figure is reported beside it
    gemm_ms = timing["gemm"]["ms"] / n_timed
    gemm_gbs = sb["gemm_shared"] / 1e9 / (gemm_ms * 1e-3) if gemm_ms > 0 else 0.0
    step_gbs = sb["total_shared"] / 1e9 / (ms_step * 1e-3)
    step_gbs_sep = sb["total"] / 1e9 / (ms_step * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.shape.dtype,
        "data": "synthetic",
        "config": {"workload": wl.name, "batch": wl.batch, "ctx": wl.ctx, "draft_nodes": wl.n_nodes,
                   "routed_layers": wl.n_routed, "layers": wl.shape.n_layers, "mode": wl.mode, "gate": args.gate,
                   "l2": "inputs larger than L2: the step streams %.1f GB of weights" % (sb["gemm_shared"] / 1e9),
                   "replicas": world},
        "roofline": {"bound": "hbm", "kernel": "projection GEMMs (all launches of the step)",
                     "achieved": gemm_gbs, "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                     "unit": "GB/s", "frac": gemm_gbs / peak, "traffic": gemm_traffic(wl),
                     "algorithmic_bytes_per_step": sb["gemm_shared"], "ms_per_step": gemm_ms,
                     "launches_per_step": timing["gemm"]["launches"] // n_timed,
                     "note": "one CUDA-event pair per run of consecutive GEMM launches (the four projections between two "
                             "attention calls, which keep their programmatic overlap); the runs are cut off from the "
                             "attention kernels around them, so this is a lower bound on the untimed step"},
        "step_roofline": {"algorithmic_bytes": sb["total_shared"], "achieved_gbs": step_gbs,
                          "frac_of_measured": step_gbs / peak, "frac_of_8tbs": step_gbs / HBM_NOMINAL_GBS,
                          "algorithmic_bytes_two_separate_passes": sb["total"],
                          "achieved_gbs_two_separate_passes": step_gbs_sep,
                          "tensor_frac": sb["flops"] / (ms_step * 1e-3) / 1.67e15},
        "kernel_ms_per_step": {k: v["ms"] / n_timed for k, v in timing.items() if isinstance(v, dict)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "clocks": clk,
    }
    if world == 1 and not args.no_cpu_baseline:
        # the bounded sample, repeated until about ten seconds of CPU work are on the clock (at most 12 times)
        samp = _OracleSample(wl)
        runs, spent = [], 0.0
        while spent < 10.0 and len(runs) < 12:
            runs.append(samp.run())
            spent += runs[-1]["measured"]
        t_step = float(np.mean([r["t_step"] for r in runs]))
        line["cpu_baseline"] = {"value": wl.batch * wl.n_nodes / t_step, "unit": UNIT, "cores": cpu_cores(),
                                "kind": "oracle", "sample": oracle_sample_text(wl) + f"; mean of {len(runs)} repeats",
                                "seconds_measured": spent, "seconds_per_step_extrapolated": t_step}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_7b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gate", default="drafter", choices=["drafter", "slim"],
                    help="whose confidence sets the tiers: the drafter's (default, the configuration the metric is quoted on) "
                         "or the slim verifier's with a tier-1 acceptance ending the block (Algorithm 2 as printed)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from synth import workloads as W
    wl = W.get(args.workload)
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
