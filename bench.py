#!/usr/bin/env python
"""Benchmark of the multi-tier verify step (tier -> slim pass -> full pass -> accept -> commit).

python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--no-sweep]

One step = one viasd_verify_step call over one batch of seeded synthetic input; the metric is verified draft
tokens per second (B * N tokens pushed through the step, summed over GPUs).  The default workload is the
8B-shaped model at batch 1 with the 26-node draft tree (the configuration the >= 70 % roofline target is
stated on).  Besides the headline the one JSON line carries
  per_call : each C-ABI call of the path timed on its own (median / min, GB/s, fraction of the roofline),
  sweep    : the other benchmark configurations (7B, 8B at batch 4, 13B, 32B at batch 1 and 16 with 16 / 32 /
             48 of 64 layers routed) with the slim pass charted against the routed fraction,
  roofline, cpu_baseline, e2e, clocks as the harness expects them.
With N > 1 (launched by torchrun) every rank runs an independent replica: the path has no exchange step,
so there is no collective on the data path; ranks only meet at the timing barrier.

--impl reference times the CPU oracle (plain numpy, as it stands) on the host cores instead: whole oracle
steps while they fit the time budget, otherwise a bounded sample of layers (labelled as extrapolated).
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
DEFAULT_WORKLOAD = "c3_8b_tree_b1"
SWEEP = ["c2_7b", "c3_8b_tree", "c4_13b"] + [f"c5_32b_b{b}_r{r}" for b in (1, 16) for r in (16, 32, 48)]
REFERENCE_BUDGET_S = 150.0          # CPU seconds the reference arm may spend on timed oracle steps
CPU_BASELINE_BUDGET_S = 12.0        # ... and the cpu_baseline leg of the GPU arm (at least one step)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops", 1590.0)), "measured"
    return 6650.0, 1590.0, "fallback"


# ---------------------------------------------------------------------------------------------
# CPU oracle, timed as it stands
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


def _host_bytes_free() -> int:
    try:
        import psutil
        return int(psutil.virtual_memory().available)
    except Exception:
        return 16 << 30


class OracleRunner:
    """The oracle's verify step (fp32 arithmetic, both passes, tier rule, accept walk) on the workload's inputs.

    whole = True: the whole model is generated up front (untimed) and one run() is one complete oracle step.
    whole = False (the model and its committed context do not fit the host's memory): run() passes the first
    1 and 2 layers plus the head, and the step is extrapolated as (L + L_s) * per_layer + 2 * fixed + accept.
    """

    def __init__(self, wl):
        from synth import workloads as W
        self.W, self.wl = W, wl
        s = wl.shape
        model_bytes = (s.n_layers * s.layer_params + 2 * s.vocab * s.d_model) * s.elem_bytes
        ctx_bytes = 0 if wl.real_prefill else \
            2 * (s.n_layers + wl.n_routed) * wl.batch * s.n_kv_heads * wl.ctx * s.head_dim * s.elem_bytes
        # fp32 copies of one layer and of the committed context of two layers are made inside the oracle
        self.whole = 1.25 * (model_bytes + ctx_bytes) + (8 << 30) < _host_bytes_free()
        n_keep = s.n_layers if self.whole else 2
        self.model = W.Model(wl, keep=True)
        for l in range(n_keep):
            self.model.layer(l)
        for k in ("embed", "lm_head", "final_norm"):
            self.model.tensor(-1, k)
        self.si = W.step_inputs(wl)
        self.lo, self.hi = W.thresholds(wl)
        self.ctx = None
        if not wl.real_prefill and wl.ctx:
            nf, ns = (s.n_layers, wl.n_routed) if self.whole else (2, 2)
            self.ctx = {(c, o, w): W.context_kv(wl, c, o, w) for c, n in ((0, nf), (1, ns)) for o in range(n)
                        for w in range(2)}
        self.prompt = None
        if wl.real_prefill:
            self.prompt = np.concatenate([self.si.prompt, self.si.pending[:, None]], axis=1)

    def _state(self, n_slim):
        from oracle import step
        wl = self.wl
        if self.ctx is None:
            return step.new_state(wl.shape, n_slim, wl.batch, wl.ctx + wl.rows, np.float32)
        st = step.new_state(wl.shape, n_slim, wl.batch, wl.ctx + wl.rows, np.float32, base_len=wl.ctx,
                            base_full=lambda o, w: self.ctx[(0, o, w)], base_slim=lambda o, w: self.ctx[(1, o, w)])
        st.pending[:] = self.si.pending
        return st

    def describe(self) -> str:
        wl = self.wl
        if self.whole:
            return (f"whole oracle verify step in fp32 (slim pass over {wl.n_routed} layers, full pass over "
                    f"{wl.shape.n_layers}, tier rule, accept walk, commit; all {wl.batch * wl.rows} rows, ctx {wl.ctx}); "
                    "weights and committed context generated beforehand, untimed")
        return (f"oracle fp32 passes over 1 and 2 of the {wl.shape.n_layers} layers (all {wl.batch * wl.rows} rows, ctx "
                f"{wl.ctx}) + tier rule + accept walk; the model does not fit this host's memory, so the step time is "
                "extrapolated as (L+L_s)*per_layer + 2*fixed + accept")

    def run(self) -> dict:
        """Returns seconds spent (measured) and seconds per step (t_step; equal to measured when whole)."""
        from oracle import decoder, step, tiers
        wl, si = self.wl, self.si
        P = tiers.Params(mode=wl.mode, temperature=wl.temperature, seed=wl.seed)
        if self.whole:
            st = self._state(wl.n_routed)
            if self.prompt is not None:
                step.prefill(self.model, wl.shape, wl.routed, st, self.prompt, np.float32)      # untimed: the context
            t0 = time.perf_counter()
            step.verify_step(self.model, wl.shape, wl.routed, st, si.draft_tok, wl.parent, si.prow, si.drafter_logits,
                             self.lo, self.hi, P, dt=np.float32)
            t = time.perf_counter() - t0
            return dict(t_step=t, measured=t)
        rows = step.block_rows(si.pending, si.draft_tok)
        t = {}
        for nl in (1, 2):
            st = self._state(2)
            t0 = time.perf_counter()
            logits = decoder.forward(self.model, wl.shape, range(nl), st.full, st.lens, rows, wl.parent, np.float32)
            t[nl] = time.perf_counter() - t0
        t0 = time.perf_counter()
        tier, _ = tiers.tier_rule(si.drafter_logits, si.draft_tok, si.prow, self.lo, self.hi)
        tiers.resolve(si.draft_tok, wl.parent, si.prow, tier, si.drafter_logits, logits, logits, P)
        t_acc = time.perf_counter() - t0
        per_layer = max(t[2] - t[1], 1e-9)
        fixed = max(t[1] - per_layer, 0.0)
        t_step = (wl.shape.n_layers + wl.n_routed) * per_layer + 2 * fixed + t_acc
        return dict(t_step=t_step, measured=t[1] + t[2] + t_acc)


def time_oracle(wl, budget_s: float, max_runs: int):
    """Runs the oracle until budget_s of CPU time is on the clock (at least once, at most max_runs times)."""
    orc = OracleRunner(wl)
    runs, spent = [], 0.0
    while not runs or (spent + runs[-1]["measured"] <= budget_s and len(runs) < max_runs):
        runs.append(orc.run())
        spent += runs[-1]["measured"]
    return orc, runs, spent


def config_of(wl, **extra) -> dict:
    c = {"workload": wl.name, "batch": wl.batch, "ctx": wl.ctx, "draft_nodes": wl.n_nodes, "layers": wl.shape.n_layers,
         "routed_layers": wl.n_routed, "mode": wl.mode}
    c.update(extra)
    return c


def run_reference(args, wl) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    orc, runs, spent = time_oracle(wl, REFERENCE_BUDGET_S, max(1, args.steps))
    t_step = float(np.mean([r["t_step"] for r in runs]))
    t_meas = float(np.mean([r["measured"] for r in runs]))
    value = wl.batch * wl.n_nodes / t_step
    cores = cpu_cores()
    sample = orc.describe() + f"; {len(runs)} timed runs of the {args.steps} asked for ({spent:.1f} s of a " \
                              f"{REFERENCE_BUDGET_S:.0f} s budget), no warm-up runs"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(runs), "warmup": 0, "steps_requested": args.steps, "warmup_requested": args.warmup,
            "ms_per_step": t_meas * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_of(wl, gate=args.gate, replicas=1),
            "extrapolated": not orc.whole,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "extrapolated": not orc.whole, "seconds_measured": spent,
                             "seconds_per_step": t_step},
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
class Bench:
    """One workload resident in HBM and the five calls of the path, each timed with CUDA events on the stream
    the library launches on."""

    def __init__(self, wl, rank: int = 0, gate: str = "drafter", weights_from=None, fill_context=True, **engine_kw):
        import torch
        from synth import workloads as W
        from paper_2606_12243_b200 import binding as vb
        from paper_2606_12243_b200.engine import Engine
        self.torch, self.vb, self.wl = torch, vb, wl
        self.eng = Engine(wl, weights_from=weights_from.eng if weights_from is not None else None,
                          fill_context=fill_context, **engine_kw)
        self.eng.set_inputs(W.step_inputs(wl, step=rank))      # every rank: its own seed-shifted inputs, same shapes
        self.sl, self.fl = self.eng.logits_buffer(), self.eng.logits_buffer()
        self.res = vb.alloc_result(wl.batch, wl.n_nodes)
        self.len0, self.pend0 = self.eng.len.clone(), self.eng.pending.clone()
        self.stream = torch.cuda.current_stream()
        self.pkw = dict(conf_source=1, strict_break=1) if gate == "slim" else {}

    def rewind(self):
        # bench-only: the cache is rewound instead of refilled (rollback is "do not keep the rows")
        self.eng.len.copy_(self.len0, non_blocking=True)
        self.eng.pending.copy_(self.pend0, non_blocking=True)

    def params(self, i):
        return self.eng.params(step=i, **self.pkw)

    def verify_step(self, i):
        e = self.eng
        self.rewind()
        self.vb.verify_step(e.model, e.cache, e.draft, self.params(i), self.sl, self.fl, self.res)

    def full_forward(self, i):
        e = self.eng
        self.vb.full_forward(e.model, e.cache, e.draft, self.fl)

    def slim_forward(self, i):
        e = self.eng
        self.vb.slim_forward(e.model, e.cache, e.draft, self.sl)

    def tier_accept(self, i):
        e = self.eng
        self.vb.tier_accept(e.model, e.draft, self.params(i), self.sl, self.fl, 3, self.res)

    def kv_commit(self, i):
        e = self.eng
        self.vb.kv_commit(e.model, e.cache, e.draft, self.res)

    def time_each(self, fn, n: int, warmup: int = 3):
        """n individually timed calls (one event pair each; the cache is rewound before each, outside the pair)
        -> (median ms, min ms)."""
        torch = self.torch
        for i in range(warmup):
            self.rewind()
            fn(i)
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        torch.cuda.synchronize()
        for i, (a, b) in enumerate(ev):
            self.rewind()
            a.record(self.stream)
            fn(i)
            b.record(self.stream)
        torch.cuda.synchronize()
        ms = sorted(a.elapsed_time(b) for a, b in ev)
        return float(np.median(ms)), float(ms[0])

    def status_ok(self) -> bool:
        return self.vb.get_stats(self.eng.model).device_status == 0


def call_record(ms_med: float, ms_min: float, nbytes, peak: float, flops=None, tf_peak=None) -> dict:
    r = {"ms_median": ms_med, "ms_min": ms_min}
    if nbytes:
        gbs = nbytes / 1e9 / (ms_med * 1e-3)
        r.update({"algorithmic_bytes": int(nbytes), "gbs": gbs, "frac_of_measured": gbs / peak,
                  "frac_of_8tbs": gbs / HBM_NOMINAL_GBS})
    if flops and tf_peak:
        r["tensor_frac"] = flops / (ms_med * 1e-3) / (tf_peak * 1e12)
    return r


def per_call(b: Bench, n: int, peak: float, tf_peak: float) -> dict:
    from paper_2606_12243_b200 import roofline as RL
    sb = RL.step_bytes(b.wl)
    cb = RL.call_bytes(b.wl)
    out = {}
    b.verify_step(0)                                    # leaves logits and a result for the later calls
    for name, fn, nbytes, flops in (("verify_step", b.verify_step, sb["total_shared"], sb["flops"]),
                                    ("full_forward", b.full_forward, sb["full"]["total"], sb["full"]["flops"]),
                                    ("slim_forward", b.slim_forward, sb["slim"]["total"], sb["slim"]["flops"]),
                                    ("tier_accept", b.tier_accept, cb["tier_accept"], None),
                                    ("kv_commit", b.kv_commit, cb["kv_commit"], None)):
        med, mn = b.time_each(fn, n)
        out[name] = call_record(med, mn, nbytes, peak, flops, tf_peak)
    return out


def graph_replay(b: Bench, n: int) -> dict:
    """The same verify step captured once into a CUDA graph (the library's launches are capturable: caller's stream
    only, no synchronisation, no allocation) and replayed: what the host-side launch cost of the ~170 kernels is worth."""
    torch = b.torch
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            b.verify_step(0)
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            b.verify_step(0)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(n):
            g.replay()
        ev1.record()
        torch.cuda.synchronize()
        return {"ms_per_step": ev0.elapsed_time(ev1) / n, "steps": n, "device_status_ok": b.status_ok()}
    except Exception as e:                                       # a bench key, not a requirement of the path
        return {"error": repr(e)[:200]}


def run_routed_policy(weights_from: Bench, n_steps: int = 48, replay: int = 18) -> dict:
    """Decoding loops of n_steps verify steps on the 7B-shaped workload with thresholds at the 5th / 50th percentile
    of drafter confidence (most drafted tokens in tiers 0 and 1), once with both passes in every step (policy 0) and
    once with routed execution (policy 1: the full verifier only when the walk needs it, up to `replay` committed
    tokens replayed when it does).  Eight input sets, resident on the device, are used in turn; the cache grows as
    tokens are committed.  Reports ms per step of each loop and the share of steps in which the full verifier ran."""
    import torch
    from synth import workloads as W
    from paper_2606_12243_b200 import binding as vb
    wl = W.get("c2_7b_routed")
    out = {"config": config_of(wl, replay_rows=replay, steps=n_steps)}
    for policy in (0, 1):
        b = Bench(wl, weights_from=weights_from, fill_context="device", max_query=wl.rows + replay,
                  extra_ctx=(n_steps + 4) * wl.rows)
        e = b.eng
        sets = []
        for k in range(8):
            e.set_inputs(W.step_inputs(wl, step=k), set_pending=(k == 0))
            sets.append(e.draft)
        torch.cuda.synchronize()

        def loop(n, first):
            for i in range(n):
                vb.verify_step(e.model, e.cache, sets[(first + i) % 8], e.params(step=first + i, policy=policy), b.sl, b.fl, b.res)

        loop(4, 0)                                              # warm-up steps, committed like the rest
        torch.cuda.synchronize()
        s0 = vb.get_stats(e.model)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(b.stream)
        loop(n_steps, 4)
        ev1.record(b.stream)
        torch.cuda.synchronize()
        s1 = vb.get_stats(e.model)
        skipped = int(s1.full_skipped - s0.full_skipped)
        out[f"policy_{policy}"] = {"ms_per_step": ev0.elapsed_time(ev1) / n_steps,
                                   "full_pass_share": (n_steps - skipped) / n_steps,
                                   "tokens_emitted_per_step": float(s1.emitted - s0.emitted) / n_steps,
                                   "tier_share": [float(s1.tier_count[i] - s0.tier_count[i]) /
                                                  max(1.0, float(sum(s1.tier_count) - sum(s0.tier_count))) for i in range(3)],
                                   "device_status_ok": s1.device_status == 0}
        del b, e, sets
    out["speedup_of_policy_1"] = out["policy_0"]["ms_per_step"] / out["policy_1"]["ms_per_step"]
    return out


def run_sweep(main: Bench, peak: float, tf_peak: float, n: int) -> dict:
    """The other benchmark configurations, one after the other (weights of a model shape are uploaded once and
    shared by its workloads; committed context drawn on the device): step, full pass and slim pass each."""
    import gc
    import torch
    from synth import workloads as W
    from paper_2606_12243_b200 import roofline as RL
    out, holder = {}, None          # holder: the engine whose weights the current model shape's workloads share
    t_begin = time.perf_counter()
    for name in SWEEP:
        wl = W.get(name)
        key = (wl.shape, wl.seed)
        if (main.wl.shape, main.wl.seed) == key:
            share = main
        elif holder is not None and (holder.wl.shape, holder.wl.seed) == key:
            share = holder
        else:
            share = holder = None
            gc.collect()
            torch.cuda.empty_cache()
        b = Bench(wl, weights_from=share, fill_context="device")
        sb = RL.step_bytes(wl)
        rec = {"config": config_of(wl)}
        step_bytes = sb["total_shared"] if 2 * wl.batch * wl.rows <= 128 else sb["total"]
        for cname, fn, nbytes, flops in (("verify_step", b.verify_step, step_bytes, sb["flops"]),
                                         ("full_forward", b.full_forward, sb["full"]["total"], sb["full"]["flops"]),
                                         ("slim_forward", b.slim_forward, sb["slim"]["total"], sb["slim"]["flops"])):
            med, mn = b.time_each(fn, n)
            rec[cname] = call_record(med, mn, nbytes, peak, flops, tf_peak)
        rec["verified_tokens_per_s"] = wl.batch * wl.n_nodes / (rec["verify_step"]["ms_median"] * 1e-3)
        rec["device_status_ok"] = b.status_ok()
        out[name] = rec
        if name == "c2_7b":
            out["routed_policy_7b"] = run_routed_policy(b)
        if share is None:
            holder = b
        del b
        gc.collect()
        torch.cuda.empty_cache()
    holder = None
    gc.collect()
    torch.cuda.empty_cache()
    # slim pass against routed fraction on the 32B-shaped model (64 layers; the full pass is the 64-layer point):
    # least-squares line t = head + per_layer * n_layers through the four points of each batch size
    chart = {}
    for bsz in (1, 16):
        pts = [(r, out[f"c5_32b_b{bsz}_r{r}"]["slim_forward"]["ms_median"]) for r in (16, 32, 48)]
        pts.append((64, out[f"c5_32b_b{bsz}_r16"]["full_forward"]["ms_median"]))
        x, y = np.array([p[0] for p in pts], dtype=np.float64), np.array([p[1] for p in pts])
        slope, icpt = np.polyfit(x, y, 1)
        chart[f"batch_{bsz}"] = {
            "routed_layers": [int(v) for v in x], "pass_ms": [float(v) for v in y],
            "ms_per_layer": float(slope), "ms_head_and_fixed": float(icpt),
            "pass_ms_minus_head_over_routed_fraction": [float((v - icpt) / (r / 64.0)) for r, v in pts],
            "max_rel_deviation_from_line": float(np.max(np.abs(y - (icpt + slope * x)) / y))}
    out["slim_vs_routed_fraction_32b"] = chart
    out["seconds"] = time.perf_counter() - t_begin
    return out


def run_ours(args, wl) -> None:
    import torch
    from paper_2606_12243_b200 import binding as vb
    from paper_2606_12243_b200 import roofline as RL

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

    b = Bench(wl, rank=rank, gate=args.gate)
    eng, stream = b.eng, b.stream
    for i in range(args.warmup):
        b.verify_step(i)
    barrier()
    assert b.status_ok()

    clocks = ClockSampler(local)
    if rank == 0:
        clocks.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    l0 = vb.launch_count()
    ev0.record(stream)
    for i in range(args.steps):
        b.verify_step(i)
    ev1.record(stream)
    barrier()
    launches = vb.launch_count() - l0
    ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    ms_step = ms / args.steps
    value = job_value(world, wl.batch, wl.n_nodes, ms_step)

    # second timed region with one event pair per run of launches of a kernel class
    n_timed = min(args.steps, 5)
    vb.set_timing(eng.model, True)
    for i in range(n_timed):
        b.verify_step(i)
    timing = vb.get_timing(eng.model)
    vb.set_timing(eng.model, False)

    # end to end: host buffers in, host result out, every step
    pin = lambda t: t.cpu().pin_memory()
    h_tok, h_logits, h_pend = pin(eng.draft_tok), pin(eng.drafter_logits), pin(b.pend0)
    h_out = torch.empty((wl.batch, wl.n_nodes + 1), dtype=torch.int32).pin_memory()
    h_ne = torch.empty((wl.batch,), dtype=torch.int32).pin_memory()
    h2d = h_tok.numel() * 4 + h_logits.numel() * 4 + h_pend.numel() * 4
    d2h = h_out.numel() * 4 + h_ne.numel() * 4

    def e2e_step(i):
        eng.len.copy_(b.len0, non_blocking=True)
        eng.draft_tok.copy_(h_tok, non_blocking=True)
        eng.drafter_logits.copy_(h_logits, non_blocking=True)
        eng.pending.copy_(h_pend, non_blocking=True)
        vb.verify_step(eng.model, eng.cache, eng.draft, b.params(i), b.sl, b.fl, b.res)
        h_out.copy_(b.res.out_tok, non_blocking=True)
        h_ne.copy_(b.res.n_emit, non_blocking=True)
        stream.synchronize()

    e2e_step(0)
    barrier()
    ev0.record(stream)
    for i in range(args.steps):
        e2e_step(i)
    ev1.record(stream)
    barrier()
    ms_e2e = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
    clk = clocks.stop() if rank == 0 else None          # sampled over the timed regions above
    e2e_value = job_value(world, wl.batch, wl.n_nodes, ms_e2e / args.steps)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, tf_peak, peak_kind = measured_peaks()
    sb = RL.step_bytes(wl)
    one_sweep = 2 * wl.batch * wl.rows <= 128
    # When both verifiers' rows fit one launch, verify_step streams every layer's weights once and applies the routed
    # layers to both row streams: the bytes its GEMM launches move are the "shared" figure.
    gemm_bytes = sb["gemm_shared"] if one_sweep else sb["gemm"]
    total_bytes = sb["total_shared"] if one_sweep else sb["total"]
    gemm_ms = timing["gemm"]["ms"] / n_timed
    gemm_gbs = gemm_bytes / 1e9 / (gemm_ms * 1e-3) if gemm_ms > 0 else 0.0
    step_gbs = total_bytes / 1e9 / (ms_step * 1e-3)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": wl.shape.dtype,
        "data": "synthetic",
        "config": config_of(wl, gate=args.gate, replicas=world,
                            l2="inputs larger than L2: the step streams %.1f GB of weights" % (gemm_bytes / 1e9)),
        "roofline": {"bound": "hbm", "kernel": "gemm_tc_kernel (all projection launches of the step)",
                     "achieved": gemm_gbs, "peak": peak, "peak_kind": peak_kind + " copy bandwidth",
                     "unit": "GB/s", "frac": gemm_gbs / peak, "traffic": RL.gemm_traffic(wl),
                     "algorithmic_bytes_per_step": gemm_bytes, "ms_per_step": gemm_ms,
                     "launches_per_step": timing["gemm"]["launches"] // n_timed,
                     "note": "one CUDA-event pair per run of consecutive GEMM launches (the four projections between two "
                             "attention calls, which keep their programmatic overlap); the runs are cut off from the "
                             "attention kernels around them, so this is a lower bound on the untimed step"},
        "step_roofline": {"algorithmic_bytes": total_bytes, "achieved_gbs": step_gbs,
                          "frac_of_measured": step_gbs / peak, "frac_of_8tbs": step_gbs / HBM_NOMINAL_GBS,
                          "algorithmic_bytes_two_separate_passes": sb["total"],
                          "achieved_gbs_two_separate_passes": sb["total"] / 1e9 / (ms_step * 1e-3),
                          "tensor_frac": sb["flops"] / (ms_step * 1e-3) / (tf_peak * 1e12)},
        "kernel_ms_per_step": {k: v["ms"] / n_timed for k, v in timing.items() if isinstance(v, dict)},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "gpu_launches": int(launches),
        "clocks": clk,
    }
    if world == 1:
        n_each = max(args.steps, 20)
        line["per_call"] = per_call(b, n_each, peak, tf_peak)
        line["graph_replay"] = graph_replay(b, n_each)
        ff = line["per_call"]["full_forward"]
        line["target"] = {"what": "full-tier pass (viasd_full_forward) of the 8B-shaped model at batch 1: >= 70 % of "
                                  "the HBM roofline at 8 TB/s",
                          "workload": wl.name, "ms_median": ff["ms_median"],
                          "frac_of_8tbs": ff.get("frac_of_8tbs"), "frac_of_measured": ff.get("frac_of_measured"),
                          "ms_at_70pct_of_8tbs": ff["algorithmic_bytes"] / (0.7 * HBM_NOMINAL_GBS * 1e9) * 1e3,
                          "met": bool(ff.get("frac_of_8tbs", 0.0) >= 0.7)}
        assert b.status_ok()
        if not args.no_sweep and wl.name == DEFAULT_WORKLOAD:
            line["sweep"] = run_sweep(b, peak, tf_peak, 20)
        if not args.no_cpu_baseline:
            del b, eng
            orc, runs, spent = time_oracle(wl, CPU_BASELINE_BUDGET_S, 6)
            t_step = float(np.mean([r["t_step"] for r in runs]))
            line["cpu_baseline"] = {"value": wl.batch * wl.n_nodes / t_step, "unit": UNIT, "cores": cpu_cores(),
                                    "kind": "oracle", "sample": orc.describe() + f"; mean of {len(runs)} runs",
                                    "extrapolated": not orc.whole, "seconds_measured": spent,
                                    "seconds_per_step": t_step}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true",
                    help="time the named workload only (the sweep over the other configurations runs with the default workload)")
    ap.add_argument("--gate", default="drafter", choices=["drafter", "slim"],
                    help="whose confidence sets the tiers: the drafter's (default, what the benchmark configurations "
                         "say) or the slim verifier's with a tier-1 acceptance ending the block (Algorithm 2 as printed)")
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
