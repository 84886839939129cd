"""Helpers shared by the GPU parity tests: run the oracle on a workload, compare under the margin rule."""
from __future__ import annotations

from typing import List, Optional

import numpy as np

from synth import workloads as W
from oracle import decoder, step, tiers

# Logit tolerances (GPU vs oracle): the bf16 path rounds GEMM operands, new K/V rows and attention
# probabilities to bf16 (relative 2^-9 each) and accumulates in fp32; the stated bound for that path is
# max-abs 3e-2 and relative L2 1e-2.  The fp32 configuration differs from the oracle by summation order
# only: 1e-4.
TOL = {"bf16": dict(max_abs=3e-2, rel_l2=1e-2), "f32": dict(max_abs=1e-4, rel_l2=1e-5)}


def oracle_state(wl: W.Workload, dt=np.float64, extra: int = 0) -> step.State:
    cap = wl.ctx + wl.rows + extra
    if wl.real_prefill or wl.ctx == 0:
        return step.new_state(wl.shape, wl.n_routed, wl.batch, cap, dt)
    return step.new_state(wl.shape, wl.n_routed, wl.batch, cap, dt, base_len=wl.ctx,
                          base_full=lambda o, which: W.context_kv(wl, 0, o, which),
                          base_slim=lambda o, which: W.context_kv(wl, 1, o, which))


def oracle_params(wl: W.Workload, step_no: int = 0, **kw) -> tiers.Params:
    kw.setdefault("mode", wl.mode)
    kw.setdefault("temperature", wl.temperature)
    kw.setdefault("seed", wl.seed)
    return tiers.Params(step=step_no, **kw)


def logit_errors(got: np.ndarray, want: np.ndarray):
    g, w = got.astype(np.float64), want.astype(np.float64)
    return float(np.abs(g - w).max()), float(np.linalg.norm(g - w) / np.linalg.norm(w))


def assert_logits_close(got, want, dtype: str, what: str = "logits"):
    ma, rl = logit_errors(got, want)
    t = TOL[dtype]
    assert ma <= t["max_abs"] and rl <= t["rel_l2"], f"{what}: max-abs {ma:.3e} rel-L2 {rl:.3e} (tol {t})"
    return ma, rl


def compare_resolution(seqs: List[tiers.SeqResult], n_acc, path, out_tok, n_emit, corr_src, eps_row: float):
    """Margin rule: a decision is pinned when its oracle margin exceeds 4 * eps_row (eps_row = observed
    max-abs logit difference).  Walk the oracle's decisions in order; everything up to the first unpinned
    one must match exactly.  Returns (pinned decisions, total decisions, fully compared sequences)."""
    pinned = total = full = 0
    for b, s in enumerate(seqs):
        ok_all = True
        n_ok_path = 0          # accepted prefix known to be pinned
        for dcs in s.decisions:
            total += 1
            if dcs.margin > 4.0 * eps_row:
                pinned += 1
            else:
                ok_all = False
                break
        if ok_all:
            full += 1
            assert int(n_acc[b]) == s.n_acc, (b, int(n_acc[b]), s.n_acc)
            assert [int(x) for x in path[b][:s.n_acc]] == s.path, b
            assert int(n_emit[b]) == len(s.out_tok), b
            assert [int(x) for x in out_tok[b][:len(s.out_tok)]] == s.out_tok, (b, out_tok[b], s.out_tok)
            assert int(corr_src[b]) == s.corr_src, b
    return pinned, total, full
