"""Helpers shared by the GPU parity tests: run the oracle on a workload, compare under the margin rule."""
from __future__ import annotations

from typing import List, Optional, Sequence

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


def pinned_prefix(s: tiers.SeqResult, eps_row: float):
    """How far one sequence's result is fixed by the margin rule.

    Walks the oracle's decisions in order and stops at the first whose margin does not exceed 4 * eps_row.
    Returns (number of leading decisions that are pinned, number of path nodes fixed by them, whether every
    decision is pinned).  The decisions before the first unpinned one at block row r fix the accepted path up
    to the node that owns row r (node r - 1; nothing when r is the pending token's row).
    """
    n_pinned = 0
    for dcs in s.decisions:
        if dcs.margin > 4.0 * eps_row:
            n_pinned += 1
            continue
        k = 0 if dcs.row == 0 else s.path.index(dcs.row - 1) + 1
        return n_pinned, k, False
    return n_pinned, s.n_acc, True


def compare_resolution(seqs: List[tiers.SeqResult], n_acc, path, out_tok, n_emit, corr_src, eps_row: float,
                       only: Optional[Sequence[int]] = None):
    """Margin rule: a decision is pinned when its oracle margin exceeds 4 * eps_row (eps_row = observed
    max-abs logit difference).  Per sequence the oracle's decisions are walked in order; the accepted path
    and the emitted tokens up to the first unpinned decision must match exactly (the whole result when
    every decision is pinned).  ``only`` restricts the comparison to those sequences (the others count as
    not compared).  Returns (pinned leading decisions, total decisions, sequences compared to the end)."""
    pinned = total = full = 0
    for b, s in enumerate(seqs):
        if only is not None and b not in only:
            total += len(s.decisions)
            continue
        total += len(s.decisions)
        n_pin, k, ok_all = pinned_prefix(s, eps_row)
        pinned += n_pin
        got_path = [int(x) for x in path[b][:int(n_acc[b])]]
        got_tok = [int(x) for x in out_tok[b][:int(n_emit[b])]]
        # the fixed prefix: the device accepted at least these nodes, in this order, and emitted their tokens
        assert int(n_acc[b]) >= k, (b, int(n_acc[b]), k)
        assert got_path[:k] == s.path[:k], (b, got_path, s.path, k)
        assert got_tok[:k] == s.out_tok[:k], (b, got_tok, s.out_tok, k)
        if ok_all:
            full += 1
            assert int(n_acc[b]) == s.n_acc, (b, int(n_acc[b]), s.n_acc)
            assert got_path == s.path, (b, got_path, s.path)
            assert int(n_emit[b]) == len(s.out_tok), b
            assert got_tok == s.out_tok, (b, got_tok, s.out_tok)
            assert int(corr_src[b]) == s.corr_src, b
    return pinned, total, full


def assert_pinned(what: str, pinned: int, total: int, full: int, n_seq: int, min_frac: float, min_full: int):
    """The share of decisions the margin rule fixes is a property of the workload (logit spread against the
    bf16 path's error), so its floor is set per case from what is observed, less a margin; the message
    carries the counts either way."""
    msg = f"{what}: pinned decisions {pinned}/{total}, sequences compared to the end {full}/{n_seq}"
    print("PINNED " + msg)
    assert total == 0 or pinned / total >= min_frac, msg
    assert full >= min_full, msg
