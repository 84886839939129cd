"""CPU oracle, part 3: one verification cycle end to end, and plain autoregressive decoding.

TEST INFRASTRUCTURE ONLY; see decoder.py and tiers.py for the pieces.

One cycle (Algorithm 1 inside the while loop; Sec. 3.5 steps 3-4): tiers from
the gating confidence -> slim-verifier pass -> full-verifier pass -> tiered
acceptance and replacement token -> commit of the emitted tokens to both KV
caches.  Both passes always run here; skipping a pass whose tier is empty is an
execution policy that does not change any output.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

from . import decoder, tiers


@dataclass
class State:
    """Decoding state of a batch: two caches kept at one shared length per sequence."""
    full: decoder.KVCache
    slim: decoder.KVCache
    lens: np.ndarray            # [B] committed length
    pending: np.ndarray         # [B] last emitted token (K/V not cached)
    tokens: List[list]          # committed token ids per sequence


def new_state(shape, n_routed: int, batch: int, capacity: int, dt=np.float64, base_len: int = 0,
              base_full=None, base_slim=None, pending=None) -> State:
    mk = lambda nl, base: decoder.KVCache(nl, batch, shape.n_kv_heads, shape.head_dim, capacity, dt,
                                          base_len, base)
    return State(mk(shape.n_layers, base_full), mk(n_routed, base_slim),
                 np.full(batch, base_len, dtype=np.int64),
                 np.zeros(batch, dtype=np.int64) if pending is None else np.array(pending, dtype=np.int64),
                 [[] for _ in range(batch)])


def block_rows(pending: np.ndarray, draft_tok: np.ndarray) -> np.ndarray:
    return np.concatenate([np.asarray(pending, dtype=np.int64)[:, None],
                           np.asarray(draft_tok, dtype=np.int64)], axis=1)


def prefill(weights, shape, routed: Sequence[int], st: State, prompt: np.ndarray, dt=np.float64) -> None:
    """Push a prompt [B, T] through both models; afterwards len = T-1 and pending = last prompt token."""
    B, T = prompt.shape
    if T > 1:
        rows = np.asarray(prompt[:, :T - 1], dtype=np.int64)
        ch = tuple(range(-1, T - 3))   # T-1 rows: a chain of T-2 nodes after the first
        decoder.forward(weights, shape, range(shape.n_layers), st.full, st.lens, rows, ch, dt)
        decoder.forward(weights, shape, routed, st.slim, st.lens, rows, ch, dt)
        for b in range(B):
            st.tokens[b].extend(int(t) for t in prompt[b, :T - 1])
        st.lens += T - 1
    st.pending[:] = prompt[:, T - 1]


@dataclass
class StepOut:
    tier: np.ndarray
    conf: np.ndarray
    slim_logits: np.ndarray
    full_logits: np.ndarray
    seqs: List[tiers.SeqResult]


def verify_step(weights, shape, routed: Sequence[int], st: State, draft_tok: np.ndarray,
                parent: Sequence[int], prow: Sequence[int], drafter_logits: np.ndarray,
                log_tau_lo: float, log_tau_hi: float, P: tiers.Params, conf_source: int = 0,
                dt=np.float64, do_commit: bool = True) -> StepOut:
    rows = block_rows(st.pending, draft_tok)
    slim_logits = decoder.forward(weights, shape, routed, st.slim, st.lens, rows, parent, dt)
    if conf_source == 0:
        tier, conf = tiers.tier_rule(drafter_logits, draft_tok, prow, log_tau_lo, log_tau_hi)
    else:   # Algorithm 2 as printed: the slim verifier's own confidence at the parent row
        tier, conf = tiers.tier_rule(slim_logits.astype(np.float32), draft_tok,
                                     [p + 1 for p in parent], log_tau_lo, log_tau_hi)
    full_logits = decoder.forward(weights, shape, range(shape.n_layers), st.full, st.lens, rows,
                                  parent, dt)
    seqs = tiers.resolve(draft_tok, parent, prow, tier, drafter_logits, slim_logits, full_logits, P)
    if do_commit:
        decoder.commit([st.full, st.slim], st.lens, st.pending, st.tokens,
                       [s.n_acc for s in seqs], [s.path for s in seqs], [s.out_tok for s in seqs])
    return StepOut(tier, conf, slim_logits, full_logits, seqs)


def greedy_decode(weights, shape, st: State, n_new: int, dt=np.float64) -> List[List[int]]:
    """Plain autoregressive greedy decoding of the full model: one row per step."""
    B = len(st.lens)
    out: List[List[int]] = [[] for _ in range(B)]
    for _ in range(n_new):
        rows = np.asarray(st.pending, dtype=np.int64)[:, None]
        logits = decoder.forward(weights, shape, range(shape.n_layers), st.full, st.lens, rows, (), dt)
        nxt = logits[:, 0].argmax(axis=-1)
        for b in range(B):
            st.tokens[b].append(int(st.pending[b]))
            out[b].append(int(nxt[b]))
        st.lens += 1
        st.pending[:] = nxt
    return out
