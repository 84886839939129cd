"""Workload definitions and seeded input builders for the multi-tier verify step.

Every tensor is produced by the counter-based generator in this package, so a
workload is fully described by (shape, seed).  The five named workloads follow
the benchmark configurations (tiny fp32 model; 7B-, 8B-, 13B- and 32B-shaped
bf16 models); the ``mini_*`` ones keep head_dim, the query/KV-head ratio and the
draft shape of their big sibling but shrink width and depth so that a CPU
reference finishes in seconds.

Nothing here computes anything the verification method computes: thresholds are
read from ``thresholds.json`` (written by a script that lives with the CPU
reference), not derived here.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np

from . import bf16_to_f32, index_i32, normal_bf16, normal_f32

_HERE = os.path.dirname(os.path.abspath(__file__))

# tensor ids ---------------------------------------------------------------
_LAYER_STRIDE = 16
_KINDS = {"wq": 0, "wk": 1, "wv": 2, "wo": 3, "wg": 4, "wu": 5, "wd": 6, "norm1": 7, "norm2": 8}
_T_EMBED, _T_HEAD, _T_FNORM = 100000, 100001, 100002
_T_PROMPT, _T_PENDING, _T_DRAFT, _T_DLOGITS, _T_CALIB = 110000, 110001, 110002, 110003, 110004
_T_KV = 200000   # + cache*100000 + layer_ordinal*2 + (0 K, 1 V)


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    dtype: str = "bf16"            # "f32" or "bf16": storage type of weights and KV cache
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0

    @property
    def layer_params(self) -> int:
        d, H, Hk, hd, ff = self.d_model, self.n_heads, self.n_kv_heads, self.head_dim, self.d_ff
        return 2 * d * H * hd + 2 * d * Hk * hd + 3 * d * ff + 2 * d

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


@dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    batch: int
    ctx: int                       # committed cache length when the step starts
    parent: Tuple[int, ...]        # draft tree, topological order; -1 = child of the pending token
    n_routed: int
    quantiles: Tuple[float, float] = (0.40, 0.75)
    mode: str = "greedy"           # or "sampling"
    temperature: float = 1.0
    seed: int = 0
    real_prefill: bool = False     # True: the context is a real prompt pushed through the model
    weight_sigma: float = 0.02
    logit_sigma: float = 2.0
    plant: float = 3.0
    gain_jitter: float = 0.0       # norm gains = 1 + N(0, gain_jitter)

    @property
    def n_nodes(self) -> int:
        return len(self.parent)

    @property
    def rows(self) -> int:
        return self.n_nodes + 1

    @property
    def routed(self) -> List[int]:
        return routed_layers(self.shape.n_layers, self.n_routed)

    @property
    def max_ctx(self) -> int:
        return self.ctx + self.rows


def routed_layers(n_layers: int, n_routed: int) -> List[int]:
    """Evenly spread routed layers: floor(i * L / L_s)."""
    return [(i * n_layers) // n_routed for i in range(n_routed)]


def chain(k: int) -> Tuple[int, ...]:
    return tuple(range(-1, k - 1))


def tree26() -> Tuple[int, ...]:
    """26-node static tree, depth 5, fan-out 4/3/2/1/1 pruned to first children."""
    par = [-1] * 4
    par += [i for i in range(4) for _ in range(3)]          # nodes 4..15
    par += [4 + 3 * i for i in range(4) for _ in range(2)]  # nodes 16..23
    par += [16, 24]                                         # nodes 24, 25
    assert len(par) == 26
    return tuple(par)


def small_tree() -> Tuple[int, ...]:
    """7-node tree (fan-out 3, then 2 under the first child, then a tail) for tests."""
    return (-1, -1, -1, 0, 0, 3, 1)


def drafter_rows(parent) -> Tuple[np.ndarray, int]:
    """prow[n]: which drafter-logit row node n was drafted from (one row per distinct parent)."""
    order: Dict[int, int] = {}
    prow = np.empty(len(parent), dtype=np.int32)
    for n, p in enumerate(parent):
        if p not in order:
            order[p] = len(order)
        prow[n] = order[p]
    return prow, len(order)


# ---------------------------------------------------------------------------
# named workloads
# ---------------------------------------------------------------------------
def _wl() -> Dict[str, Workload]:
    tiny = ModelShape(2, 256, 4, 4, 64, 1024, 1024, dtype="f32")
    s7b = ModelShape(32, 4096, 32, 32, 128, 11008, 32000)
    s8b = ModelShape(32, 4096, 32, 8, 128, 14336, 128256)
    s13b = ModelShape(40, 5120, 40, 40, 128, 13824, 32000)
    s32b = ModelShape(64, 5120, 40, 8, 128, 27648, 152064)
    w = {
        "c1_tiny": Workload("c1_tiny", tiny, 1, 128, chain(4), 1, seed=0, real_prefill=True),
        "c2_7b": Workload("c2_7b", s7b, 1, 1024, chain(8), 16, seed=2000),
        "c3_8b_tree": Workload("c3_8b_tree", s8b, 4, 2048, tree26(), 12, mode="sampling", seed=3000),
        "c3_8b_tree_b1": Workload("c3_8b_tree_b1", s8b, 1, 2048, tree26(), 12, mode="sampling", seed=3000),
        "c4_13b": Workload("c4_13b", s13b, 8, 4096, chain(6), 20, quantiles=(0.30, 0.70), seed=4000),
    }
    for b in (1, 2, 4, 8, 16):
        for ls in (16, 32, 48):
            w[f"c5_32b_b{b}_r{ls}"] = Workload(f"c5_32b_b{b}_r{ls}", s32b, b, 4096, chain(5), ls,
                                               seed=5000)
    # the 7B workload with thresholds that leave most drafted tokens to tiers 0 and 1 (quantiles 0.05 / 0.50): the case the
    # routed execution policy is for; 18 committed tokens can be replayed (max_query 27)
    w["c2_7b_routed"] = replace(w["c2_7b"], name="c2_7b_routed", quantiles=(0.05, 0.50))
    # profiling-sized cut of the 7B workload: same layer shapes, 2 layers (about 1.3 GB on the device)
    w["c2_7b_l2"] = Workload("c2_7b_l2", replace(s7b, n_layers=2), 1, 1024, chain(8), 1, seed=2000)
    w["c3_8b_tree_b1_l2"] = Workload("c3_8b_tree_b1_l2", replace(s8b, n_layers=2), 1, 2048, tree26(), 1, mode="sampling", seed=3000)
    w["c4_13b_l2"] = Workload("c4_13b_l2", replace(s13b, n_layers=2), 8, 4096, chain(6), 1, quantiles=(0.30, 0.70), seed=4000)
    # shrunken siblings: same head_dim, same query/KV-head ratio, same draft shape
    m7 = ModelShape(4, 512, 4, 4, 128, 1408, 2048)
    m8 = ModelShape(4, 512, 4, 1, 128, 1536, 4096)
    m13 = ModelShape(4, 640, 5, 5, 128, 1728, 2048)
    m32 = ModelShape(4, 640, 5, 1, 128, 1792, 4864)
    w["mini_7b"] = Workload("mini_7b", m7, 1, 300, chain(8), 2, seed=2100, gain_jitter=0.1,
                            weight_sigma=0.05)
    w["mini_8b_tree"] = Workload("mini_8b_tree", m8, 4, 333, tree26(), 2, mode="sampling",
                                 seed=3100, gain_jitter=0.1, weight_sigma=0.05)
    w["mini_8b_tree_greedy"] = replace(w["mini_8b_tree"], name="mini_8b_tree_greedy", mode="greedy")
    w["mini_13b"] = Workload("mini_13b", m13, 8, 517, chain(6), 2, quantiles=(0.30, 0.70),
                             seed=4100, gain_jitter=0.1, weight_sigma=0.05)
    w["mini_32b"] = Workload("mini_32b", m32, 16, 260, chain(5), 3, seed=5100, gain_jitter=0.1,
                             weight_sigma=0.05)
    w["mini_32b_b3"] = replace(w["mini_32b"], name="mini_32b_b3", batch=3)
    tiny_t = replace(tiny, n_layers=3)
    w["tiny_tree_f32"] = Workload("tiny_tree_f32", tiny_t, 2, 37, small_tree(), 2, seed=100,
                                  real_prefill=True, gain_jitter=0.1, weight_sigma=0.05)
    return w


WORKLOADS: Dict[str, Workload] = _wl()


def get(name: str) -> Workload:
    return WORKLOADS[name]


# ---------------------------------------------------------------------------
# model weights
# ---------------------------------------------------------------------------
class Model:
    """Lazily generated random-init decoder weights ([out, in] row-major).

    Arrays are fp32 for dtype "f32" and raw bf16 words (uint16) for "bf16".
    Generated on demand and, by default, not kept, so that a 7B-shaped model does
    not have to sit in host memory.
    """

    def __init__(self, wl: Workload, keep: bool = False):
        self.wl, self.shape, self.keep = wl, wl.shape, keep
        self._store: Dict[Tuple[int, str], np.ndarray] = {}

    def _gen(self, tensor: int, shape, sigma: float) -> np.ndarray:
        if self.shape.dtype == "f32":
            return normal_f32(self.wl.seed, tensor, shape, sigma)
        return normal_bf16(self.wl.seed, tensor, shape, sigma)

    def _gain(self, tensor: int) -> np.ndarray:
        d = self.shape.d_model
        g = np.ones(d, dtype=np.float32)
        if self.wl.gain_jitter:
            g = g + normal_f32(self.wl.seed, tensor, (d,), self.wl.gain_jitter)
        return g

    def matrix_shape(self, kind: str) -> Tuple[int, int]:
        s = self.shape
        return {"wq": (s.n_heads * s.head_dim, s.d_model), "wk": (s.n_kv_heads * s.head_dim, s.d_model),
                "wv": (s.n_kv_heads * s.head_dim, s.d_model), "wo": (s.d_model, s.n_heads * s.head_dim),
                "wg": (s.d_ff, s.d_model), "wu": (s.d_ff, s.d_model), "wd": (s.d_model, s.d_ff),
                "embed": (s.vocab, s.d_model), "lm_head": (s.vocab, s.d_model)}[kind]

    def tensor(self, layer: int, kind: str) -> np.ndarray:
        """layer = -1 for embed / lm_head / final_norm."""
        k = (layer, kind)
        if k in self._store:
            return self._store[k]
        if kind in ("norm1", "norm2"):
            a = self._gain(layer * _LAYER_STRIDE + _KINDS[kind])
        elif kind == "final_norm":
            a = self._gain(_T_FNORM)
        elif kind == "embed":
            a = self._gen(_T_EMBED, self.matrix_shape(kind), self.wl.weight_sigma)
        elif kind == "lm_head":
            a = self._gen(_T_HEAD, self.matrix_shape(kind), self.wl.weight_sigma)
        else:
            a = self._gen(layer * _LAYER_STRIDE + _KINDS[kind], self.matrix_shape(kind),
                          self.wl.weight_sigma)
        if self.keep:
            self._store[k] = a
        return a

    def layer(self, layer: int) -> Dict[str, np.ndarray]:
        return {k: self.tensor(layer, k) for k in _KINDS}


def as_f32(a: np.ndarray) -> np.ndarray:
    """Widen a generated tensor (fp32 or raw bf16 words) to fp32 values."""
    return bf16_to_f32(a) if a.dtype == np.uint16 else a


# ---------------------------------------------------------------------------
# step inputs
# ---------------------------------------------------------------------------
@dataclass
class StepInputs:
    pending: np.ndarray            # [B] int32
    draft_tok: np.ndarray          # [B, N] int32
    parent: np.ndarray             # [N] int32
    prow: np.ndarray               # [N] int32
    n_prows: int
    drafter_logits: np.ndarray     # [B, R, V] fp32
    prompt: Optional[np.ndarray] = None   # [B, ctx] int32 (real-prefill workloads)


def step_inputs(wl: Workload, step: int = 0) -> StepInputs:
    """Draft tokens, drafter logits (N(0, sigma) with +plant on each drafted token), pending ids."""
    B, N, V = wl.batch, wl.n_nodes, wl.shape.vocab
    parent = np.asarray(wl.parent, dtype=np.int32)
    prow, R = drafter_rows(wl.parent)
    off = step * 7919
    pending = index_i32(wl.seed, _T_PENDING, (B,), V, first=off * B)
    tok = index_i32(wl.seed, _T_DRAFT, (B, N), V, first=off * B * N)
    # siblings must carry distinct ids: bump collisions to the next free id
    for b in range(B):
        seen: Dict[int, set] = {}
        for n in range(N):
            s = seen.setdefault(int(parent[n]), set())
            t = int(tok[b, n])
            while t in s:
                t = (t + 1) % V
            s.add(t)
            tok[b, n] = t
    logits = normal_f32(wl.seed, _T_DLOGITS, (B, R, V), wl.logit_sigma, first=off * B * R * V)
    for b in range(B):
        for n in range(N):
            logits[b, prow[n], tok[b, n]] += np.float32(wl.plant)
    prompt = None
    if wl.real_prefill:
        prompt = index_i32(wl.seed, _T_PROMPT, (B, wl.ctx), V)
    return StepInputs(pending, tok, parent, prow, R, logits, prompt)


def calibration_rows(wl: Workload, n: int = 4096, first: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """Synthetic (drafter-logit row, drafted token) pairs first..first+n-1 of a disjoint counter range."""
    V = wl.shape.vocab
    tok = index_i32(wl.seed, _T_CALIB, (n,), V, first=first)
    logits = normal_f32(wl.seed, _T_CALIB + 1, (n, V), wl.logit_sigma, first=first * V)
    logits[np.arange(n), tok] += np.float32(wl.plant)
    return logits, tok


def kv_sigma(wl: Workload) -> float:
    """Std of synthetic context K/V: what the model's own projections give on unit-RMS input."""
    return wl.weight_sigma * float(np.sqrt(wl.shape.d_model))


def context_kv(wl: Workload, cache: int, layer_ordinal: int, which: int) -> np.ndarray:
    """Synthetic committed context for one layer of one cache.

    cache: 0 full verifier, 1 slim verifier.  which: 0 K, 1 V.
    Returns [B, H_kv, ctx, head_dim], fp32 or raw bf16 words by model dtype.
    """
    s = wl.shape
    shape = (wl.batch, s.n_kv_heads, wl.ctx, s.head_dim)
    t = _T_KV + cache * 100000 + layer_ordinal * 2 + which
    if s.dtype == "f32":
        return normal_f32(wl.seed, t, shape, kv_sigma(wl))
    return normal_bf16(wl.seed, t, shape, kv_sigma(wl))


def thresholds(wl: Workload) -> Tuple[float, float]:
    """(log_tau_lo, log_tau_hi) on log relative confidence, from the stored calibration."""
    with open(os.path.join(_HERE, "thresholds.json")) as f:
        tab = json.load(f)
    e = tab[wl.name]
    return float(np.float32(e["log_tau_lo"])), float(np.float32(e["log_tau_hi"]))
