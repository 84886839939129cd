"""CPU oracle, part 1: the verifier forward pass over a drafted block.

TEST INFRASTRUCTURE ONLY.  A plain, slow numpy restatement used to check the
CUDA path; nothing in the product may import it.  It shares no code with the
CUDA sources.

What it computes
  * the full verifier q: an L-layer pre-norm decoder (RMSNorm, rotary position
    embedding, multi-head or grouped-query attention, SwiGLU MLP) evaluated on
    the M = N + 1 rows {pending token, N draft nodes} against the KV cache,
    which yields, in one pass, the next-token distributions of the sequential
    model on the successive prefixes of the block (Sec. 3.1; Algorithm 2, the
    "run in parallel on prefixes" line);
  * the slim verifier q'_z = Pi_z(q): the same weights with every layer whose
    mask bit z_l is 0 bypassed by the residual identity; embeddings and output
    head are shared with q (Sec. 3.4, routing-mask formulation; Sec. 3.3).
    q' keeps its own KV cache over its routed layers.

Row i of a block attends to the committed cache rows 0..n-1 and to the block
rows on its own root path (itself included): a causal mask for a chain draft, an
ancestor mask for a tree draft.

The decoder block itself is the textbook Llama-style layer, so it is pinned
against closed forms and a second, independently written fp64 restatement in
the tests rather than against paper values (the paper prints none).

Precision: arithmetic runs in ``dt`` (fp64 by default, fp32 on request) on the
stored weight values widened exactly; no intermediate is rounded to bf16.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------
# small pieces
# --------------------------------------------------------------------------
def widen(a: np.ndarray, dt) -> np.ndarray:
    """Stored tensor (fp32, or bf16 as raw 16-bit words) -> values in dt, exactly."""
    if a.dtype == np.uint16:
        a = (a.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return a.astype(dt, copy=False)


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    ms = np.mean(np.square(x, dtype=np.float64), axis=-1, keepdims=True)
    return (x / np.sqrt(ms + eps)).astype(x.dtype) * gain.astype(x.dtype)


def rope_tables(pos: np.ndarray, head_dim: int, theta: float):
    """cos/sin of pos * theta^(-2p/head_dim), p = 0..head_dim/2-1, in fp64."""
    p = np.arange(head_dim // 2, dtype=np.float64)
    inv = np.power(np.float64(theta), -2.0 * p / head_dim)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv
    return np.cos(ang), np.sin(ang)


def rope(x: np.ndarray, cos: np.ndarray, sin: np.ndarray) -> np.ndarray:
    """Rotate pairs (p, p + head_dim/2) of the last axis.  x [..., heads, hd]; cos/sin [..., hd/2]."""
    h = x.shape[-1] // 2
    x1, x2 = x[..., :h], x[..., h:]
    c, s = cos[..., None, :].astype(x.dtype), sin[..., None, :].astype(x.dtype)
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def tree_layout(parent: Sequence[int]):
    """Rows of a block: row 0 = pending token, row n+1 = draft node n.

    Returns depth[M] (row 0 has depth 0) and vis[M, M] with vis[i, r] true when
    row r is on the root path of row i (r = i included).
    """
    n = len(parent)
    M = n + 1
    depth = np.zeros(M, dtype=np.int64)
    vis = np.zeros((M, M), dtype=bool)
    vis[0, 0] = True
    for node in range(n):
        pr = parent[node] + 1            # parent row (-1 -> row 0)
        assert 0 <= pr <= node, "parents must precede children"
        i = node + 1
        depth[i] = depth[pr] + 1
        vis[i] = vis[pr]
        vis[i, i] = True
    return depth, vis


# --------------------------------------------------------------------------
# KV cache
# --------------------------------------------------------------------------
class KVCache:
    """Per-model cache [layer ordinal][b][kv head][slot][head_dim].

    Slots below ``base_len`` may come from a read-only provider (synthetic
    committed context, stored as fp32 or bf16 words); everything from
    ``base_len`` on is held in dt and written by the forward pass and by commit.
    """

    def __init__(self, n_layers: int, batch: int, n_kv_heads: int, head_dim: int, capacity: int,
                 dt=np.float64, base_len: int = 0,
                 base: Optional[Callable[[int, int], np.ndarray]] = None):
        self.n_layers, self.batch, self.base_len, self.base, self.dt = n_layers, batch, base_len, base, dt
        own = capacity - base_len
        self.k = [np.zeros((batch, n_kv_heads, own, head_dim), dtype=dt) for _ in range(n_layers)]
        self.v = [np.zeros((batch, n_kv_heads, own, head_dim), dtype=dt) for _ in range(n_layers)]
        self._memo = {}

    def _base(self, layer: int, which: int) -> np.ndarray:
        key = (layer, which)
        if key not in self._memo:
            self._memo.clear() if len(self._memo) >= 2 else None
            self._memo[key] = widen(self.base(layer, which), self.dt)
        return self._memo[key]

    def read(self, layer: int, which: int, b: int, g: int, n: int) -> np.ndarray:
        """Committed rows 0..n-1 of (layer, b, kv head g): [n, hd]."""
        own = (self.k if which == 0 else self.v)[layer]
        if self.base_len == 0:
            return own[b, g, :n]
        basepart = self._base(layer, which)[b, g, :min(n, self.base_len)]
        if n <= self.base_len:
            return basepart
        return np.concatenate([basepart, own[b, g, :n - self.base_len]], axis=0)

    def write(self, layer: int, b: int, slot: int, k: np.ndarray, v: np.ndarray) -> None:
        """k, v: [H_kv, hd] for one slot."""
        assert slot >= self.base_len, "committed synthetic context is read-only"
        self.k[layer][b, :, slot - self.base_len] = k
        self.v[layer][b, :, slot - self.base_len] = v

    def move(self, b: int, src: int, dst: int) -> None:
        if src == dst:
            return
        o = self.base_len
        for l in range(self.n_layers):
            self.k[l][b, :, dst - o] = self.k[l][b, :, src - o]
            self.v[l][b, :, dst - o] = self.v[l][b, :, src - o]


# --------------------------------------------------------------------------
# forward
# --------------------------------------------------------------------------
def forward(weights, shape, layers: Sequence[int], cache: KVCache, lens: Sequence[int],
            row_tok: np.ndarray, parent: Sequence[int], dt=np.float64) -> np.ndarray:
    """Logits [B, M, V] of the sub-network made of ``layers`` on one drafted block.

    weights.tensor(layer, kind) supplies stored tensors ([out, in] matrices;
    layer -1 for "embed", "lm_head", "final_norm").  ``layers`` lists the layers
    that run, in increasing order (all of them for q, the routed ones for q');
    the cache is indexed by the ordinal within that list.  row_tok[b] = pending
    token followed by the N draft tokens.  K/V of every row are written at
    slots lens[b] + row; lens is not changed.
    """
    B, M = row_tok.shape
    H, Hk, hd, d = shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_model
    grp = H // Hk
    depth, vis = tree_layout(parent)
    lens = np.asarray(lens, dtype=np.int64)
    pos = lens[:, None] + depth[None, :]                       # [B, M]
    cos, sin = rope_tables(pos, hd, shape.rope_theta)          # [B, M, hd/2]
    scale = 1.0 / np.sqrt(np.float64(hd))

    E = weights.tensor(-1, "embed")
    h = widen(E[row_tok.reshape(-1)], dt).reshape(B, M, d).copy()

    for ordinal, l in enumerate(layers):
        W = {k: widen(weights.tensor(l, k), dt) for k in
             ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2")}
        a = rmsnorm(h, W["norm1"], shape.rms_eps)
        q = (a @ W["wq"].T).reshape(B, M, H, hd)
        k = (a @ W["wk"].T).reshape(B, M, Hk, hd)
        v = (a @ W["wv"].T).reshape(B, M, Hk, hd)
        q = rope(q, cos, sin)
        k = rope(k, cos, sin)
        o = np.zeros((B, M, H, hd), dtype=dt)
        for b in range(B):
            n = int(lens[b])
            for i in range(M):
                cache.write(ordinal, b, n + i, k[b, i], v[b, i])
            for g in range(Hk):
                Kc = cache.read(ordinal, 0, b, g, n)           # [n, hd]
                Vc = cache.read(ordinal, 1, b, g, n)
                Kn, Vn = k[b, :, g], v[b, :, g]                # [M, hd]
                for hh in range(g * grp, (g + 1) * grp):
                    qh = q[b, :, hh]                           # [M, hd]
                    s = np.concatenate([qh @ Kc.T, np.where(vis, qh @ Kn.T, -np.inf)], axis=1)
                    s = s.astype(np.float64) * scale
                    s -= s.max(axis=1, keepdims=True)
                    w = np.exp(s)
                    w /= w.sum(axis=1, keepdims=True)
                    w = w.astype(dt)
                    o[b, :, hh] = w[:, :n] @ Vc + w[:, n:] @ Vn
        h = h + o.reshape(B, M, H * hd) @ W["wo"].T
        a = rmsnorm(h, W["norm2"], shape.rms_eps)
        h = h + (silu(a @ W["wg"].T) * (a @ W["wu"].T)) @ W["wd"].T
        del W

    a = rmsnorm(h, widen(weights.tensor(-1, "final_norm"), dt), shape.rms_eps)
    return a @ widen(weights.tensor(-1, "lm_head"), dt).T


def commit(caches: List[KVCache], lens: np.ndarray, pending: np.ndarray, tokens: Optional[List[list]],
           n_acc: Sequence[int], path: Sequence[Sequence[int]], out_tok: Sequence[Sequence[int]]) -> None:
    """Append the emitted tokens; discard the rest of the block (Algorithm 1, the append/advance
    lines; Sec. 3.5 step 4).

    Before: slots lens[b] .. lens[b]+M-1 hold K/V of the block rows.  After: the
    accepted path's rows sit at lens[b]+1 .. lens[b]+n_acc (moved there if the
    draft was a tree), lens[b] has grown by the number of emitted tokens and the
    last emitted token is the new pending token (its K/V is not cached yet).
    Rows beyond the new length are dead: rollback is simply not keeping them.
    """
    for b in range(len(lens)):
        n = int(lens[b])
        for j in range(int(n_acc[b])):
            for c in caches:
                c.move(b, n + int(path[b][j]) + 1, n + 1 + j)
        emitted = [int(t) for t in out_tok[b]]
        if not emitted:
            continue
        if tokens is not None:
            tokens[b].extend([int(pending[b])] + emitted[:-1])
        lens[b] = n + len(emitted)
        pending[b] = emitted[-1]
