"""Algorithmic bytes and flops of the verify step (what a pass must move, nothing avoided is counted).

Per layer: P_l = 2 d H hd + 2 d Hkv hd + 3 d ff weights (norm gains ignored: 2 d floats).
A pass over n_l layers streams n_l P_l + V d weights (the output head; the embedding is a gather of B M
rows), reads the committed K/V of those layers once, appends M rows per sequence, and writes the logits,
which the accept kernel reads once.
"""
from __future__ import annotations

from synth.workloads import Workload


def layer_weight_params(s) -> int:
    return 2 * s.d_model * s.n_heads * s.head_dim + 2 * s.d_model * s.n_kv_heads * s.head_dim + 3 * s.d_model * s.d_ff


def pass_bytes(wl: Workload, n_layers: int) -> dict:
    s = wl.shape
    es = s.elem_bytes
    rows = wl.batch * wl.rows
    weights = (n_layers * (layer_weight_params(s) + 2 * s.d_model) + s.vocab * s.d_model + s.d_model) * es
    kv_tok = 2 * s.n_kv_heads * s.head_dim * es
    kv_read = n_layers * kv_tok * wl.batch * wl.ctx
    kv_append = n_layers * kv_tok * rows
    embed = rows * s.d_model * es
    logits = 2 * rows * s.vocab * 4
    flops = 2 * rows * (n_layers * layer_weight_params(s) + s.vocab * s.d_model) \
        + n_layers * wl.batch * 4 * wl.rows * (wl.ctx + wl.rows) * s.n_heads * s.head_dim
    total = weights + kv_read + kv_append + embed + logits
    return dict(weights=weights, kv_read=kv_read, kv_append=kv_append, embed=embed, logits=logits, total=total,
                flops=flops)


def gemm_bytes(wl: Workload, n_layers: int) -> int:
    """Algorithmic bytes of the projection GEMMs of one pass: each weight once, activations in and out."""
    s = wl.shape
    es = s.elem_bytes
    rows = wl.batch * wl.rows
    qd, kvd = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    per_layer = layer_weight_params(s) * es
    per_layer += rows * (s.d_model * es + (qd + 2 * kvd) * 4)            # qkv: normed input, fp32 output
    per_layer += rows * (qd * es + s.d_model * 4)                        # o projection into the residual
    per_layer += rows * (s.d_model * es + s.d_ff * es)                   # gate/up with fused SwiGLU
    per_layer += rows * (s.d_ff * es + s.d_model * 4)                    # down projection into the residual
    head = s.vocab * s.d_model * es + rows * (s.d_model * es + s.vocab * 4)
    return n_layers * per_layer + head


def step_bytes(wl: Workload) -> dict:
    """Bytes of one verify step.

    "total" / "gemm": the two passes counted separately (each pass streams its own layers and the head).
    "total_shared" / "gemm_shared": what the one-sweep schedule of viasd_verify_step has to move: every layer's
    weights and the head once, with the routed layers applied to both row streams; KV caches, appended rows,
    embeddings and logits of both verifiers as before.
    """
    s = wl.shape
    es = s.elem_bytes
    full, slim = pass_bytes(wl, s.n_layers), pass_bytes(wl, wl.n_routed)
    tier = wl.batch * len(set(wl.parent)) * s.vocab * 4
    rows = wl.batch * wl.rows
    qd, kvd = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    act_per_layer = rows * ((s.d_model * es + (qd + 2 * kvd) * 4) + (qd * es + s.d_model * 4)
                            + (s.d_model * es + s.d_ff * es) + (s.d_ff * es + s.d_model * 4))
    head_act = rows * (s.d_model * es + s.vocab * 4)
    slim_weights = (wl.n_routed * (layer_weight_params(s) + 2 * s.d_model) + s.vocab * s.d_model + s.d_model) * es
    gemm_sep = gemm_bytes(wl, s.n_layers) + gemm_bytes(wl, wl.n_routed)
    gemm_shared = gemm_bytes(wl, s.n_layers) + wl.n_routed * act_per_layer + head_act
    total_sep = full["total"] + slim["total"] + tier
    return dict(full=full, slim=slim, tier=tier, total=total_sep, flops=full["flops"] + slim["flops"], gemm=gemm_sep,
                gemm_shared=gemm_shared, total_shared=total_sep - slim_weights)
