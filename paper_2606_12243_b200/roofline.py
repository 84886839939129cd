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


def call_bytes(wl: Workload) -> dict:
    """Algorithmic bytes of the two small calls.  tier_accept: the tier kernel reads every gating row once, the row
    statistics read every drafter / slim / full logits row once (the accept walk then works from the statistics).
    kv_commit: at most depth-of-tree rows of K and V per layer and kv head move (read + write), in both caches."""
    s = wl.shape
    R = len(set(wl.parent))
    tier_accept = wl.batch * R * s.vocab * 4 + (2 * wl.batch * wl.rows + wl.batch * R) * s.vocab * 4
    depth = {-1: 0}
    for n, p in enumerate(wl.parent):
        depth[n] = depth[p] + 1
    kv_commit = 2 * (s.n_layers + wl.n_routed) * wl.batch * max(depth.values()) * 2 * s.n_kv_heads * s.head_dim * s.elem_bytes
    return dict(tier_accept=tier_accept, kv_commit=kv_commit)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per launch of gemm_tc_kernel, in MB, from the ncu
# captures summarised under profiles/ (gemm_tc_kernel_*_layer_shapes.md), keyed by (output features, input features)
# of the launch: QKV, O, gate/up (both matrices), down, head.  The weights are all but a per cent of it at the token
# rows of these workloads (activation tiles hit in L2), so one figure serves launches of 9 to 54 rows.
NCU_GEMM_TRAFFIC_MB = {
    # 7B layer shapes (captured with 18 token rows)
    (12288, 4096): 105.2, (4096, 4096): 34.1, (22016, 4096): 185.3, (4096, 11008): 96.6, (32000, 4096): 271.6,
    # 8B layer shapes (captured with 27 token rows; the head with 54); (4096, 4096) is shared with the 7B shapes
    (6144, 4096): 51.5, (28672, 4096): 243.0, (4096, 14336): 124.7, (128256, 4096): 1085.1,
}


def gemm_traffic(wl: Workload):
    """Measured DRAM bytes of the step's GEMM launches: per-launch ncu figures of the workload's layer shapes scaled
    by the launches of the step (traffic is per launch, and every layer launches the same shapes).  None when a
    shape of this workload has no capture."""
    s = wl.shape
    qd, kvd = s.n_heads * s.head_dim, s.n_kv_heads * s.head_dim
    shapes = [(qd + 2 * kvd, s.d_model), (s.d_model, qd), (2 * s.d_ff, s.d_model), (s.d_model, s.d_ff)]
    one_sweep = 2 * wl.batch * wl.rows <= 128
    layer_launches = s.n_layers if one_sweep else s.n_layers + wl.n_routed
    head_launches = 1 if one_sweep else 2
    total = 0.0
    for n, k in shapes + [(s.vocab, s.d_model)]:
        t = NCU_GEMM_TRAFFIC_MB.get((n, k))
        if t is None:
            return None
        total += t * (head_launches if n == s.vocab else layer_launches)
    return int(total * 1e6)
