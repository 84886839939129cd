"""The numerators of the reported roofline fractions: the bytes a pass has to move, checked against parameter counts
worked out by hand from the model shapes (Llama-style blocks: 4 attention projections with grouped KV heads, 3 MLP
matrices, untied output head) and against the sizes the KV cache must have."""
import pytest

from paper_2606_12243_b200 import roofline as RF
from synth import workloads as W

GB = 1e9


def _hand_layer_params(d, h, hkv, hd, ff):
    return d * h * hd + 2 * d * hkv * hd + h * hd * d + 3 * d * ff      # q, k + v, o, gate + up + down


@pytest.mark.parametrize("name,d,h,hkv,hd,ff,V,L,weights_gb", [
    ("c2_7b", 4096, 32, 32, 128, 11008, 32000, 32, 13.2),
    ("c3_8b_tree_b1", 4096, 32, 8, 128, 14336, 128256, 32, 15.0),
    ("c4_13b", 5120, 40, 40, 128, 13824, 32000, 40, 25.7),
    ("c5_32b_b1_r16", 5120, 40, 8, 128, 27648, 152064, 64, 64.0),
])
def test_weight_bytes_of_a_full_pass(name, d, h, hkv, hd, ff, V, L, weights_gb):
    wl = W.get(name)
    s = wl.shape
    assert (s.d_model, s.n_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.vocab, s.n_layers) == (d, h, hkv, hd, ff, V, L)
    assert RF.layer_weight_params(s) == _hand_layer_params(d, h, hkv, hd, ff)
    pb = RF.pass_bytes(wl, L)
    hand = (L * (_hand_layer_params(d, h, hkv, hd, ff) + 2 * d) + V * d + d) * 2      # bf16; norm gains included
    assert pb["weights"] == hand
    assert abs(pb["weights"] / GB - weights_gb) < 0.06 * weights_gb       # the round figure of the model card
    # the committed cache is read once: 2 (K and V) x kv heads x head dim x 2 bytes per token and layer
    assert pb["kv_read"] == L * wl.batch * wl.ctx * 2 * hkv * hd * 2
    assert pb["kv_append"] == L * wl.batch * wl.rows * 2 * hkv * hd * 2
    assert pb["total"] == pb["weights"] + pb["kv_read"] + pb["kv_append"] + pb["embed"] + pb["logits"]


def test_slim_pass_streams_its_layer_fraction_plus_the_head():
    for name in ("c5_32b_b1_r16", "c5_32b_b1_r32", "c5_32b_b1_r48"):
        wl = W.get(name)
        s = wl.shape
        full, slim = RF.pass_bytes(wl, s.n_layers), RF.pass_bytes(wl, wl.n_routed)
        head = (s.vocab * s.d_model + s.d_model) * 2
        frac = (slim["weights"] - head) / (full["weights"] - head)
        assert abs(frac - wl.n_routed / s.n_layers) < 1e-12
        assert slim["kv_read"] * s.n_layers == full["kv_read"] * wl.n_routed


def test_one_sweep_step_reads_every_weight_once():
    wl = W.get("c3_8b_tree_b1")
    sb = RF.step_bytes(wl)
    full, slim = sb["full"], sb["slim"]
    # both verifiers in one sweep: the routed layers' weights and the head are not read a second time
    assert sb["total_shared"] == sb["total"] - slim["weights"]
    assert sb["total"] == full["total"] + slim["total"] + sb["tier"]
    # the GEMM class of the shared sweep: all weights once, the routed layers' activations twice
    assert sb["gemm_shared"] < sb["gemm"]
    assert sb["gemm_shared"] > RF.gemm_bytes(wl, wl.shape.n_layers)
    # 8B shape at batch 1: the step is weight-bound (K/V and logits are a few per cent)
    assert full["weights"] / full["total"] > 0.95


def test_measured_traffic_table_stays_close_to_the_algorithmic_bytes():
    for name in ("c2_7b", "c3_8b_tree_b1"):
        wl = W.get(name)
        t = RF.gemm_traffic(wl)
        assert t is not None
        assert 0.98 < t / RF.step_bytes(wl)["gemm_shared"] < 1.06
