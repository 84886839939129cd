"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test is chosen so that a plausible slip in the oracle (a dropped term, a wrong sign or
index, a transposed operand, an off-by-one in the cache) makes it fail.
"""
import os
from dataclasses import replace

import numpy as np
import pytest

import synth
from synth import workloads as W
from oracle import decoder, step, tiers

GOLD = os.path.join(os.path.dirname(__file__), "golden")

SHAPE = W.ModelShape(n_layers=3, d_model=64, n_heads=4, n_kv_heads=2, head_dim=16, d_ff=96, vocab=53,
                     dtype="f32")


def small_workload(parent=W.chain(4), batch=2, seed=11, shape=SHAPE, n_routed=2):
    return W.Workload("pin", shape, batch, 0, tuple(parent), n_routed, seed=seed, gain_jitter=0.2,
                      weight_sigma=0.3)


def fresh(wl, cap=64, dt=np.float64):
    return step.new_state(wl.shape, wl.n_routed, wl.batch, cap, dt)


# --------------------------------------------------------------------------
# generator
# --------------------------------------------------------------------------
def _mix_py(z):
    m = (1 << 64) - 1
    z &= m
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & m
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & m
    return z ^ (z >> 31)


def test_generator_matches_python_restatement():
    g = 0x9E3779B97F4A7C15
    key = synth.key(7, 3)
    a = synth.normal_f32(7, 3, (5,), 0.02, first=10)
    for i in range(5):
        s = 0
        for j in range(3):
            w = _mix_py(key + (3 * (10 + i) + j) * g)
            s += (w & 0xFFFF) + ((w >> 16) & 0xFFFF) + ((w >> 32) & 0xFFFF) + (w >> 48)
        want = np.float32(s - 6 * 65535) * np.float32(np.float32(0.02) * np.float32(1 / 65536))
        assert a[i] == want
    idx = synth.index_i32(7, 4, (4,), 1000, first=2)
    assert [int(x) for x in idx] == [_mix_py(synth.key(7, 4) + (2 + i) * g) % 1000 for i in range(4)]


def test_generator_moments_and_bf16():
    x = synth.normal_f32(1, 1, (400000,), 2.0)
    assert abs(x.mean()) < 0.02 and abs(x.std() - 2.0) < 0.02
    assert np.abs(x).max() <= 12.0
    h = synth.normal_bf16(1, 1, (4096,), 2.0)
    back = synth.bf16_to_f32(h)
    assert np.all(np.abs(back - x[:4096]) <= np.abs(x[:4096]) * 2.0 ** -8)
    assert np.array_equal(h, synth.f32_to_bf16(x[:4096]))


# --------------------------------------------------------------------------
# decoder pieces: closed forms
# --------------------------------------------------------------------------
def test_rope_identities():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 1, 2, 16))
    c0, s0 = decoder.rope_tables(np.array([[0]]), 16, 10000.0)
    assert np.array_equal(decoder.rope(x, c0, s0), x)                 # position 0 is the identity
    c, s = decoder.rope_tables(np.array([[37]]), 16, 10000.0)
    y = decoder.rope(x, c, s)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))
    # <R_m q, R_n k> depends on m - n only
    q, k = rng.standard_normal((2, 1, 1, 1, 16))
    def dot(m, n):
        cm, sm = decoder.rope_tables(np.array([[m]]), 16, 10000.0)
        cn, sn = decoder.rope_tables(np.array([[n]]), 16, 10000.0)
        return float((decoder.rope(q, cm, sm) * decoder.rope(k, cn, sn)).sum())
    assert abs(dot(5, 2) - dot(103, 100)) < 1e-9
    assert abs(dot(5, 2) - dot(2, 5)) > 1e-6                          # and is not symmetric
    # first pair rotates by exactly pos radians: (1, 0) -> (cos, sin) on dims (0, hd/2)
    e = np.zeros((1, 1, 1, 16)); e[..., 0] = 1.0
    r = decoder.rope(e, c, s)
    assert np.allclose([r[0, 0, 0, 0], r[0, 0, 0, 8]], [np.cos(37.0), np.sin(37.0)])
    # last pair uses the smallest frequency theta^(-(hd-2)/hd)
    e = np.zeros((1, 1, 1, 16)); e[..., 7] = 1.0
    r = decoder.rope(e, c, s)
    ang = 37.0 * 10000.0 ** (-14.0 / 16.0)
    assert np.allclose([r[0, 0, 0, 7], r[0, 0, 0, 15]], [np.cos(ang), np.sin(ang)])


def test_rmsnorm_and_silu_closed_forms():
    x = np.full((1, 8), 3.0)
    g = np.arange(1, 9, dtype=np.float64)
    assert np.allclose(decoder.rmsnorm(x, g, 0.0), g)
    assert np.allclose(decoder.rmsnorm(-x, g, 0.0), -g)
    y = decoder.rmsnorm(np.array([[3.0, 4.0]]), np.ones(2), 0.0)
    assert np.allclose(y, np.array([[3.0, 4.0]]) / np.sqrt(12.5))
    assert decoder.silu(np.array([0.0]))[0] == 0.0
    assert np.isclose(decoder.silu(np.array([2.0]))[0], 2.0 / (1.0 + np.exp(-2.0)))
    assert np.isclose(decoder.silu(np.array([-2.0]))[0], -2.0 / (1.0 + np.exp(2.0)))


def test_tree_layout():
    depth, vis = decoder.tree_layout(W.small_tree())      # (-1,-1,-1,0,0,3,1)
    assert list(depth) == [0, 1, 1, 1, 2, 2, 3, 2]
    assert [list(np.nonzero(v)[0]) for v in vis] == [[0], [0, 1], [0, 2], [0, 3], [0, 1, 4], [0, 1, 5],
                                                      [0, 1, 4, 6], [0, 2, 7]]
    d26, v26 = decoder.tree_layout(W.tree26())
    assert d26.max() == 5 and len(d26) == 27
    assert [int((d26 == k).sum()) for k in range(6)] == [1, 4, 12, 8, 1, 1]
    dch, vch = decoder.tree_layout(W.chain(5))
    assert np.array_equal(vch, np.tril(np.ones((6, 6), dtype=bool)))


class _OneLayerIdentity:
    """Weights that make attention observable: Wq = Wk = 0 (uniform attention), Wv = Wo = I, MLP off."""

    def __init__(self, shape, embed):
        self.s, self.embed = shape, embed

    def tensor(self, layer, kind):
        s = self.s
        d = s.d_model
        if kind == "embed":
            return self.embed
        if kind == "lm_head":
            return np.eye(d, dtype=np.float32)            # vocab == d
        if kind in ("norm1", "norm2", "final_norm"):
            return np.ones(d, dtype=np.float32)
        if kind in ("wv", "wo"):
            return np.eye(d, dtype=np.float32)
        if kind in ("wq", "wk"):
            return np.zeros((d, d), dtype=np.float32)
        if kind in ("wg", "wu"):
            return np.zeros((s.d_ff, d), dtype=np.float32)
        return np.zeros((d, s.d_ff), dtype=np.float32)    # wd


def test_attention_uniform_average_and_single_key():
    """With zero scores attention is the mean of the visible V rows; with one visible key it is that row."""
    s = W.ModelShape(1, 8, 2, 2, 4, 4, 8, dtype="f32")
    rng = np.random.default_rng(1)
    E = rng.standard_normal((8, 8)).astype(np.float32)
    wts = _OneLayerIdentity(s, E)
    st = step.new_state(s, 1, 1, 16)
    toks = np.array([[3, 5, 1]])
    # expected, by hand: h_i = e_i + mean_{r<=i} rmsnorm(e_r); logits = rmsnorm(h_i)
    e = E[toks[0]].astype(np.float64)
    nrm = lambda x: x / np.sqrt((x * x).mean(-1, keepdims=True) + s.rms_eps)
    a = nrm(e)
    want = nrm(np.stack([e[0] + a[0], e[1] + a[:2].mean(0), e[2] + a[:3].mean(0)]))
    got = decoder.forward(wts, s, [0], st.full, st.lens, toks, W.chain(2))
    assert np.allclose(got[0], want, atol=1e-12)
    # tree (-1, -1): rows 1 and 2 are siblings and must not see each other
    got = decoder.forward(wts, s, [0], st.full, st.lens, toks, (-1, -1))
    want = nrm(np.stack([e[0] + a[0], e[1] + a[:2].mean(0), e[2] + (a[0] + a[2]) / 2]))
    assert np.allclose(got[0], want, atol=1e-12)


# --------------------------------------------------------------------------
# decoder: structural invariants
# --------------------------------------------------------------------------
def test_block_forward_equals_sequential_forwards():
    """Algorithm 2, parallel block verification: row j of a K-row pass is the sequential model's
    distribution on the prefix extended by the first j draft tokens."""
    wl = small_workload()
    m = W.Model(wl, keep=True)
    toks = synth.index_i32(5, 1, (wl.batch, 6), wl.shape.vocab)
    L = range(wl.shape.n_layers)
    st = fresh(wl)
    blk = decoder.forward(m, wl.shape, L, st.full, st.lens, toks.astype(np.int64), W.chain(5))
    st2 = fresh(wl)
    for i in range(6):
        one = decoder.forward(m, wl.shape, L, st2.full, st2.lens, toks[:, i:i + 1].astype(np.int64), ())
        assert np.allclose(one[:, 0], blk[:, i], atol=1e-10), i
        st2.lens += 1


def test_tree_paths_equal_chain_forwards():
    wl = small_workload(parent=W.small_tree())
    m = W.Model(wl, keep=True)
    par = W.small_tree()
    toks = synth.index_i32(5, 2, (wl.batch, len(par) + 1), wl.shape.vocab).astype(np.int64)
    L = range(wl.shape.n_layers)
    st = fresh(wl)
    # a committed prefix first, so that both cache and block rows are attended to
    pre = synth.index_i32(5, 3, (wl.batch, 7), wl.shape.vocab).astype(np.int64)
    decoder.forward(m, wl.shape, L, st.full, st.lens, pre, W.chain(6)); st.lens += 7
    tree = decoder.forward(m, wl.shape, L, st.full, st.lens, toks, par)
    for leaf in (6, 7, 5, 3):                       # rows
        rows = [leaf]
        while rows[-1] != 0:
            rows.append(par[rows[-1] - 1] + 1)
        rows = rows[::-1]
        ch = decoder.forward(m, wl.shape, L, st.full, st.lens, toks[:, rows], W.chain(len(rows) - 1))
        assert np.allclose(ch, tree[:, rows], atol=1e-10), leaf


def test_slim_with_all_layers_is_full_and_skipping_matters():
    """q'_z with z = 1^L is q itself (definition of the routed sub-network); a bypassed layer is the
    residual identity, so z with one zero equals a model with that layer removed."""
    wl = small_workload()
    m = W.Model(wl, keep=True)
    toks = synth.index_i32(5, 4, (wl.batch, 5), wl.shape.vocab).astype(np.int64)
    st = fresh(wl)
    full = decoder.forward(m, wl.shape, range(3), st.full, st.lens, toks, W.chain(4))
    st_b = step.new_state(wl.shape, 3, wl.batch, 64)
    slim_all = decoder.forward(m, wl.shape, [0, 1, 2], st_b.slim, st_b.lens, toks, W.chain(4))
    assert np.array_equal(full, slim_all)
    slim = decoder.forward(m, wl.shape, [0, 2], st.slim, st.lens, toks, W.chain(4))
    assert np.abs(slim - full).max() > 1e-3

    class Two:                                       # the 2-layer model made of layers 0 and 2
        def tensor(self, layer, kind):
            return m.tensor({0: 0, 1: 2, -1: -1}[layer], kind)
    st_c = step.new_state(replace(wl.shape, n_layers=2), 2, wl.batch, 64)
    two = decoder.forward(Two(), replace(wl.shape, n_layers=2), [0, 1], st_c.full, st_c.lens, toks,
                          W.chain(4))
    assert np.array_equal(two, slim)


def _torch_full_sequence_logits(m, shape, toks):
    """Second opinion: the whole sequence recomputed from scratch, no cache, torch fp64, complex-number
    rotary embedding and a dense causal mask."""
    import torch
    t = lambda a: torch.from_numpy(W.as_f32(a).astype(np.float64))
    T = len(toks)
    H, Hk, hd = shape.n_heads, shape.n_kv_heads, shape.head_dim
    x = t(m.tensor(-1, "embed"))[torch.as_tensor(toks)]
    freqs = torch.outer(torch.arange(T, dtype=torch.float64),
                        shape.rope_theta ** (-torch.arange(0, hd, 2, dtype=torch.float64) / hd))
    rot = torch.polar(torch.ones_like(freqs), freqs)                 # [T, hd/2]
    def rotary(z):                                                    # z [T, heads, hd]
        zc = torch.complex(z[..., :hd // 2], z[..., hd // 2:]) * rot[:, None, :]
        return torch.cat([zc.real, zc.imag], dim=-1)
    def norm(z, g):
        return z * torch.rsqrt(z.pow(2).mean(-1, keepdim=True) + shape.rms_eps) * t(g)
    mask = torch.ones(T, T, dtype=torch.bool).tril()
    for l in range(shape.n_layers):
        a = norm(x, m.tensor(l, "norm1"))
        q = rotary((a @ t(m.tensor(l, "wq")).T).view(T, H, hd))
        k = rotary((a @ t(m.tensor(l, "wk")).T).view(T, Hk, hd))
        v = (a @ t(m.tensor(l, "wv")).T).view(T, Hk, hd)
        k = k.repeat_interleave(H // Hk, dim=1)
        v = v.repeat_interleave(H // Hk, dim=1)
        sc = torch.einsum("thd,shd->hts", q, k) / hd ** 0.5
        sc = sc.masked_fill(~mask, float("-inf"))
        o = torch.einsum("hts,shd->thd", torch.softmax(sc, dim=-1), v).reshape(T, H * hd)
        x = x + o @ t(m.tensor(l, "wo")).T
        a = norm(x, m.tensor(l, "norm2"))
        x = x + (torch.nn.functional.silu(a @ t(m.tensor(l, "wg")).T) * (a @ t(m.tensor(l, "wu")).T)) \
            @ t(m.tensor(l, "wd")).T
    return (norm(x, m.tensor(-1, "final_norm")) @ t(m.tensor(-1, "lm_head")).T).numpy()


def test_decoder_against_cacheless_torch_restatement():
    wl = small_workload(batch=1)
    m = W.Model(wl, keep=True)
    toks = synth.index_i32(9, 1, (1, 19), wl.shape.vocab).astype(np.int64)
    want = _torch_full_sequence_logits(m, wl.shape, toks[0])
    st = fresh(wl)
    L = range(wl.shape.n_layers)
    a = decoder.forward(m, wl.shape, L, st.full, st.lens, toks[:, :11], W.chain(10)); st.lens += 11
    b = decoder.forward(m, wl.shape, L, st.full, st.lens, toks[:, 11:], W.chain(7))
    got = np.concatenate([a[0], b[0]])
    assert np.abs(got - want).max() < 1e-9
    assert np.abs(want).max() > 0.5        # the comparison is not vacuous


def test_oracle_fp32_close_to_fp64():
    wl = small_workload(batch=1)
    m = W.Model(wl, keep=True)
    toks = synth.index_i32(9, 2, (1, 6), wl.shape.vocab).astype(np.int64)
    s64, s32 = fresh(wl), fresh(wl, dt=np.float32)
    a = decoder.forward(m, wl.shape, range(3), s64.full, s64.lens, toks, W.chain(5))
    b = decoder.forward(m, wl.shape, range(3), s32.full, s32.lens, toks, W.chain(5), dt=np.float32)
    assert b.dtype == np.float32 and np.abs(a - b).max() < 2e-4


# --------------------------------------------------------------------------
# tier rule
# --------------------------------------------------------------------------
def test_regions_golden():
    rows = [l.split() for l in open(os.path.join(GOLD, "regions_b1_b3.txt")) if l.strip() and l[0] != "#"]
    for c, region in rows:
        logits = np.log(np.array([1.0, float(c), 0.0001], dtype=np.float64)).astype(np.float32)
        d = tiers.log_confidence(logits, 1)
        # thresholds a hair below log(tau) so that c == tau lands on the ">=" side despite fp32 logs
        t = tiers.tier_of(d, np.log(0.3) - 1e-6, np.log(0.5) - 1e-6)
        assert t == int(region), (c, region, t)


def test_tier_partition_and_monotonicity():
    """Regions are exclusive and exhaustive (B.1-B.3); escalation shrinks as its threshold drops, the
    accept region grows as its threshold drops (Eq. B.18-B.19)."""
    wl = W.get("c1_tiny")
    si = W.step_inputs(replace(wl, batch=16, parent=W.chain(8)))
    prev_full, prev_acc = None, None
    for lo, hi in [(-6.0, -1.0), (-5.0, -1.0), (-4.0, -1.5), (-3.0, -2.0), (-3.0, -3.0)]:
        tier, d = tiers.tier_rule(si.drafter_logits, si.draft_tok, si.prow, lo, hi)
        assert set(np.unique(tier)) <= {0, 1, 2}
        assert np.array_equal(tier == 0, d >= np.float32(hi))
        assert np.array_equal(tier == 2, d < np.float32(lo))
        assert np.array_equal(tier == 1, (d >= np.float32(lo)) & (d < np.float32(hi)))
        assert np.all(d <= 0)
    lo_sweep = [int((tiers.tier_rule(si.drafter_logits, si.draft_tok, si.prow, lo, 0.0)[0] == 2).sum())
                for lo in (-1.0, -2.0, -3.0, -5.0, -8.0)]
    assert lo_sweep == sorted(lo_sweep, reverse=True) and lo_sweep[0] > lo_sweep[-1]
    hi_sweep = [int((tiers.tier_rule(si.drafter_logits, si.draft_tok, si.prow, -50.0, hi)[0] == 0).sum())
                for hi in (0.0, -1.0, -2.0, -4.0, -8.0)]
    assert hi_sweep == sorted(hi_sweep) and hi_sweep[0] < hi_sweep[-1]


def test_quantile_thresholds_brute_force():
    rng = np.random.default_rng(3)
    d = -np.abs(rng.standard_normal(1000)).astype(np.float32)
    lo, hi = tiers.quantile_thresholds(d, 0.40, 0.75)
    t = np.array([tiers.tier_of(x, lo, hi) for x in d])
    # nearest rank: exactly 399 values lie strictly below P40 (-> full), 250 lie above P75
    assert (t == 2).sum() == 399 and (t == 0).sum() == 251 and (t == 1).sum() == 350


# --------------------------------------------------------------------------
# acceptance rule: exact enumeration
# --------------------------------------------------------------------------
def _rand_dist(rng, n, sharp=1.5):
    z = rng.standard_normal(n) * sharp
    e = np.exp(z - z.max())
    return e / e.sum()


def _enumerate_single(p, j, alpha, beta):
    """Exact output distribution and rejection probability of (A.2, A.3) for one drafted token ~ p."""
    out = np.zeros_like(p)
    rej = 0.0
    for v in range(len(p)):
        if p[v] == 0:
            continue
        a = min(1.0, float(np.exp(tiers.log_accept_ratio(j, p, v, alpha))))
        out[v] += p[v] * a
        out += p[v] * (1 - a) * tiers.residual(j, p, beta)
        rej += p[v] * (1 - a)
    return out, rej


def test_lossless_case_reproduces_judge_distribution():
    """alpha = 0, beta = 1: the emitted token is distributed exactly as the judge (App. A, lossless case)."""
    rng = np.random.default_rng(0)
    for n in (4, 6, 8):
        p, q = _rand_dist(rng, n), _rand_dist(rng, n)
        out, rej = _enumerate_single(p, q, 0.0, 1.0)
        assert np.allclose(out, q, atol=1e-12)
        assert np.isclose(rej, 0.5 * np.abs(p - q).sum(), atol=1e-12)        # Eq. 2-3


def test_rejection_rate_golden_and_lossy_form():
    for line in open(os.path.join(GOLD, "tv_rejection.txt")):
        if not line.strip() or line[0] == "#":
            continue
        ps, qs, tv = [x.strip() for x in line.split(";")]
        p = np.array([float(x) for x in ps.split(",")]); q = np.array([float(x) for x in qs.split(",")])
        _, rej = _enumerate_single(p, q, 0.0, 1.0)
        assert np.isclose(rej, float(tv), atol=1e-12)
    # alpha > 0: rejection probability of A.2 is sum max(0, p - q / (1 - alpha))
    rng = np.random.default_rng(5)
    p, q = _rand_dist(rng, 7), _rand_dist(rng, 7)
    for alpha in (0.1, 0.3):
        _, rej = _enumerate_single(p, q, alpha, 1.0 - alpha)
        assert np.isclose(rej, np.maximum(0, p - q / (1 - alpha)).sum(), atol=1e-12)
        assert rej < 0.5 * np.abs(p - q).sum()          # a lossy gate rejects less


def test_multi_child_without_replacement_is_lossless():
    """Siblings drawn one after another without replacement from p, judged in order with the residual
    updated after each rejection: the emitted token is still distributed as the judge."""
    rng = np.random.default_rng(1)
    n = 5
    p, q = _rand_dist(rng, n), _rand_dist(rng, n)
    for n_children in (2, 3):
        out = np.zeros(n)

        def rec(prob, prop, judge, left):
            if left == 0:
                out[:] += prob * judge                                  # final draw from the residual
                return
            for v in range(n):
                if prop[v] <= 0:
                    continue
                a = min(1.0, float(np.exp(tiers.log_accept_ratio(judge, prop, v, 0.0))))
                out[v] += prob * prop[v] * a
                if a < 1.0:
                    rec(prob * prop[v] * (1 - a), tiers.drop_token(prop, v),
                        tiers.residual(judge, prop, 1.0), left - 1)
        rec(1.0, p, q, n_children)
        assert np.allclose(out, q, atol=1e-12), n_children


def _fake_logits(dist):
    with np.errstate(divide="ignore"):
        return np.log(dist)


def test_resolve_sampling_monte_carlo_matches_judges():
    """The RNG path (hash -> uniform -> accept test; Gumbel-max draw) through resolve_sequence itself:
    tier 2 emits ~ q, tier 1 emits ~ q', tier 0 keeps the draft."""
    rng = np.random.default_rng(2)
    V, n_trials = 6, 24000
    p, qs, qf = _rand_dist(rng, V), _rand_dist(rng, V), _rand_dist(rng, V)
    dl = _fake_logits(p)[None, :]
    sl = np.stack([_fake_logits(qs)] * 2); fl = np.stack([_fake_logits(qf)] * 2)
    draws = rng.choice(V, size=n_trials, p=p)
    for t, target in ((2, qf), (1, qs)):
        cnt = np.zeros(V)
        nrej = 0
        for i in range(n_trials):
            P = tiers.Params(mode="sampling", seed=1234, step=i)
            r = tiers.resolve_sequence(0, [int(draws[i])], (-1,), (0,), (t,), dl, sl, fl, P)
            assert len(r.out_tok) == 1
            cnt[r.out_tok[0]] += 1
            nrej += r.n_acc == 0
            assert r.corr_src == (0 if r.n_acc else t)
        assert np.abs(cnt / n_trials - target).max() < 0.012, (t, cnt / n_trials, target)
        assert abs(nrej / n_trials - 0.5 * np.abs(p - target).sum()) < 0.012
    r = tiers.resolve_sequence(0, [3], (-1,), (0,), (0,), dl, sl, fl, tiers.Params(mode="sampling"))
    assert r.out_tok == [3] and r.n_acc == 1 and r.corr_src == 0


def test_sampling_bonus_token_is_a_draw_from_the_full_verifier_at_the_leaf():
    """emit_bonus in sampling mode: when the whole draft is accepted, one more token is drawn from q at
    the last accepted row (not the pending row, not q')."""
    rng = np.random.default_rng(5)
    V, n_trials = 6, 20000
    q_root, q_leaf, qs = _rand_dist(rng, V), _rand_dist(rng, V), _rand_dist(rng, V)
    assert np.abs(q_root - q_leaf).max() > 0.1 and np.abs(qs - q_leaf).max() > 0.1
    fl = np.stack([_fake_logits(q_root), _fake_logits(q_leaf)])
    sl = np.stack([_fake_logits(qs)] * 2)
    dl = np.zeros((1, V))
    cnt = np.zeros(V)
    for i in range(n_trials):
        P = tiers.Params(mode="sampling", seed=77, step=i, emit_bonus=True)
        r = tiers.resolve_sequence(0, [2], (-1,), (0,), (0,), dl, sl, fl, P)      # tier 0: always accepted
        assert r.n_acc == 1 and r.out_tok[0] == 2 and len(r.out_tok) == 2 and r.corr_src == 2
        cnt[r.out_tok[1]] += 1
    assert np.abs(cnt / n_trials - q_leaf).max() < 0.012, (cnt / n_trials, q_leaf)
    # a temperature reshapes the draw: T = 2 gives softmax(log q / 2)
    t2 = np.sqrt(q_leaf) / np.sqrt(q_leaf).sum()
    cnt = np.zeros(V)
    for i in range(n_trials):
        P = tiers.Params(mode="sampling", seed=78, step=i, emit_bonus=True, temperature=2.0)
        cnt[tiers.resolve_sequence(0, [2], (-1,), (0,), (0,), dl, sl, fl, P).out_tok[1]] += 1
    assert np.abs(cnt / n_trials - t2).max() < 0.012
    # without the flag nothing is added
    r = tiers.resolve_sequence(0, [2], (-1,), (0,), (0,), dl, sl, fl, tiers.Params(mode="sampling"))
    assert r.out_tok == [2] and r.corr_src == 0


def test_uniform_hash_statistics_and_streams():
    k = tiers.stream_key(1, 2, 3, tiers.STREAM_GUMBEL)
    u = tiers.unit_vec(k, 5 << 32, 200000)
    assert 0 < u.min() and u.max() < 1
    assert abs(u.mean() - 0.5) < 0.003 and abs(u.var() - 1 / 12) < 0.002
    assert u[7] == tiers.unit(k, (5 << 32) + 7)                      # scalar and vector forms agree
    assert tiers.stream_key(1, 2, 3, 0) != tiers.stream_key(1, 2, 3, 1) != tiers.stream_key(1, 3, 3, 1)
    g = -np.log(-np.log(u))
    assert abs(g.mean() - 0.5772) < 0.01                             # Gumbel mean = Euler's constant


# --------------------------------------------------------------------------
# greedy resolution
# --------------------------------------------------------------------------
def test_greedy_chain_cases():
    V = 5
    def row(best, second=None):
        r = np.zeros(V); r[best] = 2.0
        if second is not None:
            r[second] = 1.5
        return r
    par, prow = W.chain(3), (0, 1, 2)
    dl = np.zeros((3, V))
    full = np.stack([row(1), row(2), row(3), row(4)])
    slim = np.stack([row(1), row(0), row(3), row(4)])
    P = tiers.Params()
    # all tier 2, draft = q's own greedy continuation: everything accepted, nothing added
    r = tiers.resolve_sequence(0, [1, 2, 3], par, prow, (2, 2, 2), dl, slim, full, P)
    assert (r.n_acc, r.path, r.out_tok, r.corr_src) == (3, [0, 1, 2], [1, 2, 3], 0)
    # with the bonus flag the full verifier's next token is appended
    r = tiers.resolve_sequence(0, [1, 2, 3], par, prow, (2, 2, 2), dl, slim, full,
                               tiers.Params(emit_bonus=True))
    assert r.out_tok == [1, 2, 3, 4] and r.corr_src == 2
    # tier 1 at the second node: q' disagrees (argmax 0) -> rewrite with q', suffix dropped
    r = tiers.resolve_sequence(0, [1, 2, 3], par, prow, (2, 1, 2), dl, slim, full, P)
    assert (r.n_acc, r.out_tok, r.corr_src) == (1, [1, 0], 1)
    assert list(r.judge) == [1 | 32, 2 | 16, 0]
    # tier 0 is never judged even when both verifiers disagree
    r = tiers.resolve_sequence(0, [1, 4, 3], par, prow, (2, 0, 2), dl, slim, full, P)
    assert r.n_acc == 3 and r.out_tok == [1, 4, 3] and list(r.judge) == [1 | 32, 1, 1 | 32]
    # wrong token at a tier-2 node: q's argmax replaces it
    r = tiers.resolve_sequence(0, [1, 0, 3], par, prow, (1, 2, 2), dl, slim, full, P)
    assert (r.n_acc, r.out_tok, r.corr_src) == (1, [1, 2], 2)
    # strict break: an accepted tier-1 token still ends the block (Algorithm 2 as printed)
    r = tiers.resolve_sequence(0, [1, 2, 3], par, prow, (1, 2, 2), dl, slim, full,
                               tiers.Params(strict_break=True))
    assert (r.n_acc, r.out_tok, r.corr_src) == (0, [1], 1)
    # relaxed greedy gate: runner-up within log_acc_rel passes
    full2 = np.stack([row(1, 3), row(2), row(3), row(4)])
    r = tiers.resolve_sequence(0, [3, 2, 3], par, prow, (2, 2, 2), dl, slim, full2,
                               tiers.Params(log_acc_rel=(0.0, 0.0, -0.6)))
    assert r.n_acc >= 1 and r.out_tok[0] == 3
    r = tiers.resolve_sequence(0, [3, 2, 3], par, prow, (2, 2, 2), dl, slim, full2,
                               tiers.Params(log_acc_rel=(0.0, 0.0, -0.4)))
    assert (r.n_acc, r.out_tok) == (0, [1])


def test_greedy_tree_picks_matching_child():
    V = 6
    par = W.small_tree()                       # (-1,-1,-1,0,0,3,1); rows = node + 1
    prow, _ = W.drafter_rows(par)
    tok = [2, 3, 4, 1, 5, 0, 2]
    full = np.zeros((8, V)); slim = np.zeros((8, V))
    full[0, 3] = 1; full[2, 2] = 1             # root -> node 1 (tok 3); row 2 -> node 6 (tok 2)
    full[7, 4] = 1
    r = tiers.resolve_sequence(0, tok, par, prow, [2] * 7, np.zeros((4, V)), slim, full, tiers.Params())
    assert r.path == [1, 6] and r.out_tok == [3, 2] and r.corr_src == 0      # leaf reached
    full[2, 2] = 0; full[2, 5] = 1             # now row 2 wants token 5: node 6 rejected
    r = tiers.resolve_sequence(0, tok, par, prow, [2] * 7, np.zeros((4, V)), slim, full, tiers.Params())
    assert r.path == [1] and r.out_tok == [3, 5] and r.corr_src == 2
    assert r.judge[0] == (2 | 32) and r.judge[1] == (1 | 32) and r.judge[2] == 0


# --------------------------------------------------------------------------
# whole loop
# --------------------------------------------------------------------------
@pytest.mark.parametrize("parent", [W.chain(4), W.small_tree()])
def test_all_full_tier_greedy_equals_autoregressive_decoding(parent):
    """Every token sent to the full tier, greedy: the emitted stream is q's greedy decoding, token for
    token, whatever the drafts are (Algorithm 1: accept the longest valid prefix, regenerate, discard)."""
    wl = small_workload(parent=parent, batch=2)
    m = W.Model(wl, keep=True)
    prompt = synth.index_i32(3, 1, (2, 9), wl.shape.vocab).astype(np.int64)
    st_ar = fresh(wl, cap=96)
    step.prefill(m, wl.shape, wl.routed, st_ar, prompt)
    ref = step.greedy_decode(m, wl.shape, st_ar, 24)

    st = fresh(wl, cap=96)
    step.prefill(m, wl.shape, wl.routed, st, prompt)
    emitted = [[], []]
    prow, R = W.drafter_rows(parent)
    N = len(parent)
    it = 0
    accepted_any = False
    while min(len(e) for e in emitted) < 20:
        # drafts: a mix of the true continuation (so that acceptances happen) and noise
        draft = synth.index_i32(77, it, (2, N), wl.shape.vocab).astype(np.int64)
        for b in range(2):
            k = len(emitted[b])
            depth = decoder.tree_layout(parent)[0][1:]
            for n in range(N):
                if (it + n + b) % 3 != 0 and parent[n] <= 0:
                    draft[b, n] = ref[b][k + depth[n] - 1]
        dl = np.zeros((2, R, wl.shape.vocab), dtype=np.float32)
        out = step.verify_step(m, wl.shape, wl.routed, st, draft, parent, prow, dl, 1.0, 2.0,
                               tiers.Params())            # thresholds above 0: every node is tier 2
        assert np.all(out.tier == 2)
        for b in range(2):
            assert 1 <= len(out.seqs[b].out_tok) <= max(decoder.tree_layout(parent)[0]) + 1
            emitted[b].extend(out.seqs[b].out_tok)
            accepted_any |= out.seqs[b].n_acc > 0
        it += 1
    assert accepted_any
    for b in range(2):
        n = min(len(emitted[b]), 24)
        assert emitted[b][:n] == ref[b][:n]
        # committed ids = prompt + emitted (minus the pending one); lengths agree
        assert st.lens[b] == 8 + len(emitted[b]) and st.pending[b] == emitted[b][-1]
        assert st.tokens[b] == list(prompt[b]) + emitted[b][:-1]


def test_self_draft_is_fully_accepted_and_slim_cache_stays_consistent():
    """Draft = q's own greedy continuation, tiers forced to 2: n_acc = K every time; and after commits
    the slim cache equals what a fresh slim prefill of the same tokens produces."""
    wl = small_workload(batch=1)
    m = W.Model(wl, keep=True)
    prompt = synth.index_i32(3, 2, (1, 6), wl.shape.vocab).astype(np.int64)
    st_ar = fresh(wl); step.prefill(m, wl.shape, wl.routed, st_ar, prompt)
    ref = step.greedy_decode(m, wl.shape, st_ar, 12)[0]
    st = fresh(wl); step.prefill(m, wl.shape, wl.routed, st, prompt)
    pos = 0
    for it in range(3):
        # pending = ref[pos-1] (or the last prompt token); the draft continues from ref[pos]
        draft = np.array([ref[pos:pos + 4]])
        out = step.verify_step(m, wl.shape, wl.routed, st, draft, W.chain(4), (0, 1, 2, 3),
                               np.zeros((1, 4, wl.shape.vocab), np.float32), 1.0, 2.0, tiers.Params())
        assert out.seqs[0].n_acc == 4 and out.seqs[0].out_tok == ref[pos:pos + 4]
        pos += 4
    st2 = fresh(wl)
    allt = np.array([list(prompt[0]) + ref[:pos]])
    step.prefill(m, wl.shape, wl.routed, st2, allt)
    assert st2.lens[0] == st.lens[0] and st2.pending[0] == st.pending[0]
    n = int(st.lens[0])
    for l in range(wl.n_routed):
        assert np.allclose(st.slim.k[l][0, :, :n], st2.slim.k[l][0, :, :n], atol=1e-10)
        assert np.allclose(st.slim.v[l][0, :, :n], st2.slim.v[l][0, :, :n], atol=1e-10)


def test_tree_commit_moves_accepted_rows():
    """After a tree step the cache must equal the cache of a chain step on the accepted path."""
    par = W.small_tree()
    wl = small_workload(parent=par, batch=1)
    m = W.Model(wl, keep=True)
    prompt = synth.index_i32(3, 5, (1, 5), wl.shape.vocab).astype(np.int64)
    st = fresh(wl); step.prefill(m, wl.shape, wl.routed, st, prompt)
    st_ar = fresh(wl); step.prefill(m, wl.shape, wl.routed, st_ar, prompt)
    ref = step.greedy_decode(m, wl.shape, st_ar, 4)[0]
    tok = synth.index_i32(3, 6, (1, 7), wl.shape.vocab).astype(np.int64)
    tok[0, 1] = ref[0]; tok[0, 6] = ref[1]          # accepted path: node 1 then node 6 (rows 2, 7)
    if tok[0, 0] == ref[0]: tok[0, 0] = (ref[0] + 1) % wl.shape.vocab
    if tok[0, 2] == ref[0]: tok[0, 2] = (ref[0] + 2) % wl.shape.vocab
    prow, R = W.drafter_rows(par)
    out = step.verify_step(m, wl.shape, wl.routed, st, tok, par, prow,
                           np.zeros((1, R, wl.shape.vocab), np.float32), 1.0, 2.0, tiers.Params())
    assert out.seqs[0].path == [1, 6] and out.seqs[0].out_tok == ref[:2]
    assert st.lens[0] == 4 + 2 and st.pending[0] == ref[1]
    st2 = fresh(wl)
    step.prefill(m, wl.shape, wl.routed, st2, np.array([list(prompt[0]) + ref[:2]]))
    for c, c2 in ((st.full, st2.full), (st.slim, st2.slim)):
        for l in range(c.n_layers):
            assert np.allclose(c.k[l][0, :, :6], c2.k[l][0, :, :6], atol=1e-10)
            assert np.allclose(c.v[l][0, :, :6], c2.v[l][0, :, :6], atol=1e-10)


# --------------------------------------------------------------------------
# Algorithm 2 as printed: the slim verifier's own confidence gates the tiers
# --------------------------------------------------------------------------
def _uniform_attention_logits(E, toks, n_layers, eps):
    """Closed form of the _OneLayerIdentity model on a chain: every layer adds to row i the mean of the
    normalised rows 0..i; the head is the identity, so the logits are the final norm of the stream."""
    nrm = lambda x: x / np.sqrt((x * x).mean(-1, keepdims=True) + eps)
    h = E[toks].astype(np.float64)
    for _ in range(n_layers):
        a = nrm(h)
        h = h + np.stack([a[:i + 1].mean(0) for i in range(len(toks))])
    return nrm(h)


def test_algorithm_2_gate_reads_the_slim_verifier_at_the_parent_row():
    """conf_source 1 through oracle.step.verify_step: a drafted token is placed by q'_{t+j}, the slim
    verifier's distribution that predicts its position (the row of its parent), with M' the maximum
    of that row (App. B, Eq. B.1-B.3; Algorithm 2, the per-position loop), and with strict_break the
    block ends exactly as the printed loop says.  The expected values come from the closed form of a
    model with uniform attention and from the loop of Algorithm 2 written out here."""
    s = W.ModelShape(2, 8, 2, 2, 4, 4, 8, dtype="f32")
    rng = np.random.default_rng(3)
    E = (rng.standard_normal((8, 8)) * 1.5).astype(np.float32)
    wts = _OneLayerIdentity(s, E)
    K, B = 3, 40
    log_lo, log_hi = np.log(0.3), np.log(0.75)
    routed = [0]
    seen_regions, seen_ends, discriminating = set(), set(), 0
    pend = rng.integers(0, 8, size=B)
    draft = rng.integers(0, 8, size=(B, K))
    st = step.new_state(s, 1, B, 16)
    st.pending[:] = pend
    dl = rng.standard_normal((B, K, 8)).astype(np.float32)           # drafter logits: must not be what gates
    out = step.verify_step(wts, s, routed, st, draft, W.chain(K), tuple(range(K)), dl, log_lo, log_hi,
                           tiers.Params(strict_break=True), conf_source=1, do_commit=False)
    region = lambda d: 0 if d >= np.float32(log_hi) else (1 if d >= np.float32(log_lo) else 2)
    for b in range(B):
        toks = np.concatenate([[pend[b]], draft[b]])
        S = _uniform_attention_logits(E, toks, 1, s.rms_eps)          # q' = layer 0 only
        F = _uniform_attention_logits(E, toks, 2, s.rms_eps)          # q = both layers
        assert np.allclose(out.slim_logits[b], S, atol=1e-9) and np.allclose(out.full_logits[b], F, atol=1e-9)
        S32 = S.astype(np.float32)
        want_tier = []
        for j in range(K):
            d_parent = np.float32(S32[j][draft[b, j]] - S32[j].max())         # row j predicts draft j
            d_own = np.float32(S32[j + 1][draft[b, j]] - S32[j + 1].max())    # the node's own row: the wrong one
            d_full = np.float32(F[j][draft[b, j]] - F[j].max())
            d_draft = np.float32(dl[b, j][draft[b, j]] - dl[b, j].max())
            want_tier.append(region(d_parent))
            discriminating += (region(d_own) != region(d_parent)) + (region(d_full) != region(d_parent)) \
                + (region(d_draft) != region(d_parent))
            assert out.conf[b, j] == d_parent
        assert list(out.tier[b]) == want_tier, (b, list(out.tier[b]), want_tier)
        seen_regions.update(want_tier)
        # Algorithm 2, lines of the per-position loop, greedy: accept in region A; in region B rewrite with q'
        # and break; in region C ask q, accept if it agrees, else rewrite with q and break
        emitted, src = [], 0
        for j in range(K):
            x = int(draft[b, j])
            if want_tier[j] == 0:
                emitted.append(x)
                continue
            judge = S if want_tier[j] == 1 else F
            if int(np.argmax(judge[j])) == x:                        # cannot happen in region B: x is below the mode
                emitted.append(x)
                assert want_tier[j] == 2
                continue
            emitted.append(int(np.argmax(judge[j])))
            src = want_tier[j]
            break
        r = out.seqs[b]
        assert r.out_tok == emitted and r.corr_src == src, (b, r.out_tok, emitted, r.corr_src, src)
        assert r.n_acc == len(emitted) - (1 if src else 0)
        seen_ends.add(src)
    assert seen_regions == {0, 1, 2} and seen_ends == {0, 1, 2}
    assert discriminating > 20          # the other candidate rows would have placed many tokens elsewhere


# --------------------------------------------------------------------------
# more than one slim verifier (the n-tier remark of Sec. 3.2; Table 1)
# --------------------------------------------------------------------------
def test_n_tier_rule_cuts_the_confidence_axis_and_contains_the_three_tier_rule():
    rng = np.random.default_rng(9)
    d = rng.uniform(-8.0, 0.0, size=400).astype(np.float32)
    taus = [-1.0, -2.5, -4.0, -6.5]                       # descending: five tiers
    t = np.array([tiers.tier_of_n(x, taus) for x in d])
    for k in range(5):
        hi = 0.0 if k == 0 else taus[k - 1]
        lo = -np.inf if k == 4 else taus[k]
        inside = (d >= np.float32(lo)) & ((d < np.float32(hi)) if k else np.ones_like(d, dtype=bool))
        assert np.array_equal(t == k, inside), k
    assert set(t) == {0, 1, 2, 3, 4}
    # two thresholds: exactly the three-tier rule of Eq. B.1-B.3
    assert [tiers.tier_of_n(x, [-2.0, -5.0]) for x in d] == [tiers.tier_of(x, -5.0, -2.0) for x in d]
    # lowering a threshold can only move tokens to a weaker tier
    t2 = np.array([tiers.tier_of_n(x, [-1.0, -3.0, -4.0, -6.5]) for x in d])
    assert (t2 <= t).all() and (t2 < t).any()


def test_n_tier_sampling_draws_from_the_judge_of_the_token_s_tier():
    """Four verifiers (five tiers): a tier-k token ends as a draw from verifier k (lossless rule, Eq. A.2-A.3 with
    u_k as the judge), rejected with probability D_TV(p, u_k); a full acceptance with the bonus flag draws from q."""
    rng = np.random.default_rng(4)
    V, n_trials = 6, 16000
    p = _rand_dist(rng, V)
    judges = [_rand_dist(rng, V) for _ in range(4)]
    dl = _fake_logits(p)[None, :]
    jl = [np.stack([_fake_logits(j)] * 2) for j in judges]
    draws = rng.choice(V, size=n_trials, p=p)
    for t in (1, 2, 3, 4):
        cnt, nrej = np.zeros(V), 0
        for i in range(n_trials):
            P = tiers.Params(mode="sampling", seed=99, step=i)
            r = tiers.resolve_sequence_n(0, [int(draws[i])], (-1,), (0,), (t,), dl, jl, P)
            cnt[r.out_tok[0]] += 1
            nrej += r.n_acc == 0
            assert r.corr_src == (0 if r.n_acc else t)
        assert np.abs(cnt / n_trials - judges[t - 1]).max() < 0.015, (t, cnt / n_trials, judges[t - 1])
        assert abs(nrej / n_trials - 0.5 * np.abs(p - judges[t - 1]).sum()) < 0.015
    r = tiers.resolve_sequence_n(0, [2], (-1,), (0,), (0,), dl, jl, tiers.Params(mode="sampling", emit_bonus=True, seed=5))
    assert r.n_acc == 1 and r.corr_src == 4 and len(r.out_tok) == 2


def test_n_tier_greedy_cases():
    V = 6
    def row(best):
        r = np.zeros(V); r[best] = 2.0
        return r
    par, prow, dl = W.chain(3), (0, 1, 2), np.zeros((3, V))
    u1 = np.stack([row(1), row(5), row(5), row(5)])      # weakest verifier
    u2 = np.stack([row(1), row(2), row(4), row(5)])
    q = np.stack([row(1), row(2), row(3), row(0)])
    J = [u1, u2, q]
    # every node in the tier of a verifier that agrees: all accepted, nothing added; the bonus comes from q
    r = tiers.resolve_sequence_n(0, [1, 2, 3], par, prow, (1, 2, 3), dl, J, tiers.Params())
    assert (r.n_acc, r.out_tok, r.corr_src) == (3, [1, 2, 3], 0) and list(r.judge) == [1 | 16, 1 | 32, 1 | 48]
    r = tiers.resolve_sequence_n(0, [1, 2, 3], par, prow, (1, 2, 3), dl, J, tiers.Params(emit_bonus=True))
    assert r.out_tok == [1, 2, 3, 0] and r.corr_src == 3
    # the second node left to the weakest verifier, which wants token 5: it rewrites, the rest is dropped
    r = tiers.resolve_sequence_n(0, [1, 2, 3], par, prow, (1, 1, 3), dl, J, tiers.Params())
    assert (r.n_acc, r.out_tok, r.corr_src) == (1, [1, 5], 1) and list(r.judge) == [1 | 16, 2 | 16, 0]
    # the third node left to the middle verifier (wants 4): replacement from it, not from q (wants 3)
    r = tiers.resolve_sequence_n(0, [1, 2, 3], par, prow, (3, 3, 2), dl, J, tiers.Params())
    assert (r.n_acc, r.out_tok, r.corr_src) == (2, [1, 2, 4], 2)
    # Algorithm 2's literal break applies to every slim verifier's acceptance, not to q's
    r = tiers.resolve_sequence_n(0, [1, 2, 3], par, prow, (3, 2, 3), dl, J, tiers.Params(strict_break=True))
    assert (r.n_acc, r.out_tok, r.corr_src) == (1, [1, 2], 2)
    # two verifiers: the three-tier walk
    a = tiers.resolve_sequence_n(0, [1, 2, 0], par, prow, (1, 2, 2), dl, [u2, q], tiers.Params())
    b = tiers.resolve_sequence(0, [1, 2, 0], par, prow, (1, 2, 2), dl, u2, q, tiers.Params())
    assert (a.n_acc, a.out_tok, a.corr_src, list(a.judge)) == (b.n_acc, b.out_tok, b.corr_src, list(b.judge)) == (2, [1, 2, 3], 2, [17, 33, 34])
