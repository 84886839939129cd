"""Pins for the oracle's region masses (Eq. B.4-B.10): closed forms, the link to the tier rule, and sampling."""
import numpy as np

from oracle import tiers


def _rows(seed, n, v, sigma=2.0):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((n, v)) * sigma).astype(np.float32)


def test_masses_sum_to_one_and_are_probabilities():
    gate, prop = _rows(1, 6, 500), _rows(2, 6, 500)
    m = tiers.region_masses(gate, prop, np.log(0.05), np.log(0.4), temperature=0.8)
    assert m.shape == (6, 3) and np.all(m >= 0.0)
    assert np.allclose(m.sum(axis=-1), 1.0, atol=1e-12)          # delta_p + delta_1bar + delta_2 = 1 (below Eq. B.6)


def test_uniform_proposal_counts_tokens_per_region():
    # p uniform: each mass is the fraction of the vocabulary in the region (Eq. B.8-B.10 with p(u) = 1 / V)
    gate = np.array([[0.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -9.0]], dtype=np.float32)
    m = tiers.region_masses(gate, np.zeros((1, 8), np.float32), log_tau_lo=-2.0, log_tau_hi=-1.0)
    assert np.allclose(m[0], [3 / 8, 2 / 8, 3 / 8])               # d >= -1: 3 tokens; -2 <= d < -1: 2; below: 3


def test_two_token_closed_form():
    # gate l = (0, -x): token 1 has relative confidence e^{-x}; proposal logits (a, 0): p = (s, 1 - s), s = sigmoid(a)
    x, a = 1.2, 0.7
    s = 1.0 / (1.0 + np.exp(-a))
    gate, prop = np.array([[0.0, -x]], np.float32), np.array([[a, 0.0]], np.float32)
    assert np.allclose(tiers.region_masses(gate, prop, -2.0, -1.5)[0], [1.0, 0.0, 0.0])       # both tokens above tau_hi
    assert np.allclose(tiers.region_masses(gate, prop, -2.0, -1.0)[0], [s, 1.0 - s, 0.0])     # token 1 in region B
    assert np.allclose(tiers.region_masses(gate, prop, -1.0, -0.5)[0], [s, 0.0, 1.0 - s])     # token 1 in region C


def test_region_of_every_token_is_the_tier_rule():
    # brute force: the mask behind each mass is tier_of(log_confidence(.)) token by token (Eq. B.1-B.3)
    gate, prop = _rows(3, 3, 200), _rows(4, 3, 200)
    lo, hi = np.log(0.02), np.log(0.3)
    m = tiers.region_masses(gate, prop, lo, hi)
    for r in range(3):
        p = tiers.softmax64(prop[r], 1.0)
        want = np.zeros(3)
        for u in range(200):
            want[tiers.tier_of(tiers.log_confidence(gate[r], u), lo, hi)] += p[u]
        assert np.allclose(m[r], want, atol=1e-12)


def test_degenerate_thresholds():
    gate, prop = _rows(5, 4, 300), _rows(6, 4, 300)
    same = tiers.region_masses(gate, prop, np.log(0.1), np.log(0.1))
    assert np.all(same[:, 1] == 0.0)                               # tau_lo = tau_hi: region B is empty
    none_c = tiers.region_masses(gate, prop, -np.inf, np.log(0.1))
    assert np.all(none_c[:, 2] == 0.0)                             # tau_lo = 0: nothing escalates
    all_a = tiers.region_masses(gate, prop, -np.inf, -np.inf)
    assert np.allclose(all_a[:, 0], 1.0)
    only_mode = tiers.region_masses(gate, prop, 0.0, 0.0)          # tau = 1: only the gate's mode is accepted outright
    p = np.stack([tiers.softmax64(prop[r], 1.0) for r in range(4)])
    assert np.allclose(only_mode[:, 0], p[np.arange(4), gate.argmax(axis=-1)])


def test_tier_frequencies_of_sampled_drafts_converge_to_the_masses():
    # Eq. B.4-B.6 define the deltas as probabilities over v ~ p; Eq. B.8-B.10 are their sums over the vocabulary
    gate, prop = _rows(7, 1, 400), _rows(8, 1, 400)
    lo, hi = np.log(0.03), np.log(0.35)
    m = tiers.region_masses(gate, prop, lo, hi)[0]
    p = tiers.softmax64(prop[0], 1.0)
    rng = np.random.default_rng(9)
    n = 40000
    toks = rng.choice(400, size=n, p=p)
    t, _ = tiers.tier_rule(gate[None], toks[None], [0] * n, lo, hi)
    freq = np.bincount(t[0], minlength=3) / n
    assert np.all(np.abs(freq - m) < 4.0 * np.sqrt(m * (1 - m) / n) + 1e-4), (freq, m)


def test_output_mixture_is_a_distribution():
    # Eq. B.7: pi = delta_p p + delta_1bar q' + delta_2 q is a convex combination of three distributions
    gate, prop, full = _rows(10, 2, 100), _rows(11, 2, 100), _rows(12, 2, 100)
    m = tiers.region_masses(gate, prop, np.log(0.05), np.log(0.5))
    for r in range(2):
        mix = m[r, 0] * tiers.softmax64(prop[r], 1.0) + m[r, 1] * tiers.softmax64(gate[r], 1.0) + m[r, 2] * tiers.softmax64(full[r], 1.0)
        assert abs(mix.sum() - 1.0) < 1e-12 and np.all(mix >= 0.0)
