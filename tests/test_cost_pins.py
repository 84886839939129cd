"""Pins of the KL-style cost oracle (Eq. 9-11, App. F) against things other than itself: closed forms on two tokens,
the identity that ties the positive-part sums to the KL divergence (computed by scipy), the softplus sandwich of
App. F (F.8), monotonicity in alpha and beta, and a pure-Python brute force."""
import math
import os

import numpy as np
import pytest
from scipy.special import rel_entr

from oracle import cost

HERE = os.path.dirname(os.path.abspath(__file__))


def _logits_of(p):
    return np.log(np.asarray(p, dtype=np.float64))


def test_two_token_closed_forms():
    rows = [l.split("#")[0].split() for l in open(os.path.join(HERE, "golden", "kl_cost_two_tokens.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 5
    for a, b, alpha, beta, want in [[float(x) for x in r] for r in rows]:
        got = cost.step_cost(_logits_of([b, 1 - b]), _logits_of([a, 1 - a]), alpha=alpha, beta=beta)
        assert abs(got - want) < 1e-12, (a, b, alpha, beta, got, want)


def test_equal_distributions_cost_nothing_and_temperature_only_rescales_logits():
    rng = np.random.default_rng(1)
    l = rng.normal(size=(3, 50))
    assert np.allclose(cost.step_cost(l, l), 0.0, atol=1e-15)
    m = rng.normal(size=(3, 50))
    assert np.allclose(cost.step_cost(l, m, temperature=2.0), cost.step_cost(l / 2.0, m / 2.0))
    # softmax ignores a constant added to a row
    assert np.allclose(cost.step_cost(l + 3.0, m - 1.5), cost.step_cost(l, m))


def test_positive_part_sums_differ_by_the_kl_divergence():
    # sum_v p max(0, log p/q) - sum_v p max(0, log q/p) = sum_v p log(p/q) = KL(p || q); scipy computes the right side
    rng = np.random.default_rng(2)
    lp, lq = rng.normal(size=(4, 200)) * 2, rng.normal(size=(4, 200)) * 2
    p, q = np.exp(cost.log_softmax64(lp)), np.exp(cost.log_softmax64(lq))
    kl_pq = rel_entr(p, q).sum(-1)
    kl_qp = rel_entr(q, p).sum(-1)
    pos_p = (p * np.maximum(0, np.log(p / q))).sum(-1)          # first term of Eq. 11 at alpha = 0
    pos_q = (q * np.maximum(0, np.log(p / q))).sum(-1)          # second term at beta = 1
    r = cost.step_cost(lq, lp)                                  # judge q, proposal p
    assert np.allclose(r, pos_p + pos_q)
    # each positive part exceeds its signed sum: first term >= KL(p || q); and the second equals
    # sum_v q max(0, -log q/p) = (sum_v q |log q/p| - KL(q || p)) / 2
    assert np.all(pos_p >= kl_pq - 1e-12)
    assert np.allclose(pos_q, ((q * np.abs(np.log(q / p))).sum(-1) - kl_qp) / 2)
    assert np.allclose(pos_p, ((p * np.abs(np.log(p / q))).sum(-1) + kl_pq) / 2)


def test_softplus_sandwich():
    rng = np.random.default_rng(3)
    lp, lq = rng.normal(size=(5, 300)) * 3, rng.normal(size=(5, 300)) * 3
    for tau in (0.05, 0.5, 2.0):
        for alpha, beta in ((0.0, 1.0), (0.1, 0.8), (0.3, 1.5)):
            relu = cost.step_cost(lq, lp, alpha=alpha, beta=beta)
            soft = cost.step_cost(lq, lp, alpha=alpha, beta=beta, phi="softplus", tau=tau)
            assert np.all(soft >= relu - 1e-12)
            assert np.all(soft <= relu + 2 * tau * math.log(2) + 1e-12)      # F.8


def test_monotone_in_alpha_and_beta():
    rng = np.random.default_rng(4)
    lp, lq = rng.normal(size=(6, 120)) * 2, rng.normal(size=(6, 120)) * 2
    prev = None
    for alpha in (0.0, 0.1, 0.3, 0.6):                  # a looser acceptance threshold can only lower the first term
        r = cost.step_cost(lq, lp, alpha=alpha)
        assert prev is None or np.all(r <= prev + 1e-12)
        prev = r
    prev = None
    for beta in (0.25, 0.5, 1.0, 2.0):                  # a larger beta can only raise the second term
        r = cost.step_cost(lq, lp, beta=beta)
        assert prev is None or np.all(r >= prev - 1e-12)
        prev = r


def test_brute_force_and_block_sum_and_routed_gain():
    rng = np.random.default_rng(5)
    lp, lu, lq = (rng.normal(size=(3, 7)) for _ in range(3))

    def brute(judge, prop, alpha, beta):
        out = []
        for jr, pr in zip(judge, prop):
            zq, zp = sum(math.exp(x) for x in jr), sum(math.exp(x) for x in pr)
            r = 0.0
            for v in range(len(jr)):
                pv, qv = math.exp(pr[v]) / zp, math.exp(jr[v]) / zq
                r += pv * max(0.0, math.log((1 - alpha) * pv / qv)) + qv * max(0.0, math.log(beta * pv / qv))
            out.append(r)
        return out

    for alpha, beta in ((0.0, 1.0), (0.2, 0.7)):
        want = brute(lq, lp, alpha, beta)
        assert np.allclose(cost.step_cost(lq, lp, alpha=alpha, beta=beta), want)
        assert abs(cost.block_cost(lq, lp, alpha=alpha, beta=beta) - sum(want)) < 1e-12
    gain = cost.routed_gain(lp, lu, lq)
    assert abs(gain - (sum(brute(lq, lp, 0, 1)) - sum(brute(lu, lp, 0, 1)) - sum(brute(lq, lu, 0, 1)))) < 1e-12
    # a middle distribution equal to the proposal or to the judge changes nothing
    assert abs(cost.routed_gain(lp, lp, lq)) < 1e-12 and abs(cost.routed_gain(lp, lq, lq)) < 1e-12
