"""CPU oracle, part 4: KL-style verification cost of one judge against one proposal.

TEST INFRASTRUCTURE ONLY.

Plain numpy in float64, written from the paper's definitions:

* single-step cost with the positive-part margin (Eq. 11): for log-probabilities lp = log p_t, lq = log q_t,
  z1(v) = log(1 - alpha) + lp(v) - lq(v),  z2(v) = log(beta) + lp(v) - lq(v),
  R(q || p) = sum_v p(v) phi(z1(v)) + sum_v q(v) phi(z2(v)),  phi(z) = max(0, z);
* the smooth margin of App. F: phi_tau(z) = tau log(1 + exp(z / tau));
* block cost (Eq. 10): the sum of the single-step costs over the decoding steps of a block;
* gain of the routed path p -> u -> q over the direct path p -> q (Sec. 2.2):
  Delta = C(q || p) - C(u || p) - C(q || u).

Nothing here is shared with the CUDA path; only tests, the smoke check and the benchmark's CPU leg may import it.
"""
from __future__ import annotations

import numpy as np


def log_softmax64(logits: np.ndarray, temperature: float = 1.0) -> np.ndarray:
    x = np.asarray(logits, dtype=np.float64) / float(temperature)
    x = x - x.max(axis=-1, keepdims=True)
    return x - np.log(np.exp(x).sum(axis=-1, keepdims=True))


def margin(z: np.ndarray, phi: str = "relu", tau: float = 1.0) -> np.ndarray:
    """phi(z): "relu" = max(0, z) (Eq. 11); "softplus" = tau log(1 + exp(z / tau)) (App. F)."""
    if phi == "relu":
        return np.maximum(z, 0.0)
    if phi == "softplus":
        return tau * np.logaddexp(0.0, z / tau)
    raise ValueError(phi)


def step_cost(judge_logits: np.ndarray, proposal_logits: np.ndarray, alpha: float = 0.0, beta: float = 1.0,
              temperature: float = 1.0, phi: str = "relu", tau: float = 1.0) -> np.ndarray:
    """R(q || p) per row (Eq. 11): q = softmax(judge_logits / T), p = softmax(proposal_logits / T); [..., V] -> [...]."""
    lq = log_softmax64(judge_logits, temperature)
    lp = log_softmax64(proposal_logits, temperature)
    z1 = np.log1p(-alpha) + lp - lq
    z2 = np.log(beta) + lp - lq
    return (np.exp(lp) * margin(z1, phi, tau)).sum(axis=-1) + (np.exp(lq) * margin(z2, phi, tau)).sum(axis=-1)


def block_cost(judge_logits: np.ndarray, proposal_logits: np.ndarray, **kw) -> float:
    """C(q || p | pi) (Eq. 10): the single-step costs summed over the rows (decoding steps) given."""
    return float(step_cost(judge_logits, proposal_logits, **kw).sum())


def routed_gain(proposal_logits: np.ndarray, middle_logits: np.ndarray, judge_logits: np.ndarray, **kw) -> float:
    """Delta (Sec. 2.2): cost of p -> q minus the cost of p -> u -> q; positive when the routed path is cheaper."""
    return (block_cost(judge_logits, proposal_logits, **kw) - block_cost(middle_logits, proposal_logits, **kw)
            - block_cost(judge_logits, middle_logits, **kw))
