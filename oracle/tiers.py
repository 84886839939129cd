"""CPU oracle, part 2: confidence tiers, tiered acceptance, prefix resolution.

TEST INFRASTRUCTURE ONLY.  Plain numpy / Python loops restating the paper's
verification cycle; nothing in the product may import it, and it shares no code
with the CUDA sources.

Tier rule (App. B, Eq. B.1-B.3): a drafted token v is placed by its confidence
relative to the mode of the gating distribution m, c = m(v) / max_u m(u):
region A (accept) c >= tau_hi, region B (slim verifier decides) tau_lo <= c <
tau_hi, region C (escalate to the full verifier) c < tau_lo.  With logits the
test is d = l[v] - max_u l[u] compared with log tau; the log thresholds are the
inputs, so the decision is one fp32 subtraction and a comparison.
Readings taken where the paper leaves a choice:
thresholds are given directly as tau_hi >= tau_lo; the gating distribution is
the drafter's (conf_source 0) or the slim verifier's at the parent row
(conf_source 1, Algorithm 2 as printed).

Accept / resolve (Algorithm 2, the per-position loop; Algorithm 1, what gets
appended; App. A, Eq. A.2-A.3 for the sampling test and the residual):
walk from the pending token; at each step try the children of the current row
in index order; a tier-0 child is taken at once, a tier-1 child is judged by
q', a tier-2 child by q; greedy judging accepts when the token's logit is within
log_acc_rel of the judge's maximum (0 = it is the argmax), sampling judging
accepts with probability min(1, j(v) / ((1 - alpha) p(v))).  The first row where
no child passes ends the walk: the strongest judge that rejected there emits the
replacement token (argmax, or a draw from norm(max(0, j/beta - p))).  The
accepted path plus that token are emitted; if every level was accepted nothing
is added unless emit_bonus asks for a token from q at the leaf.

Region masses (Eq. B.4-B.10): the probability, under the proposal, that a drafted token falls in region A, B, C;
as sums over the vocabulary they are what the empirical tier frequencies converge to.

Random numbers: a counter-based hash of (seed, step, sequence, stream, index);
categorical draws use the Gumbel-max form so that no prefix sum is involved.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_MASK = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15


# --------------------------------------------------------------------------
# counter-based uniforms
# --------------------------------------------------------------------------
def _mix(z: int) -> int:
    z &= _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def stream_key(seed: int, step: int, b: int, stream: int) -> int:
    k = _mix(seed + _GAMMA)
    k = _mix(k + step * _GAMMA + 1)
    return _mix(k + (b * 256 + stream) * _GAMMA + 2)


def unit(key: int, idx: int) -> float:
    """Uniform on (0, 1) with 23 random bits, ((word >> 41) + 0.5) / 2^23: exact in fp32, never 0 or 1."""
    return ((_mix(key + idx * _GAMMA + 3) >> 41) + 0.5) * 2.0 ** -23


def unit_vec(key: int, idx0: int, n: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        idx = np.uint64(idx0) + np.arange(n, dtype=np.uint64)
        z = np.uint64(key) + idx * np.uint64(_GAMMA) + np.uint64(3)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return ((z >> np.uint64(41)).astype(np.float64) + 0.5) * 2.0 ** -23


STREAM_ACCEPT, STREAM_GUMBEL = 0, 1


# --------------------------------------------------------------------------
# tier rule
# --------------------------------------------------------------------------
def log_confidence(src_row: np.ndarray, tok: int) -> np.float32:
    """d = l[v] - max_u l[u], in the fp32 the logits are stored in."""
    r = np.asarray(src_row, dtype=np.float32)
    return np.float32(r[tok] - r.max())


def tier_of(d: np.float32, log_tau_lo: float, log_tau_hi: float) -> int:
    if d >= np.float32(log_tau_hi):
        return 0
    if d >= np.float32(log_tau_lo):
        return 1
    return 2


def tier_of_n(d: np.float32, log_taus: Sequence[float]) -> int:
    """More than one slim verifier (Sec. 3.2, the n-tier remark; Table 1): descending log thresholds cut the
    confidence axis into len(log_taus) + 1 tiers, tier 0 accepted outright, tier k judged by verifier k, the
    last tier by the full verifier."""
    for k, t in enumerate(log_taus):
        if d >= np.float32(t):
            return k
    return len(log_taus)


def tier_rule_n(conf_logits: np.ndarray, draft_tok: np.ndarray, src_row: Sequence[int], log_taus: Sequence[float]):
    B, N = draft_tok.shape
    tier = np.zeros((B, N), dtype=np.uint8)
    d = np.zeros((B, N), dtype=np.float32)
    for b in range(B):
        for n in range(N):
            d[b, n] = log_confidence(conf_logits[b, src_row[n]], int(draft_tok[b, n]))
            tier[b, n] = tier_of_n(d[b, n], log_taus)
    return tier, d


def tier_rule(conf_logits: np.ndarray, draft_tok: np.ndarray, src_row: Sequence[int],
              log_tau_lo: float, log_tau_hi: float):
    """conf_logits [B, R, V]; src_row[n] = which row gates node n.  Returns tier [B,N] u8, d [B,N] f32."""
    B, N = draft_tok.shape
    tier = np.zeros((B, N), dtype=np.uint8)
    d = np.zeros((B, N), dtype=np.float32)
    for b in range(B):
        for n in range(N):
            d[b, n] = log_confidence(conf_logits[b, src_row[n]], int(draft_tok[b, n]))
            tier[b, n] = tier_of(d[b, n], log_tau_lo, log_tau_hi)
    return tier, d


def region_masses(gate_logits: np.ndarray, proposal_logits: np.ndarray, log_tau_lo: float, log_tau_hi: float,
                  temperature: float = 1.0) -> np.ndarray:
    """(delta_p, delta_1bar, delta_2) per row (Eq. B.8-B.10): how much of the proposal p = softmax(proposal / T) lies on
    the tokens that the gating row places in region A, B and C (Eq. B.1-B.3).  [..., V] x2 -> [..., 3].

    A token's region is decided exactly as tier_of decides a drafted token's: d = l[u] - max l in the fp32 the logits
    are stored in, compared with the fp32 log thresholds.  The masses are sums of p in float64.
    """
    g = np.asarray(gate_logits, dtype=np.float32)
    d = g - g.max(axis=-1, keepdims=True)
    in_a = d >= np.float32(log_tau_hi)
    in_b = ~in_a & (d >= np.float32(log_tau_lo))
    z = np.asarray(proposal_logits, dtype=np.float64) / float(temperature)
    z = z - z.max(axis=-1, keepdims=True)
    p = np.exp(z)
    p = p / p.sum(axis=-1, keepdims=True)
    return np.stack([(p * in_a).sum(axis=-1), (p * in_b).sum(axis=-1), (p * ~(in_a | in_b)).sum(axis=-1)], axis=-1)


def quantile_thresholds(d: np.ndarray, q_lo: float, q_hi: float):
    """Nearest-rank quantiles of a sample of log-confidences: sorted[ceil(q n) - 1]."""
    s = np.sort(np.asarray(d, dtype=np.float32))
    n = len(s)
    pick = lambda q: s[max(0, int(np.ceil(q * n)) - 1)]
    return np.float32(pick(q_lo)), np.float32(pick(q_hi))


# --------------------------------------------------------------------------
# accept / resolve
# --------------------------------------------------------------------------
@dataclass
class Params:
    mode: str = "greedy"                 # "greedy" or "sampling"
    temperature: float = 1.0
    alpha: float = 0.0                   # Eq. A.2
    beta: float = 1.0                    # Eq. A.3; beta >= 1 - alpha
    log_acc_rel: Sequence[float] = (0.0, 0.0, 0.0)
    strict_break: bool = False           # a tier-1 acceptance still ends the block (Alg. 2 as printed)
    emit_bonus: bool = False
    seed: int = 0
    step: int = 0


@dataclass
class Decision:
    kind: str            # "accept" (a judged child) or "draw" (replacement / bonus token)
    row: int             # block row whose logits were read
    judge: int           # 1 slim, 2 full
    margin: float        # distance of the deciding quantity from its flip point (logit units)


@dataclass
class SeqResult:
    n_acc: int = 0
    path: List[int] = field(default_factory=list)
    out_tok: List[int] = field(default_factory=list)
    corr_src: int = 0
    judge: Optional[np.ndarray] = None   # [N] u8: 0 untouched, 1 accepted, 2 rejected, | tier << 4
    decisions: List[Decision] = field(default_factory=list)


def softmax64(logits: np.ndarray, temperature: float) -> np.ndarray:
    z = np.asarray(logits, dtype=np.float64) / temperature
    z = z - z.max()
    e = np.exp(z)
    return e / e.sum()


def log_accept_ratio(judge_dist: np.ndarray, proposal: np.ndarray, v: int, alpha: float) -> float:
    """log of j(v) / ((1 - alpha) p(v)); the token is accepted with probability min(1, that) (Eq. A.2)."""
    with np.errstate(divide="ignore"):
        return float(np.log(judge_dist[v]) - np.log1p(-alpha) - np.log(proposal[v]))


def residual(judge_dist: np.ndarray, proposal: np.ndarray, beta: float) -> np.ndarray:
    """norm(max(0, j / beta - p)) (Eq. A.3); j itself when that is identically zero."""
    nr = np.maximum(0.0, judge_dist / beta - proposal)
    s = nr.sum()
    return nr / s if s > 0.0 else judge_dist


def drop_token(proposal: np.ndarray, v: int) -> np.ndarray:
    """The proposal the next sibling was drawn from: v removed, renormalised."""
    p = proposal.copy()
    p[v] = 0.0
    s = p.sum()
    return p / s if s > 0.0 else p


def _top2_gap(x: np.ndarray) -> float:
    if x.size < 2:
        return float("inf")
    i = int(np.argmax(x))
    rest = np.delete(x, i)
    return float(x[i] - rest.max())


def gumbel_draw(dist: np.ndarray, key: int, row: int):
    """argmax_v (log dist[v] - log(-log u_v)): a draw from dist.  Returns (token, top-2 gap)."""
    V = dist.shape[0]
    u = unit_vec(key, row << 32, V)
    with np.errstate(divide="ignore"):
        score = np.log(dist) - np.log(-np.log(u))
    return int(np.argmax(score)), _top2_gap(score)


def resolve_sequence(b: int, tok: Sequence[int], parent: Sequence[int], prow: Sequence[int],
                     tier: Sequence[int], drafter_logits: np.ndarray, slim_logits: np.ndarray,
                     full_logits: np.ndarray, P: Params) -> SeqResult:
    """One sequence.  drafter_logits [R, V]; slim_logits / full_logits [M, V] (row 0 = pending)."""
    return resolve_sequence_n(b, tok, parent, prow, tier, drafter_logits, [slim_logits, full_logits], P)


def resolve_sequence_n(b: int, tok: Sequence[int], parent: Sequence[int], prow: Sequence[int],
                       tier: Sequence[int], drafter_logits: np.ndarray, judge_logits: Sequence[np.ndarray],
                       P: Params) -> SeqResult:
    """The same walk with J = len(judge_logits) verifiers, weakest first and the full verifier last (Sec. 3.2,
    n-tier remark): a tier-k child is judged by verifier k; J = 2 is the three-tier method.  The greedy gate of
    the slim verifiers is log_acc_rel[1], the full verifier's log_acc_rel[2]."""
    J = len(judge_logits)
    full_logits = judge_logits[J - 1]
    gate = lambda t: P.log_acc_rel[1] if t < J else P.log_acc_rel[2]
    N = len(parent)
    children = [[] for _ in range(N + 1)]
    for n, p in enumerate(parent):
        children[p + 1].append(n)
    res = SeqResult(judge=np.zeros(N, dtype=np.uint8))
    sampling = P.mode == "sampling"
    k_acc = stream_key(P.seed, P.step, b, STREAM_ACCEPT)
    k_gum = stream_key(P.seed, P.step, b, STREAM_GUMBEL)
    L = {k + 1: judge_logits[k] for k in range(J)}
    cur = 0
    corr = None
    while True:
        C = children[cur]
        if not C:
            if P.emit_bonus:
                if sampling:
                    corr, gap = gumbel_draw(softmax64(full_logits[cur], P.temperature), k_gum, cur)
                else:
                    row = np.asarray(full_logits[cur])
                    corr, gap = int(np.argmax(row)), _top2_gap(row)
                res.corr_src = J
                res.decisions.append(Decision("draw", cur, J, gap))
            break
        if sampling:
            r = {k: softmax64(L[k][cur], P.temperature) for k in L}
            ptil = softmax64(drafter_logits[prow[C[0]]], P.temperature)
        failed, taken = 0, None
        for c in C:
            v, t = int(tok[c]), int(tier[c])
            if t == 0:
                taken = c
                res.judge[c] = 1
                break
            if sampling:
                u = unit(k_acc, c)
                lr = log_accept_ratio(r[t], ptil, v, P.alpha)
                ok = bool(np.log(u) < lr)                 # u < j(v) / ((1 - alpha) p(v)), Eq. A.2
                margin = abs(float(lr - np.log(u)))
            else:
                row = np.asarray(L[t][cur])
                dlt = float(row[v] - row.max()) - float(gate(t))
                ok = dlt >= 0.0
                if gate(t) == 0.0:                        # argmax test: flip point is the runner-up
                    margin = _top2_gap(row) if ok else -dlt
                else:
                    margin = abs(dlt)
            res.decisions.append(Decision("accept", cur, t, margin))
            if ok:
                taken = c
                res.judge[c] = 1 | (t << 4)
                break
            res.judge[c] = 2 | (t << 4)
            failed = max(failed, t)
            if sampling:
                # Eq. A.3 applied round by round: the rejecting judge's distribution becomes its
                # residual against the proposal; the rejected token leaves the proposal.
                r[t] = residual(r[t], ptil, P.beta)
                ptil = drop_token(ptil, v)
        if taken is not None:
            if P.strict_break and 1 <= int(tier[taken]) < J:
                corr, res.corr_src = int(tok[taken]), int(tier[taken])
                res.judge[taken] = 1 | (int(tier[taken]) << 4)
                break
            res.path.append(taken)
            cur = taken + 1
            continue
        res.corr_src = failed
        if sampling:
            corr, gap = gumbel_draw(r[failed], k_gum, cur)
        else:
            row = np.asarray(L[failed][cur])
            corr, gap = int(np.argmax(row)), _top2_gap(row)
        res.decisions.append(Decision("draw", cur, failed, gap))
        break
    res.n_acc = len(res.path)
    res.out_tok = [int(tok[n]) for n in res.path] + ([corr] if corr is not None else [])
    return res


def resolve_n(draft_tok: np.ndarray, parent: Sequence[int], prow: Sequence[int], tier: np.ndarray,
              drafter_logits: np.ndarray, judge_logits: Sequence[np.ndarray], P: Params) -> List[SeqResult]:
    return [resolve_sequence_n(b, draft_tok[b], parent, prow, tier[b], drafter_logits[b],
                               [j[b] for j in judge_logits], P) for b in range(draft_tok.shape[0])]


def resolve(draft_tok: np.ndarray, parent: Sequence[int], prow: Sequence[int], tier: np.ndarray,
            drafter_logits: np.ndarray, slim_logits: np.ndarray, full_logits: np.ndarray,
            P: Params) -> List[SeqResult]:
    return [resolve_sequence(b, draft_tok[b], parent, prow, tier[b], drafter_logits[b],
                             slim_logits[b], full_logits[b], P) for b in range(draft_tok.shape[0])]
