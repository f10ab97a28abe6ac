"""Vocabulary-wide arithmetic of the decode step in fp64 (oracle; test
infrastructure only): SampleFromLogits / ScoreFromLogits, the speculative
acceptance scan with residual resampling (Algorithm "SampleBlock for S2D2",
the left-to-right loop), and the confidence-threshold branch taken when
verification is skipped (same algorithm, else-branch; also Algorithm
"SampleBlock for standard BD3").

Naming: pi_d is the drafter's distribution (the paper's P_l with probability
p_i for the drafted token), pi_v the verifier's (the paper's P_l^ver with
q_i).  d_i = pi_d,i(xhat_i), v_i = pi_v,i(xhat_i).  Accept iff
u_i < min(1, (v_i / d_i)^gamma), strict, gamma = 1 by default (Appendix
"ratio tempering" gives the exponent).  At the first rejection the token is
redrawn from (pi_v - pi_d)_+ normalised, by inverse CDF in vocabulary order
with one uniform, and the scan stops.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np


def logsumexp(row: np.ndarray) -> float:
    row = np.asarray(row, dtype=np.float64)
    m = row.max()
    return float(m + np.log(np.exp(row - m).sum()))


def softmax(row: np.ndarray) -> np.ndarray:
    row = np.asarray(row, dtype=np.float64)
    return np.exp(row - logsumexp(row))


def inverse_cdf(weights: np.ndarray, u: float) -> int:
    """Smallest index w with sum_{w' <= w} weights[w'] > u * sum(weights)."""
    c = np.cumsum(np.asarray(weights, dtype=np.float64))
    t = u * c[-1]
    w = int(np.searchsorted(c, t, side="right"))
    return min(w, len(c) - 1)


@dataclass
class DraftStats:
    xhat: int          # proposed token
    d: float           # pi_d(xhat)
    top1: float        # largest draft probability
    margin: float      # top-1 minus top-2 draft probability
    entropy: float     # Shannon entropy of pi_d (nats)
    lse: float


def sample_from_logits(row: np.ndarray, mode: str = "greedy", u: Optional[float] = None) -> DraftStats:
    """SampleFromLogits: proposal xhat and its confidence from draft logits.

    greedy: xhat = argmax (ties -> lowest id), confidence = its full softmax
    probability.  sample: xhat ~ pi_d by inverse CDF with the given uniform."""
    row = np.asarray(row, dtype=np.float64)
    lse = logsumexp(row)
    p = np.exp(row - lse)
    order_top = int(np.argmax(row))
    if mode == "greedy":
        xhat = order_top
    elif mode == "sample":
        xhat = inverse_cdf(p, float(u))
    else:
        raise ValueError(mode)
    top1 = float(p[order_top])
    rest = np.delete(p, order_top)
    top2 = float(rest.max()) if rest.size else 0.0
    nz = p > 0
    entropy = float(-(p[nz] * (row[nz] - lse)).sum())
    return DraftStats(xhat, float(p[xhat]), top1, top1 - top2, entropy, lse)


def score_from_logits(row: np.ndarray, token: int) -> float:
    """ScoreFromLogits: probability of ``token`` under softmax(row)."""
    return float(np.exp(float(row[token]) - logsumexp(row)))


def accept_probability(d: float, v: float, gamma: float = 1.0) -> float:
    ratio = v / d
    if gamma != 1.0:
        ratio = ratio ** gamma
    return min(1.0, ratio)


def residual_weights(verify_row: np.ndarray, draft_row: np.ndarray) -> np.ndarray:
    """Unnormalised residual (pi_v - pi_d)_+ over the vocabulary."""
    return np.maximum(softmax(verify_row) - softmax(draft_row), 0.0)


def resample_residual(verify_row: np.ndarray, draft_row: np.ndarray, u: float) -> int:
    r = residual_weights(verify_row, draft_row)
    if not r.sum() > 0.0:      # cannot follow a true rejection in exact arithmetic
        return inverse_cdf(softmax(verify_row), u)
    return inverse_cdf(r, u)


@dataclass
class AcceptResult:
    n_accepted: int                 # accepted drafted tokens (prefix length)
    first_reject: int               # index in the span of the first rejection, -1 if none
    resampled: int                  # token drawn from the residual, -1 if none
    v: List[float] = field(default_factory=list)      # verifier probs scanned so far
    a: List[float] = field(default_factory=list)      # acceptance probabilities
    margin_u: List[float] = field(default_factory=list)   # |u_i - a_i| for boundary counting


def accept_scan(draft_logits: np.ndarray, verify_logits: np.ndarray, xhat: Sequence[int],
                u_accept: Sequence[float], u_resample: Sequence[float],
                gamma: float = 1.0, resample: bool = True) -> AcceptResult:
    """Left-to-right scan over a drafted span of length L.

    draft_logits / verify_logits: [L, V] rows of the drafter and of the
    verifier for the same positions; u_accept[i], u_resample[i] the uniforms
    of position i.  ``resample=False`` is the "reject only" variant that stops
    without committing a replacement."""
    L = len(xhat)
    res = AcceptResult(0, -1, -1)
    for i in range(L):
        d_i = score_from_logits(draft_logits[i], int(xhat[i]))
        v_i = score_from_logits(verify_logits[i], int(xhat[i]))
        a_i = accept_probability(d_i, v_i, gamma)
        res.v.append(v_i)
        res.a.append(a_i)
        res.margin_u.append(abs(float(u_accept[i]) - a_i))
        if float(u_accept[i]) < a_i:
            res.n_accepted += 1
            continue
        res.first_reject = i
        if resample:
            res.resampled = resample_residual(verify_logits[i], draft_logits[i], float(u_resample[i]))
        break
    return res


def threshold_select(d: Sequence[float], masked: Sequence[int], tau: float) -> List[int]:
    """S = {i in M_t : d_i > tau} ∪ {argmax_{i in M_t} d_i} (ties -> leftmost).
    ``d`` is indexed like ``masked`` (one confidence per masked position)."""
    masked = list(masked)
    d = list(d)
    best = max(range(len(masked)), key=lambda k: (d[k], -k))
    return sorted({masked[k] for k in range(len(masked)) if d[k] > tau} | {masked[best]})
