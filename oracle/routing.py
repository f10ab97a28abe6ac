"""Verification routing policies (oracle side; test infrastructure only).

Section "Verification Routing Policies": expected accepted prefix length
K_hat = sum_k prod_{i<=k} alpha_i (Eq. khat) with a margin proxy
alpha_i = 1[m_i >= tau_margin] or an entropy proxy alpha_i = exp(-beta H_i / log V);
scores s = K_hat - c (static) or K_hat - c * N_hi (dynamic); policies of
Algorithm "DoVerify": minimum span, score threshold, hysteresis.  The
"mean draft confidence" rule is the one the 4B-class synthetic workload names.
"""
from __future__ import annotations

import math
from typing import Sequence


def khat(alpha: Sequence[float]) -> float:
    total, prod = 0.0, 1.0
    for a in alpha:
        prod *= a
        total += prod
    return total


def alpha_margin(margins: Sequence[float], tau_margin: float):
    return [1.0 if m >= tau_margin else 0.0 for m in margins]


def alpha_entropy(entropies: Sequence[float], beta: float, vocab: int):
    return [math.exp(-beta * h / math.log(vocab)) for h in entropies]


def score(k_hat: float, c: float, n_hi: int = None) -> float:
    return k_hat - c if n_hi is None else k_hat - c * n_hi


def n_hi(d: Sequence[float], tau: float) -> int:
    return sum(1 for x in d if x > tau)


def min_span(span_len: int, tau_span: int = 1) -> bool:
    return span_len >= tau_span


def score_threshold(s: float, tau_score: float) -> bool:
    return s >= tau_score


class Hysteresis:
    def __init__(self, tau_on: float, tau_off: float, on: bool = True):
        self.tau_on, self.tau_off, self.on = tau_on, tau_off, on

    def __call__(self, s: float) -> bool:
        if self.on and s < self.tau_off:
            self.on = False
        elif (not self.on) and s >= self.tau_on:
            self.on = True
        return self.on


def mean_conf(d_masked: Sequence[float], tau: float = 0.9) -> bool:
    """Verify iff the mean draft confidence over the masked positions is below tau."""
    return (sum(d_masked) / len(d_masked)) < tau


class UCBRouter:
    """Contextual-bandit router (Appendix "Contextual-bandit routing policy", Eq. (ucb)).

    Two actions: 0 = confidence-threshold step without verification, 1 = verify the span.  At
    decision t (counted from 1 over all decisions of the router) in context bucket b the action is
    argmax_a mu_hat[a, b] + beta * sqrt(log t / n[a, b]); an action never taken in the bucket has an
    unbounded bonus, and ties go to verification.  The reward of a step is decoded tokens / cost with
    cost 2 for a verified step and 1 otherwise.  The bucket is the tuple (span-length bin, progress
    bin, entropy bin), each with ``bins`` equal bins: the span length 1..B partitioned linearly, the
    fraction of the block already unmasked, and the mean over the span of H_i / log V (the paper says
    only "normalized token entropy"; the mean over the span is the reading taken here)."""

    def __init__(self, beta: float, block_size: int, vocab: int, bins: int = 2):
        self.beta, self.B, self.V, self.bins = beta, block_size, vocab, bins
        self.t = 0
        self.n = {}        # (action, bucket) -> count
        self.sum = {}      # (action, bucket) -> summed reward
        self.last = None   # (bucket, action) awaiting its reward

    def bucket(self, span_len: int, n_masked: int, span_entropies: Sequence[float]):
        nb = self.bins
        b_span = min(nb - 1, (span_len - 1) * nb // self.B)
        b_prog = min(nb - 1, int((self.B - n_masked) * nb // self.B))
        h = sum(span_entropies) / (len(span_entropies) * math.log(self.V))
        b_ent = min(nb - 1, max(0, int(math.floor(h * nb))))
        return (b_span, b_prog, b_ent)

    def index(self, action: int, bucket) -> float:
        n = self.n.get((action, bucket), 0)
        if n == 0:
            return math.inf
        return self.sum[(action, bucket)] / n + self.beta * math.sqrt(math.log(self.t) / n)

    def decide(self, span_len: int, n_masked: int, span_entropies: Sequence[float]) -> bool:
        self.t += 1
        b = self.bucket(span_len, n_masked, span_entropies)
        a = 1 if self.index(1, b) >= self.index(0, b) else 0
        self.last = (b, a)
        return bool(a)

    def update(self, decoded: int, action: int = None):
        b, a = self.last
        a = a if action is None else int(action)
        r = decoded / (2.0 if a else 1.0)
        self.n[(a, b)] = self.n.get((a, b), 0) + 1
        self.sum[(a, b)] = self.sum.get((a, b), 0.0) + r
        self.last = None
