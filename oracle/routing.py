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
