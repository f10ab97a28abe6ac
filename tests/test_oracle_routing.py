"""Hand-computed values for the routing arithmetic (Eq. khat, the static and
dynamic scores, and the policies of Algorithm DoVerify)."""
import math

from oracle import routing as R


def test_khat_hand_values():
    assert R.khat([]) == 0.0
    assert R.khat([1, 1, 1]) == 3.0
    assert abs(R.khat([0.5, 0.5, 0.5]) - (0.5 + 0.25 + 0.125)) < 1e-15
    assert R.khat([1, 0, 1, 1]) == 1.0                       # a zero stops the prefix
    assert abs(R.khat([0.9, 0.8]) - (0.9 + 0.72)) < 1e-15


def test_alpha_proxies():
    assert R.alpha_margin([0.2, 0.05, 0.1], 0.1) == [1.0, 0.0, 1.0]
    a = R.alpha_entropy([0.0, math.log(50)], beta=2.0, vocab=50)
    assert a[0] == 1.0 and abs(a[1] - math.exp(-2.0)) < 1e-15


def test_scores_and_policies():
    assert R.score(2.5, 1.0) == 1.5
    assert R.score(2.5, 0.5, n_hi=3) == 1.0
    assert R.n_hi([0.95, 0.5, 0.91], 0.9) == 2
    assert R.min_span(1) and not R.min_span(1, 2) and R.min_span(4, 4)
    assert R.score_threshold(0.0, 0.0) and not R.score_threshold(-1e-9, 0.0)


def test_hysteresis_sequence():
    h = R.Hysteresis(tau_on=1.0, tau_off=0.0, on=True)
    assert [h(s) for s in (0.5, -0.1, 0.5, 0.99, 1.0, 0.2, -0.5)] == [True, False, False, False, True, True, False]


def test_mean_conf_rule():
    assert R.mean_conf([0.5, 0.95]) and not R.mean_conf([0.95, 0.95]) and not R.mean_conf([0.9, 0.9])
