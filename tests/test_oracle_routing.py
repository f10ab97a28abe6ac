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


def test_ucb_router_hand_computed_sequence():
    """Eq. (ucb) on a short sequence worked out by hand (beta = 1, block 8, two bins per dimension)."""
    r = R.UCBRouter(beta=1.0, block_size=8, vocab=100, bins=2)
    lo = [0.1 * math.log(100)] * 3          # normalised entropy 0.1 -> entropy bin 0
    # buckets: span 3 of 8 -> bin 0 ((3-1)*2//8 = 0); nothing unmasked yet -> progress bin 0
    assert r.bucket(3, 8, lo) == (0, 0, 0)
    assert r.bucket(5, 8, lo) == (1, 0, 0) and r.bucket(8, 8, lo) == (1, 0, 0) and r.bucket(4, 8, lo) == (0, 0, 0)
    assert r.bucket(2, 4, lo) == (0, 1, 0) and r.bucket(2, 5, lo) == (0, 0, 0)      # 4 of 8 unmasked -> bin 1; 3 of 8 -> bin 0
    assert r.bucket(3, 8, [0.7 * math.log(100)] * 3) == (0, 0, 1)
    # t = 1: both actions untried, the tie goes to verification; the step decodes 3 tokens: reward 3 / 2
    assert r.decide(3, 8, lo) is True
    r.update(3)
    # t = 2: action 0 is untried in this bucket -> taken; decodes 1 token: reward 1 / 1
    assert r.decide(3, 8, lo) is False
    r.update(1)
    # t = 3: 1.5 + sqrt(ln 3 / 1) against 1.0 + sqrt(ln 3 / 1) -> verify; decodes 1 token: reward 0.5, mean of action 1 -> 1.0
    assert abs(r.index(1, (0, 0, 0)) - (1.5 + math.sqrt(math.log(2)))) < 1e-12       # index() reads the current t = 2
    assert r.decide(3, 8, lo) is True
    r.update(1)
    # t = 4: action 1: 1.0 + sqrt(ln 4 / 2) = 1.8326; action 0: 1.0 + sqrt(ln 4 / 1) = 2.1774 -> no verification
    assert r.decide(3, 8, lo) is False
    assert abs(r.index(1, (0, 0, 0)) - (1.0 + math.sqrt(math.log(4) / 2))) < 1e-12
    assert abs(r.index(0, (0, 0, 0)) - (1.0 + math.sqrt(math.log(4)))) < 1e-12
    r.update(2)
    # another bucket starts from scratch (verify first), but t keeps counting
    assert r.decide(8, 8, lo) is True and r.t == 5
    r.update(8)
    assert r.n[(1, (1, 0, 0))] == 1 and r.sum[(1, (1, 0, 0))] == 4.0
    # the caller may override the action actually taken (flags given to the verifier differ from the decision)
    r.decide(8, 8, lo)
    r.update(2, action=0)
    assert r.n[(0, (1, 0, 0))] == 1 and r.sum[(0, (1, 0, 0))] == 2.0
