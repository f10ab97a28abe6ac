"""Pins the oracle's acceptance arithmetic to closed forms of speculative
sampling, to a library logsumexp, and to brute force on tiny vocabularies."""
import itertools

import numpy as np
import pytest
from scipy.special import logsumexp as sp_lse, softmax as sp_softmax

from oracle import accept as A
from oracle import philox


def _rows(rng, L, V, scale=2.0):
    return rng.standard_normal((L, V)) * scale, rng.standard_normal((L, V)) * scale


def test_logsumexp_and_softmax_match_library():
    rng = np.random.default_rng(0)
    for _ in range(5):
        row = rng.standard_normal(1000) * 30
        assert abs(A.logsumexp(row) - sp_lse(row)) < 1e-12 * max(1, abs(sp_lse(row)))
        np.testing.assert_allclose(A.softmax(row), sp_softmax(row), rtol=1e-12, atol=0)
    assert abs(A.logsumexp(np.array([1000.0, 1000.0])) - (1000 + np.log(2))) < 1e-12


def test_sample_from_logits_greedy_fields():
    row = np.log(np.array([0.1, 0.5, 0.15, 0.25]))
    s = A.sample_from_logits(row)
    assert s.xhat == 1 and abs(s.d - 0.5) < 1e-15 and abs(s.top1 - 0.5) < 1e-15
    assert abs(s.margin - 0.25) < 1e-15
    h = -sum(p * np.log(p) for p in (0.1, 0.5, 0.15, 0.25))
    assert abs(s.entropy - h) < 1e-14
    tie = A.sample_from_logits(np.array([0.0, 2.0, 2.0, 1.0]))
    assert tie.xhat == 1 and tie.margin == 0.0          # ties -> lowest id


def test_sample_mode_is_inverse_cdf():
    row = np.log(np.array([0.2, 0.3, 0.5]))
    assert A.sample_from_logits(row, "sample", 0.1).xhat == 0
    assert A.sample_from_logits(row, "sample", 0.25).xhat == 1
    assert A.sample_from_logits(row, "sample", 0.75).xhat == 2
    assert abs(A.sample_from_logits(row, "sample", 0.25).d - 0.3) < 1e-15


def test_identical_distributions_accept_everything():
    rng = np.random.default_rng(1)
    dl, _ = _rows(rng, 6, 50)
    xhat = rng.integers(0, 50, size=6)
    for u in (1e-9, 0.5, 1 - 2.0 ** -25):
        r = A.accept_scan(dl, dl + 3.7, xhat, [u] * 6, [0.3] * 6)   # a constant shift leaves softmax unchanged
        assert r.n_accepted == 6 and r.first_reject == -1 and r.resampled == -1


def test_strict_inequality_and_stop_at_first_rejection():
    dl = np.log(np.array([[0.5, 0.5], [0.5, 0.5], [0.5, 0.5]]))
    vl = np.log(np.array([[0.25, 0.75], [0.25, 0.75], [0.25, 0.75]]))
    a = A.accept_scan(dl, vl, [0, 0, 0], [0.0, 0.0, 0.0], [0.1] * 3).a
    assert all(abs(x - 0.5) < 1e-15 for x in a)
    below = float(np.nextafter(a[1], 0.0))
    r = A.accept_scan(dl, vl, [0, 0, 0], [below, a[1], 0.0], [0.1, 0.1, 0.1])
    assert r.n_accepted == 1 and r.first_reject == 1       # u == a rejects (strict <), u just below accepts
    assert r.resampled == 1                                 # residual mass only on token 1
    assert len(r.a) == 2                                    # position 2 never scanned


def test_ratio_tempering_exponent():
    assert abs(A.accept_probability(0.5, 0.125, gamma=0.5) - 0.5) < 1e-15
    assert A.accept_probability(0.2, 0.4, gamma=3.0) == 1.0


def test_residual_is_a_distribution_and_excludes_rejected_token():
    rng = np.random.default_rng(2)
    for _ in range(20):
        dl, vl = _rows(rng, 1, 40)
        r = A.residual_weights(vl[0], dl[0])
        pv, pd = sp_softmax(vl[0]), sp_softmax(dl[0])
        assert (r >= 0).all() and r.sum() > 0
        assert np.all(r[pv <= pd] == 0)
        # total residual mass equals the total-variation distance
        assert abs(r.sum() - 0.5 * np.abs(pv - pd).sum()) < 1e-12
        rn = r / r.sum()
        assert abs(rn.sum() - 1) < 1e-12
        # any token that can be rejected (v < d) has zero residual mass, so a
        # resampled token never equals the rejected proposal
        for x in np.where(pv < pd)[0][:5]:
            for u in (0.0, 0.3, 0.999999):
                assert A.resample_residual(vl[0], dl[0], u) != x


def test_inverse_cdf_brute_force_and_monotone():
    rng = np.random.default_rng(3)
    w = rng.random(7)
    w[2] = 0.0
    c = np.cumsum(w)
    prev = -1
    for u in np.linspace(0, 1, 2001)[:-1]:
        k = A.inverse_cdf(w, u)
        brute = next(i for i in range(7) if c[i] > u * c[-1])
        assert k == brute and k >= prev and k != 2
        prev = k
    assert A.inverse_cdf(w, 0.0) == 0
    assert A.inverse_cdf(np.array([0.0, 0.0, 1.0]), 0.0) == 2


def _interval_midpoints(weights):
    """Midpoint u of each token's inverse-CDF interval and its measure."""
    c = np.concatenate([[0.0], np.cumsum(weights)]) / np.sum(weights)
    return [((c[i] + c[i + 1]) / 2, c[i + 1] - c[i]) for i in range(len(weights)) if c[i + 1] > c[i]], c


def test_single_position_output_law_is_the_verifiers():
    """x̂ ~ pi_d, accept w.p. min(1, v/d), else residual  =>  output ~ pi_v (V = 6).
    The integral over the two uniforms is exact: the scan is piecewise constant
    in them, each piece is visited once at an interior point and weighted by its measure."""
    rng = np.random.default_rng(4)
    V = 6
    for _ in range(10):
        dl, vl = _rows(rng, 1, V, 1.5)
        pd, pv = sp_softmax(dl[0]), sp_softmax(vl[0])
        law = np.zeros(V)
        for x in range(V):
            a = min(1.0, pv[x] / pd[x])
            acc = A.accept_scan(dl, vl, [x], [a / 2], [0.5])
            assert acc.n_accepted == 1 and abs(acc.a[0] - a) < 1e-14
            law[x] += pd[x] * a
            if a < 1:
                mids, _ = _interval_midpoints(np.maximum(pv - pd, 0))
                for u2, meas in mids:
                    rej = A.accept_scan(dl, vl, [x], [(1 + a) / 2], [u2])
                    assert rej.n_accepted == 0 and rej.first_reject == 0
                    law[rej.resampled] += pd[x] * (1 - a) * meas
        np.testing.assert_allclose(law, pv, rtol=0, atol=1e-13)


def test_multi_position_law_with_ar_completion_is_the_verifier_chain():
    """V = 3, L = 3.  Drafts are independent per position (as a diffusion draft is);
    the verifier is an AR chain whose row i depends on the tokens to its left.
    Committed tokens completed by sampling the remaining positions from the verifier
    must follow the verifier's joint law exactly."""
    rng = np.random.default_rng(5)
    V, L = 3, 3
    dl = rng.standard_normal((L, V))
    table = {pre: rng.standard_normal(V) for k in range(L) for pre in itertools.product(range(V), repeat=k)}
    pd = np.array([sp_softmax(r) for r in dl])
    pv = {pre: sp_softmax(r) for pre, r in table.items()}

    def chain(seq):
        return np.prod([pv[tuple(seq[:i])][seq[i]] for i in range(len(seq))])

    def complete(prefix):
        """law over V^L of prefix followed by AR samples from the verifier"""
        out = {}
        for tail in itertools.product(range(V), repeat=L - len(prefix)):
            seq = tuple(prefix) + tail
            out[seq] = np.prod([pv[seq[:i]][seq[i]] for i in range(len(prefix), L)])
        return out

    law = {seq: 0.0 for seq in itertools.product(range(V), repeat=L)}
    for xhat in itertools.product(range(V), repeat=L):
        p_draft = np.prod([pd[i][xhat[i]] for i in range(L)])
        vl = np.array([table[tuple(xhat[:i])] for i in range(L)])       # verifier rows given drafts to the left
        a = [min(1.0, pv[tuple(xhat[:i])][xhat[i]] / pd[i][xhat[i]]) for i in range(L)]
        # every accept pattern: accept 0..k-1, reject k (or accept all)
        for k in range(L + 1):
            w_acc = np.prod(a[:k])
            if k == L:
                res = A.accept_scan(dl, vl, xhat, [x / 2 for x in a], [0.5] * L)
                assert res.n_accepted == L and res.first_reject == -1
                law[tuple(xhat)] += p_draft * w_acc
                continue
            if a[k] >= 1:
                continue
            u = [x / 2 for x in a[:k]] + [(1 + a[k]) / 2] + [0.0] * (L - k - 1)
            mids, _ = _interval_midpoints(np.maximum(pv[tuple(xhat[:k])] - pd[k], 0))
            for u2, meas in mids:
                res = A.accept_scan(dl, vl, xhat, u, [u2] * L)
                assert res.n_accepted == k and res.first_reject == k
                prefix = tuple(xhat[:k]) + (res.resampled,)
                for seq, pr in complete(prefix).items():
                    law[seq] += p_draft * w_acc * (1 - a[k]) * meas * pr
    for seq in law:
        assert abs(law[seq] - chain(seq)) < 1e-13, seq
    assert abs(sum(law.values()) - 1) < 1e-12


def test_greedy_draft_closed_form():
    """With x̂ = argmax pi_d the output law is [w = x*] a + (1 - a) r(w)."""
    rng = np.random.default_rng(6)
    dl, vl = _rows(rng, 1, 5, 1.0)
    pd, pv = sp_softmax(dl[0]), sp_softmax(vl[0])
    x = int(np.argmax(pd))
    a = min(1.0, pv[x] / pd[x])
    r = np.maximum(pv - pd, 0)
    r = r / r.sum()
    want = (1 - a) * r
    want[x] += a
    got = np.zeros(5)
    s = A.sample_from_logits(dl[0])
    assert s.xhat == x
    got[x] += a
    if a < 1:
        for u2, meas in _interval_midpoints(np.maximum(pv - pd, 0))[0]:
            got[A.accept_scan(dl, vl, [x], [(1 + a) / 2], [u2]).resampled] += (1 - a) * meas
    np.testing.assert_allclose(got, want, atol=1e-13)


def test_expected_accepted_length_monte_carlo():
    """P(n_acc >= k) = prod_{i<=k} a_i and E[n_acc] = sum_k prod_{i<=k} a_i,
    over Philox uniforms of many (sequence, step) counters."""
    rng = np.random.default_rng(7)
    L, V, N = 4, 12, 4000
    dl, _ = _rows(rng, L, V, 1.0)
    vl = dl + 0.4 * rng.standard_normal((L, V))
    xhat = [int(np.argmax(r)) for r in dl]
    a = [min(1.0, sp_softmax(vl[i])[xhat[i]] / sp_softmax(dl[i])[xhat[i]]) for i in range(L)]
    assert 0.05 < np.prod(a) < 0.95
    counts = np.zeros(L + 1)
    for n in range(N):
        u = [philox.uniform(1, i, n, 0, philox.STREAM_ACCEPT) for i in range(L)]
        u2 = [philox.uniform(1, i, n, 0, philox.STREAM_RESAMPLE) for i in range(L)]
        counts[A.accept_scan(dl, vl, xhat, u, u2).n_accepted] += 1
    mean = (counts * np.arange(L + 1)).sum() / N
    want = sum(np.prod(a[:k]) for k in range(1, L + 1))
    assert abs(mean - want) < 5 * L / np.sqrt(N) / 2
    for k in range(1, L + 1):
        p = np.prod(a[:k])
        assert abs(counts[k:].sum() / N - p) < 5 * np.sqrt(p * (1 - p) / N) + 1e-3


def test_threshold_select():
    assert A.threshold_select([0.2, 0.95, 0.5], [1, 2, 5], 0.9) == [2]
    assert A.threshold_select([0.2, 0.3, 0.1], [1, 2, 5], 0.9) == [2]           # argmax always taken
    assert A.threshold_select([0.95, 0.3, 0.99], [0, 2, 3], 0.9) == [0, 3]
    assert A.threshold_select([0.4, 0.4], [2, 3], 0.9) == [2]                    # ties -> leftmost
    assert A.threshold_select([0.4, 0.7, 0.2], [0, 1, 2], 1.0) == [1]            # tau = 1: static, one per step
