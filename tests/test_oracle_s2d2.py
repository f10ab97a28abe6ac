"""Pins the oracle's decode loop: the 2L verifier pass against L literal
single-row passes, block size 1 against greedy AR decoding, the incrementally
committed K/V against a literal end-of-block causal pass, and the behaviour
the algorithms fix (progress every step, stop at first rejection, resampled
token differs from the rejected proposal)."""
import numpy as np
import pytest

from oracle import model as M
from oracle import s2d2 as S
from oracle.accept import logsumexp
from s2d2_inputs import generate_prompts, generate_weights, get_config


def test_verifier_rows_equal_literal_single_position_passes(tiny_f32):
    """MASK-copy row i of the 2L pass conditions on the prefix and the drafted
    tokens to its left and keeps position i masked: identical to a pass of
    prefix ++ x̂_<i ++ [MASK] read at its last row."""
    wl, W = tiny_f32
    cfg = wl.model
    prompt = [5, 9, 2, 44, 17, 3, 8]
    n = len(prompt)
    _, kv = M.forward(W, cfg, prompt, np.arange(n), M.causal_mask(n), need_logits=[])
    cache = M.append_kv(None, kv, np.arange(n))
    xhat = [11, 4, 30, 7]
    L = len(xhat)
    vt, vp, vm = S.verify_pass_rows(xhat, list(range(n, n + L)), cfg.mask_id)
    # the mask is [[A, 0], [A<, I]]
    assert vm[:L, :L].tolist() == np.tril(np.ones((L, L), bool)).tolist()
    assert not vm[:L, L:].any()
    assert vm[L:, :L].tolist() == np.tril(np.ones((L, L), bool), -1).tolist()
    assert vm[L:, L:].tolist() == np.eye(L, dtype=bool).tolist()
    got, _ = M.forward(W, cfg, vt, vp, vm, cache, need_logits=list(range(L, 2 * L)))
    for i in range(L):
        seq = prompt + xhat[:i] + [cfg.mask_id]
        lit, _ = M.forward(W, cfg, seq, np.arange(len(seq)), M.causal_mask(len(seq)))
        np.testing.assert_allclose(got[i], lit[-1], rtol=1e-9, atol=1e-11)


def test_block_size_one_is_greedy_autoregressive(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=4)[0][:9]
    seq = S.SequenceOracle(W, cfg, block_size=1, seed=1, seq_stream=0, keep_logits=True)
    out = seq.generate(prompt, 10)
    assert out == S.greedy_ar_decode(W, cfg, prompt, 10)
    for st in seq.trace:
        # drafter row and verifier row are the same computation: ratio 1, never rejects
        assert st.result.n_accepted == 1 and st.result.first_reject == -1
        assert abs(st.result.a[0] - 1.0) < 1e-9
        np.testing.assert_allclose(st.verify_logits, st.draft_logits[:1], rtol=1e-9, atol=1e-11)
    assert seq.n_verify_passes == 10


@pytest.mark.parametrize("B", [4, 8])
def test_loop_invariants_and_cache_is_causal(tiny_f32, B):
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=5)[1][:6]
    seq = S.SequenceOracle(W, cfg, block_size=B, seed=1, seq_stream=2, keep_logits=True)
    out = seq.generate(prompt, 24)
    assert len(out) == 24 and all(0 <= t < cfg.vocab for t in out)
    n_rej = 0
    for st in seq.trace:
        assert st.verified and len(st.committed) >= 1          # progress every step
        r = st.result
        assert st.span == list(range(st.j, st.j + len(st.span)))
        if r.first_reject >= 0:
            n_rej += 1
            assert r.first_reject == r.n_accepted
            assert len(st.committed) == r.n_accepted + 1
            assert r.resampled != st.xhat[r.first_reject]      # residual is zero at the rejected proposal
            assert st.u_accept[r.first_reject] >= r.a[r.first_reject]
        else:
            assert r.n_accepted == len(st.span)
        for k in range(r.n_accepted):
            assert st.u_accept[k] < r.a[k]
    assert n_rej >= 1                                           # the run exercises the rejection path
    # the cache holds exactly the K/V a single causal pass over the committed tokens gives
    full = list(prompt) + out
    _, kv = M.forward(W, cfg, full, np.arange(len(full)), M.causal_mask(len(full)), need_logits=[])
    assert seq.n_c <= len(full)
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(seq.cache[l][0], kv[l][0][: seq.n_c], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(seq.cache[l][1], kv[l][1][: seq.n_c], rtol=1e-9, atol=1e-12)


def test_committed_kv_equals_literal_end_of_block_pass(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    prompt = [1, 2, 3, 4, 5]
    B = 4
    seq = S.SequenceOracle(W, cfg, block_size=B, seed=3, seq_stream=0)
    seq.prefill(prompt)
    cache0 = seq.cache
    while len(seq.tokens) < len(prompt) + B:
        seq.step()
    block = seq.tokens[len(prompt):]
    lit = S.literal_block_kv(W, cfg, block, len(prompt), cache0)
    have = seq.n_c - len(prompt)                 # block tokens already cached (a pending tail may remain)
    assert 0 < have <= B
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(seq.cache[l][0][len(prompt):], lit[l][0][:have], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(seq.cache[l][1][len(prompt):], lit[l][1][:have], rtol=1e-9, atol=1e-12)


def test_confidence_branch_is_the_bd3_sampler(tiny_f32):
    """Never verifying reduces SampleBlock to confidence-threshold decoding:
    tau = 1 commits exactly the most confident masked position per step."""
    wl, W = tiny_f32
    cfg = wl.model
    seq = S.SequenceOracle(W, cfg, block_size=4, seed=1, seq_stream=0, route=lambda st: False, tau_conf=1.0)
    seq.generate([7, 8, 9], 8)
    assert seq.n_verify_passes == 0 and seq.n_draft_passes == 8
    for st in seq.trace:
        assert len(st.committed) == 1
        best = max(range(len(st.masked)), key=lambda k: (st.d[k], -k))
        assert st.committed == [st.masked[best]]
    # a low threshold commits every masked position at once
    seq2 = S.SequenceOracle(W, cfg, block_size=4, seed=1, seq_stream=0, route=lambda st: False, tau_conf=0.0)
    seq2.generate([7, 8, 9], 8)
    assert seq2.n_draft_passes == 2


def test_mixed_routing_handles_non_contiguous_commits(tiny_f32):
    """Alternate verification and the confidence branch so that known tokens
    appear to the right of masked ones; the span is then the first masked run only."""
    wl, W = tiny_f32
    cfg = wl.model
    flip = {"n": 0}

    def route(st):
        flip["n"] += 1
        return flip["n"] % 2 == 0
    seq = S.SequenceOracle(W, cfg, block_size=8, seed=2, seq_stream=1, route=route, tau_conf=1.0)
    out = seq.generate([3, 1, 4, 1, 5], 16)
    assert len(out) == 16
    assert any(len(st.span) < len(st.masked) for st in seq.trace if st.verified)
    full = [3, 1, 4, 1, 5] + out
    _, kv = M.forward(W, cfg, full, np.arange(len(full)), M.causal_mask(len(full)), need_logits=[])
    np.testing.assert_allclose(seq.cache[0][0], kv[0][0][: seq.n_c], rtol=1e-9, atol=1e-12)


def test_sequences_are_independent_of_their_stream_only_through_uniforms(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    a = S.SequenceOracle(W, cfg, 4, seed=1, seq_stream=0).generate([1, 2, 3], 8)
    b = S.SequenceOracle(W, cfg, 4, seed=1, seq_stream=0).generate([1, 2, 3], 8)
    assert a == b


def test_reject_only_commits_nothing_but_accepted_drafts(tiny_f32):
    """Reject-only variant (no residual resampling): a step commits exactly its accepted prefix, the rejected
    position stays masked and is drafted again with the same proposal (the context has not changed unless a
    prefix was accepted) but fresh uniforms; the run still ends, and it agrees with the resampling run up to
    the first rejection of either."""
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=5)[1][:6]
    ro = S.SequenceOracle(W, cfg, block_size=8, seed=1, seq_stream=4, keep_logits=True, resample=False)
    out = ro.generate(prompt, 24)
    assert len(out) == 24
    n_rej = n_empty = 0
    for k, st in enumerate(ro.trace):
        r = st.result
        assert r.resampled == -1
        assert st.committed == list(range(st.j, st.j + r.n_accepted))
        assert st.committed_tokens == [int(x) for x in st.xhat[:r.n_accepted]]
        if r.first_reject >= 0:
            n_rej += 1
            nxt = ro.trace[k + 1]
            assert nxt.j == st.j + r.n_accepted                 # the rejected position is the next first masked one
            if r.n_accepted == 0:
                n_empty += 1
                assert nxt.xhat == st.xhat and nxt.u_accept != st.u_accept
    assert n_rej >= 1 and n_empty >= 1
    ref = S.SequenceOracle(W, cfg, block_size=8, seed=1, seq_stream=4, keep_logits=True)
    ref.generate(prompt, 24)
    for a, b in zip(ro.trace, ref.trace):                       # identical until one of them rejects
        assert a.xhat == b.xhat and a.result.n_accepted == b.result.n_accepted
        if a.result.first_reject >= 0:
            break


# ---- the drafting mask of Eq. (draft_mask): the block-row half of a draft pass ---------------------
def _eq_draft_mask(B: int, j: int) -> np.ndarray:
    """M_draft^(j) typed out from its four blocks: [[A_j, 0], [1, 1]] with row sizes j and B - j."""
    m = np.zeros((B, B), dtype=bool)
    for r in range(B):
        for c in range(B):
            m[r, c] = (c <= r) if r < j else True
    return m


def _check_rows_against_eq_draft_mask(rows_fn, B: int = 8):
    for j in range(B):                       # first masked position
        want = _eq_draft_mask(B, j)
        for cached in range(j + 1):          # block positions whose K/V is already in the cache
            pend_pos = list(range(40 + cached, 40 + j))
            blk_pos = list(range(40 + j, 40 + B))
            toks, pos, mask = rows_fn([900 + p for p in pend_pos], pend_pos, [7000 + p for p in blk_pos], blk_pos)
            assert pos.tolist() == list(range(40 + cached, 40 + B))
            assert toks.tolist() == [900 + p for p in pend_pos] + [7000 + p for p in blk_pos]
            # the rows of the pass are rows cached.. of the block; what they see of each other is the lower-right part
            assert mask.shape == (B - cached, B - cached)
            assert (mask == want[cached:, cached:]).all(), (j, cached)
            # and the lower-left part is all ones: every row of the pass sees every cached block token,
            # which is what "each row attends the whole cache" relies on
            assert want[cached:, :cached].all()


def _check_draft_logits_against_one_literal_pass(rows_fn, wl, W):
    """Draft logits of a step that starts from a cache == one pass over prompt ++ block without any
    cache under the composed mask: causal on the prompt, Eq. (draft_mask) on the block, block rows see
    the whole prompt."""
    cfg = wl.model
    MASK = cfg.mask_id
    prompt = [5, 9, 2, 44, 17, 3]
    n, B, j, cached = len(prompt), 8, 3, 1
    block = [11, 4, 30, MASK, MASK, 21, MASK, MASK]       # committed prefix of 3; position 5 known out of order
    pre = prompt + block[:cached]
    _, kv = M.forward(W, cfg, pre, np.arange(len(pre)), M.causal_mask(len(pre)), need_logits=[])
    cache = M.append_kv(None, kv, np.arange(len(pre)))
    pend_pos = list(range(n + cached, n + j))
    toks, pos, mask = rows_fn([block[p - n] for p in pend_pos], pend_pos, block[j:], list(range(n + j, n + B)))
    got, _ = M.forward(W, cfg, toks, pos, mask, cache)
    full = np.zeros((n + B, n + B), dtype=bool)
    full[:n, :n] = M.causal_mask(n)
    full[n:, :n] = True
    full[n:, n:] = _eq_draft_mask(B, j)
    lit, _ = M.forward(W, cfg, prompt + block, np.arange(n + B), full)
    np.testing.assert_allclose(got, lit[n + cached:], rtol=1e-9, atol=1e-11)
    # the block rows really use what the mask gives them: a MASK row's logits move when a later block token changes
    block2 = list(block)
    block2[5] = 22
    lit2, _ = M.forward(W, cfg, prompt + block2, np.arange(n + B), full)
    assert np.abs(lit2[n + 3] - lit[n + 3]).max() > 1e-6


def test_draft_pass_rows_are_eq_draft_mask():
    _check_rows_against_eq_draft_mask(S.draft_pass_rows)


def test_draft_logits_equal_one_literal_pass_under_eq_draft_mask(tiny_f32):
    wl, W = tiny_f32
    _check_draft_logits_against_one_literal_pass(S.draft_pass_rows, wl, W)


@pytest.mark.parametrize("mutation", ["causal_block_rows", "block_rows_blind_to_pending", "pending_sees_block"])
def test_draft_mask_pins_catch_a_wrong_mask(tiny_f32, mutation):
    """The two pins above fail for plausible mistakes in the block-row half of the mask."""
    wl, W = tiny_f32

    def mutated(pending_tokens, pending_pos, block_tokens, block_pos):
        toks, pos, mask = S.draft_pass_rows(pending_tokens, pending_pos, block_tokens, block_pos)
        P = len(pending_tokens)
        mask = mask.copy()
        if mutation == "causal_block_rows":
            mask[P:, :] = np.tril(np.ones_like(mask))[P:, :]
        elif mutation == "block_rows_blind_to_pending":
            mask[P:, :P] = False
        else:
            mask[:P, P:] = True
        return toks, pos, mask

    with pytest.raises(AssertionError):
        _check_rows_against_eq_draft_mask(mutated)
    with pytest.raises(AssertionError):
        _check_draft_logits_against_one_literal_pass(mutated, wl, W)


# ---- right-shifted verifier layout (Section "Self-Verification Mode", last sentence) -------------
def test_shifted_verifier_rows_equal_literal_autoregressive_passes(tiny_f32):
    """In a right-shifted model the logits at position i - 1 score token i, so verifier row k (the last
    committed token, then the drafted tokens) must equal the last row of a plain causal pass over
    prefix ++ xhat_1..xhat_k: the literal next-token distribution, with no MASK anywhere."""
    wl, W = tiny_f32
    cfg = wl.model
    prompt = [5, 9, 2, 44, 17, 3, 8]
    n = len(prompt)
    _, kv = M.forward(W, cfg, prompt[:-1], np.arange(n - 1), M.causal_mask(n - 1), need_logits=[])
    cache = M.append_kv(None, kv, np.arange(n - 1))                 # everything before the last committed token
    xhat = [11, 4, 30, 7]
    L = len(xhat)
    vt, vp, vm = S.verify_pass_rows_shifted(prompt[-1], xhat, n)
    assert vt.tolist() == [prompt[-1]] + xhat[:-1] and vp.tolist() == list(range(n - 1, n - 1 + L))
    assert vm.tolist() == np.tril(np.ones((L, L), bool)).tolist() and len(vt) == L      # L rows, not 2L
    got, _ = M.forward(W, cfg, vt, vp, vm, cache)
    for k in range(L):
        seq = prompt + xhat[:k]
        lit, _ = M.forward(W, cfg, seq, np.arange(len(seq)), M.causal_mask(len(seq)))
        np.testing.assert_allclose(got[k], lit[-1], rtol=1e-9, atol=1e-11)


def test_shifted_block_size_one_is_plain_next_token_greedy_decoding(tiny_f32):
    """B = 1 in the shifted layout: the drafter's row and the verifier's row are the same causal row of
    the last committed token, so nothing is ever rejected and the tokens are those of the textbook
    greedy loop (full causal pass over everything so far, argmax of the last row)."""
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=4)[0][:9]
    seq = S.SequenceOracle(W, cfg, block_size=1, seed=1, seq_stream=0, keep_logits=True, layout="shifted")
    out = seq.generate(prompt, 8)
    toks = [int(t) for t in prompt]
    want = []
    for _ in range(8):
        lit, _ = M.forward(W, cfg, toks, np.arange(len(toks)), M.causal_mask(len(toks)))
        want.append(int(np.argmax(lit[-1])))
        toks.append(want[-1])
    assert out == want
    for st in seq.trace:
        assert st.result.n_accepted == 1 and st.result.first_reject == -1 and abs(st.result.a[0] - 1.0) < 1e-9
        np.testing.assert_allclose(st.verify_logits, st.draft_logits[:1], rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("B", [4, 8])
def test_shifted_loop_invariants_and_cache_is_causal(tiny_f32, B):
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=5)[1][:6]
    seq = S.SequenceOracle(W, cfg, block_size=B, seed=1, seq_stream=2, keep_logits=True, layout="shifted")
    out = seq.generate(prompt, 24)
    assert len(out) == 24 and all(0 <= t < cfg.vocab for t in out)
    n_rej = 0
    for st in seq.trace:
        assert st.verified and len(st.committed) >= 1
        r = st.result
        assert st.verify_logits.shape[0] == len(st.span)            # L verifier rows
        # the first drafted position is scored by the same causal row in both passes: ratio 1, always accepted
        assert abs(r.a[0] - 1.0) < 1e-9 and r.n_accepted >= 1
        np.testing.assert_allclose(st.verify_logits[0], st.draft_logits[0], rtol=1e-9, atol=1e-11)
        if r.first_reject >= 0:
            n_rej += 1
            assert r.resampled != st.xhat[r.first_reject]
    assert n_rej >= 1
    full = list(prompt) + out
    _, kv = M.forward(W, cfg, full, np.arange(len(full)), M.causal_mask(len(full)), need_logits=[])
    assert seq.n_c < len(full)                                       # the last committed token has no K/V of its own yet, or is re-run
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(seq.cache[l][0], kv[l][0][: seq.n_c], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(seq.cache[l][1], kv[l][1][: seq.n_c], rtol=1e-9, atol=1e-12)


# ---- block-end caching (Algorithm "Block-wise autoregressive decoding", K^b, V^b <- x_theta(x^b)) -------------
def test_block_caching_with_block_size_one_is_the_ar_cached_run(tiny_f32):
    """A block of one token: full attention inside the block is the causal mask, so block-end caching and the AR-like
    caching are the same computation, token for token and logit for logit."""
    wl, W = tiny_f32
    cfg = wl.model
    prompt = generate_prompts(wl, seed=4)[0][:9]
    a = S.SequenceOracle(W, cfg, block_size=1, seed=1, seq_stream=0, keep_logits=True, caching="block")
    b = S.SequenceOracle(W, cfg, block_size=1, seed=1, seq_stream=0, keep_logits=True)
    assert a.generate(prompt, 8) == b.generate(prompt, 8)
    for x, y in zip(a.trace, b.trace):
        np.testing.assert_allclose(x.draft_logits, y.draft_logits, rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(x.verify_logits, y.verify_logits, rtol=1e-9, atol=1e-11)
    assert a.n_cache_passes == 8


def test_block_caching_cache_is_the_block_causal_pass_and_verifier_rows_are_literal(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    MASK = cfg.mask_id
    B = 4
    prompt = [5, 9, 2, 44, 17, 3]
    n = len(prompt)
    seq = S.SequenceOracle(W, cfg, block_size=B, seed=1, seq_stream=2, keep_logits=True, caching="block")
    out = seq.generate(prompt, 32)
    assert seq.n_cache_passes == 8 and seq.n_c == n + 32
    assert any(st.result.first_reject >= 0 for st in seq.trace)
    # the cache is what ONE pass over everything gives under the block-causal pattern: causal prompt, then each block
    # sees the prompt, the earlier blocks and all of itself
    full = list(prompt) + out
    T = len(full)
    m = np.zeros((T, T), dtype=bool)
    m[:n, :n] = M.causal_mask(n)
    for b0 in range(n, T, B):
        m[b0:b0 + B, :b0 + B] = True
    _, kv = M.forward(W, cfg, full, np.arange(T), m, need_logits=[])
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(seq.cache[l][0], kv[l][0], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(seq.cache[l][1], kv[l][1], rtol=1e-9, atol=1e-12)
    # verifier rows with an uncached in-block prefix: MASK copy i == a literal pass of cache ++ prefix ++ xhat_<i ++ MASK,
    # causal over the block part (the block-size-1 view), on top of the block-causal cache of the first block
    cache1 = [(k[:n + B], v[:n + B]) for k, v in seq.cache]
    prefix, xhat = [7, 3], [11, 30]
    vt, vp, vm = S.verify_pass_rows_with_prefix(prefix, xhat, n + B, MASK)
    assert len(vt) == 2 + 2 + 2 and vp.tolist() == [n + B, n + B + 1, n + B + 2, n + B + 3, n + B + 2, n + B + 3]
    got, _ = M.forward(W, cfg, vt, vp, vm, cache1, need_logits=[4, 5])
    for i in range(2):
        toks = prefix + xhat[:i] + [MASK]
        lit, _ = M.forward(W, cfg, toks, np.arange(n + B, n + B + len(toks)), M.causal_mask(len(toks)), cache1)
        np.testing.assert_allclose(got[i], lit[-1], rtol=1e-9, atol=1e-11)
