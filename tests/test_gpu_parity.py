"""GPU parity tests: the CUDA path through the C ABI against the oracle."""
import numpy as np
import pytest

from oracle import accept as A
from oracle import philox
from oracle import s2d2 as S
from s2d2_inputs import generate_prompts, generate_weights, get_config

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")


def _engine(wl, W, **kw):
    from paper_2603_25702_b200 import Engine
    from tests.parity_util import register_prompt_lens
    args = dict(block_size=wl.block_size, max_batch=max(wl.batch, 1), max_seq_len=wl.prompt_len[1] + wl.gen_tokens + wl.block_size,
                kv_page_tokens=wl.kv_page_tokens, seed=wl.philox_seed, tau_conf=wl.tau_conf,
                stream=torch.cuda.current_stream().cuda_stream)
    args.update(kw)
    e = Engine(wl.model, **args)
    e.load_weights(W)
    return e


def _start(wl, W, prompts=None, **kw):
    from tests.parity_util import register_prompt_lens
    e = _engine(wl, W, **kw)
    prompts = generate_prompts(wl) if prompts is None else prompts
    ids = e.prefill(prompts)
    register_prompt_lens(ids, prompts)
    for k, sid in enumerate(ids):
        e.seq_set_rng_stream(sid, k)
    return e, ids, prompts


def test_c1_free_running_matches_oracle_tokens():
    """Tiny fp32 config, run end to end without teacher forcing: same committed token ids."""
    wl = get_config("c1")
    W = generate_weights(wl.model, seed=wl.weight_seed)
    e, ids, prompts = _start(wl, W)
    e.generate(ids, wl.gen_tokens)
    got = e.get_tokens(ids[0])[len(prompts[0]):].tolist()
    orc = S.SequenceOracle(W, wl.model, wl.block_size, seed=wl.philox_seed, seq_stream=0)
    want = orc.generate(prompts[0], wl.gen_tokens)
    assert got == want
    c = e.get_counters()
    assert c.n_draft_passes == orc.n_draft_passes and c.n_verify_passes == orc.n_verify_passes
    assert c.n_committed_tokens == wl.gen_tokens
    e.close()


@pytest.mark.parametrize("name,atol,rtol", [("c1", 0.0, 1e-4), ("t_f32", 0.0, 1e-4), ("t_bf16", 2e-2, 0.0),
                                            ("t_bf16_128", 2e-2, 0.0)])
def test_stepwise_parity_dense(name, atol, rtol):
    from tests.parity_util import check_kv, run_steps
    wl = get_config(name)
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.0 if name == "c1" else 0.1)
    e, ids, prompts = _start(wl, W)
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_atol=atol, logit_rtol=rtol)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.verified_steps > 0 and rep.n_committed == wl.gen_tokens * len(ids)
    for sid in ids:
        check_kv(e, W, wl.model, sid, atol=1e-5 if wl.model.dtype == "fp32" else 4e-2)
    print(name, rep)
    e.close()


def test_confidence_branch_and_mixed_routing():
    """Never / alternately verifying exercises the else-branch, non-contiguous commits and multi-token pending rows."""
    from tests.parity_util import check_kv, run_steps
    wl = get_config("t_f32", block_size=8, gen_tokens=16, model_logit_scale=12.0)
    W = generate_weights(wl.model, seed=2, gain_jitter=0.1)
    for mode in ("never", "alternate", "mean_conf"):
        e, ids, prompts = _start(wl, W, tau_conf=0.5)
        n = {"k": 0}

        def route(st):
            n["k"] += 1
            if mode == "never":
                return False
            if mode == "alternate":
                return n["k"] % 2 == 0
            return st.mean_conf < 0.5
        rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_rtol=1e-4, logit_atol=0.0,
                        tau_conf=0.5, route=route)
        assert not rep.mismatches, (mode, rep.mismatches[:5])
        assert rep.steps > rep.verified_steps or mode == "mean_conf"
        for sid in ids:
            check_kv(e, W, wl.model, sid, atol=1e-5)
        e.close()


def test_batch_composition_does_not_change_results():
    wl = get_config("t_bf16")
    W = generate_weights(wl.model, seed=1)
    prompts = generate_prompts(wl)
    e, ids, _ = _start(wl, W, prompts)
    e.generate(ids, wl.gen_tokens)
    together = [e.get_tokens(s).tolist() for s in ids]
    e.close()
    for k, p in enumerate(prompts):
        e1 = _engine(wl, W)
        sid = e1.prefill([p])[0]
        e1.seq_set_rng_stream(sid, k)
        e1.generate([sid], wl.gen_tokens)
        assert e1.get_tokens(sid).tolist() == together[k]
        e1.close()


@pytest.mark.parametrize("name", ["t_moe", "t_moe128"])
def test_moe_stepwise_parity(name):
    """t_moe (16 experts) runs the per-operation kernels, t_moe128 (128 experts, top-8) the persistent pass."""
    from tests.parity_util import moe_prefill_shadows, run_steps
    # the shadows mirror the engine's expert choice of one prefill pass: both prompts must fit 64 rows together
    wl = get_config(name, prompt_len=(9, 30))
    W = generate_weights(wl.model, seed=4, gain_jitter=0.1)
    e, ids, prompts = _start(wl, W)
    shadows = moe_prefill_shadows(e, W, wl.model, ids, prompts)
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_atol=2e-2, shadows=shadows)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.stage_b_passes > 0 and rep.n_committed == wl.gen_tokens * len(ids)
    print("moe", rep)
    e.close()


@pytest.mark.parametrize("V,L,n_seqs", [(8, 1, 3), (8, 3, 5), (4096, 4, 4), (151936, 8, 2), (157184, 32, 1), (1000, 32, 3)])
def test_accept_kernel_on_synthetic_logits(V, L, n_seqs):
    """The fused acceptance kernel alone, on logits shaped like a drafter/verifier pair
    that mostly agree (so that both acceptance and rejection occur)."""
    from paper_2603_25702_b200 import Engine
    wl = get_config("t_f32", model_vocab=V)
    e = Engine(wl.model, block_size=min(L, 32), max_batch=n_seqs, max_seq_len=64, kv_page_tokens=8, seed=9,
               stream=torch.cuda.current_stream().cuda_stream)
    rng = np.random.default_rng(V + L)
    n_rej = n_all = 0
    for trial in range(4):
        d = (rng.standard_normal((n_seqs * L, V)) * 2.0).astype(np.float32)
        v = (d + rng.standard_normal((n_seqs * L, V)).astype(np.float32) * (0.05 + 0.4 * trial)).astype(np.float32)
        if trial == 3:
            v = d.copy()                       # identical distributions: accept everything
        span = rng.integers(1, L + 1, size=n_seqs)
        xhat = d.argmax(axis=1).astype(np.int32)
        pos0 = rng.integers(0, 1000, size=n_seqs)
        streams = rng.integers(0, 100, size=n_seqs)
        steps = rng.integers(0, 50, size=n_seqs)
        td, tv = torch.from_numpy(d).cuda(), torch.from_numpy(v).cuda()
        res = e.accept_logits(td.data_ptr(), tv.data_ptr(), n_seqs, L, span, xhat, pos0, streams, steps)
        for s in range(n_seqs):
            Ls = int(span[s])
            u = [philox.uniform(9, int(pos0[s]) + i, int(streams[s]), int(steps[s]), philox.STREAM_ACCEPT) for i in range(Ls)]
            u2 = [philox.uniform(9, int(pos0[s]) + i, int(streams[s]), int(steps[s]), philox.STREAM_RESAMPLE) for i in range(Ls)]
            o = A.accept_scan(d[s * L:s * L + Ls], v[s * L:s * L + Ls], xhat[s * L:s * L + Ls], u, u2)
            r = res[s]
            if min(o.margin_u) >= 1e-4:
                assert (o.n_accepted, o.first_reject, o.resampled) == (r.n_accepted, r.first_reject, r.resampled_id), (trial, s)
            if trial == 3:
                assert r.n_accepted == Ls and r.first_reject == -1
            n_rej += int(r.first_reject >= 0)
            n_all += int(r.first_reject < 0)
    assert n_all > 0 and (n_rej > 0 or V == 8)
    e.close()


def test_error_paths_return_codes_not_faults():
    from paper_2603_25702_b200 import Engine, S2D2Error
    wl = get_config("t_f32")
    W = generate_weights(wl.model, seed=0)
    e = Engine(wl.model, block_size=4, max_batch=1, max_seq_len=32, kv_page_tokens=8, n_kv_pages=2,
               stream=torch.cuda.current_stream().cuda_stream)
    with pytest.raises(S2D2Error) as ei:                 # weights missing
        e.prefill([[1, 2, 3]])
    assert ei.value.code == -7
    e.load_weights(W)
    with pytest.raises(S2D2Error):                       # token out of range
        e.prefill([[1, wl.model.vocab]])
    with pytest.raises(S2D2Error) as ei:                 # page pool exhausted (2 pages of 8 tokens)
        e.prefill([list(range(20))])
    assert ei.value.code == -3
    assert e.get_counters().kv_pages_in_use == 0        # the failed call left neither pages nor its sequence slot behind
    sid = e.prefill([[1, 2, 3]])[0]                      # (max_batch is 1: a leaked slot would refuse this)
    assert e.get_counters().kv_pages_in_use == 1 and len(e.get_tokens(sid)) == 3
    e.close()
    e = _engine(wl, W)
    sid = e.prefill([[1, 2, 3]])[0]
    with pytest.raises(S2D2Error) as ei:                 # call order
        e.verify_block([sid], [1])
    assert ei.value.code == -4
    with pytest.raises(S2D2Error):                       # no free slot
        for _ in range(10):
            e.prefill([[1, 2, 3]])
    e.draft_block([sid])
    with pytest.raises(S2D2Error):
        e.draft_block([sid])
    e.close()
    # one step uses one id list: a later draft pass overwrites the rows an earlier one produced
    e = _engine(wl, W, max_batch=2)
    a, b = e.prefill([[1, 2, 3], [4, 5, 6, 7]])
    e.draft_block([a])
    e.draft_block([b])
    for call in (lambda: e.verify_block([a], [1]), lambda: e.accept_and_commit([a], [0])):
        with pytest.raises(S2D2Error) as ei:
            call()
        assert ei.value.code == -4 and "draft it again" in str(ei.value)
    e.verify_block([b], [1])
    with pytest.raises(S2D2Error) as ei:                 # a second verifier pass would overwrite the first one's logits
        e.verify_block([b], [1])
    assert ei.value.code == -4
    e.accept_and_commit([b], [1])
    st = e.draft_block([a, b])                           # a is drafted again, together with b's next step
    fl = e.route(st)
    e.verify_block([a, b], fl)
    res = e.accept_and_commit([a, b], fl)
    assert all(r.n_committed >= 1 for r in res)
    e.close()


def test_bounded_wait_times_out_with_a_status_not_a_hang():
    """A wait that nothing satisfies ends after its poll limit with S2D2_ERR_TIMEOUT; the context then
    decodes as usual (the status word is cleared, nothing is left in flight)."""
    from paper_2603_25702_b200 import S2D2Error
    wl = get_config("t_bf16")
    W = generate_weights(wl.model, seed=1)
    e, ids, _ = _start(wl, W)
    e.debug_wait_timeout(0)                       # satisfied at once
    with pytest.raises(S2D2Error) as ei:
        e.debug_wait_timeout(1, limit_polls=2000)
    assert ei.value.code == -5 and "status word 10" in str(ei.value)
    e.generate(ids, wl.block_size)                # still usable
    assert all(len(e.get_tokens(s)) > 0 for s in ids)
    e.close()


def test_accept_override_replaces_only_the_accept_probability():
    """The speed-study switch: with u < 1 every drafted token of the span is accepted, with a
    probability below the smallest uniform none is and position 0 is resampled from the residual,
    and switching it off restores the rule (same results as an engine that never had it on)."""
    from paper_2603_25702_b200 import S2D2Error
    wl = get_config("t_bf16")
    W = generate_weights(wl.model, seed=1)

    def one_step(e, ids):
        st = e.draft_block(ids)
        fl = [1] * len(ids)
        e.verify_block(ids, fl)
        return st, e.accept_and_commit(ids, fl)

    e, ids, _ = _start(wl, W)
    with pytest.raises(S2D2Error):
        e.set_accept_override(1.5)
    e.set_accept_override(1.0)
    st, res = one_step(e, ids)
    for s, r in zip(st, res):
        assert r.n_accepted == s.span_len and r.first_reject == -1 and r.resampled_id == -1
        assert all(a == 1.0 for a in r.a[:s.span_len])
    e.set_accept_override(1e-9)                    # uniforms are at least 2^-25
    st, res = one_step(e, ids)
    for s, r in zip(st, res):
        assert r.n_accepted == 0 and r.first_reject == 0 and r.resampled_id >= 0 and r.resampled_id != s.xhat[0]
    e.close()

    a, ids_a, _ = _start(wl, W)
    b, ids_b, _ = _start(wl, W)
    b.set_accept_override(0.5)
    b.set_accept_override(0.0)
    for _ in range(3):
        ra, rb = one_step(a, ids_a)[1], one_step(b, ids_b)[1]
        assert [(r.n_accepted, r.first_reject, r.resampled_id) for r in ra] == [(r.n_accepted, r.first_reject, r.resampled_id) for r in rb]
    a.close()
    b.close()


@pytest.mark.parametrize("tc", [1, 2])
def test_attention_items_that_span_several_pages(tc):
    """Eight sequences with 1100-1300 cached tokens on the head_dim-128 test model: with 16 (sequence, kv head)
    pairs and about 20 pages each the key splits hold two 64-token pages, so every cache item of the tcgen05
    attention runs its tile loop more than once (next K requested when the scores are complete, next V when the
    previous P V is, lazily rescaled accumulator), and the items are dealt out by cost.  tc = 1: the persistent
    kernel's 80 KB layout; tc = 2: the two-stage layout of the per-operation kernel."""
    from tests.parity_util import run_steps
    wl = get_config("t_bf16_128", batch=8, prompt_len=(1100, 1300), gen_tokens=16, block_size=4)      # 8 x 2 x 4 = 64 verifier rows
    assert wl.kv_page_tokens == 64 and wl.model.head_dim == 128
    W = generate_weights(wl.model, seed=2, gain_jitter=0.1)
    e, ids, prompts = _start(wl, W, use_tensor_cores=tc)
    e.reset_counters()
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=2, logit_atol=2e-2,
                    stage_b_seqs={ids[0], ids[3], ids[7]})
    print("pages", tc, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.verified_steps == 2 * len(ids) and rep.stage_b_passes >= 6
    launches = e.get_counters().n_kernel_launches
    assert (launches < 40) if tc == 1 else (launches > 40)       # persistent passes, or one kernel per operation
    e.close()


@pytest.mark.parametrize("kw", [dict(ratio_gamma=0.5), dict(ratio_gamma=2.0), dict(resample=False)])
def test_accept_variants_match_oracle(kw):
    """Ratio tempering (accept iff u < min(1, (v/d)^gamma), Appendix "ratio tempering") and the reject-only
    variant of the paper's failure-case study (no residual resampling: the rejected position stays masked and
    is drafted again) against the oracle's acceptance arithmetic and forward, on the workload whose peaked
    logits (scale 4) make rejections frequent."""
    from tests.parity_util import run_steps
    wl = get_config("c1")
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.0)
    e, ids, prompts = _start(wl, W, **kw)
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=80, logit_atol=0.0, logit_rtol=1e-4,
                    gamma=kw.get("ratio_gamma", 1.0), resample=kw.get("resample", True))
    print(kw, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.verified_steps > 0 and rep.n_committed > 0
    assert rep.n_resampled > 0                                  # steps that ended in a rejection
    if not kw.get("resample", True):
        assert e.get_counters().n_resampled == 0
        assert rep.n_committed == rep.n_accepted            # only accepted drafts are ever committed
    e.close()


@pytest.mark.parametrize("name,atol,rtol", [("c1", 0.0, 1e-4), ("t_f32", 0.0, 1e-4), ("t_bf16", 2e-2, 0.0), ("t_bf16_128", 2e-2, 0.0)])
def test_right_shifted_verifier_layout_matches_oracle(name, atol, rtol):
    """S2D2_VERIFIER_RIGHT_SHIFTED (Section "Self-Verification Mode": for right-shifted models the plain causal
    mask gives the verifier view): L causal verifier rows instead of 2L, logits read one row to the left in both
    passes, every pass starting at the last committed token.  Both parity stages over the whole generation,
    the cache against the oracle's causal pass, and for the fp32 workload the free-running token stream."""
    from tests.parity_util import check_kv, run_steps
    wl = get_config(name)
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.0 if name == "c1" else 0.1)
    e, ids, prompts = _start(wl, W, verifier_layout="shifted")
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_atol=atol, logit_rtol=rtol,
                    layout="shifted")
    print(name, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.verified_steps > 0 and rep.n_committed == wl.gen_tokens * len(ids)
    for sid in ids:
        check_kv(e, W, wl.model, sid, atol=1e-5 if wl.model.dtype == "fp32" else 4e-2)
    e.close()
    if name == "c1":
        e, ids, prompts = _start(wl, W, verifier_layout="shifted")
        e.generate(ids, wl.gen_tokens)
        got = e.get_tokens(ids[0])[len(prompts[0]):].tolist()
        orc = S.SequenceOracle(W, wl.model, wl.block_size, seed=wl.philox_seed, seq_stream=0, layout="shifted")
        assert got == orc.generate(prompts[0], wl.gen_tokens)
        c = e.get_counters()
        assert c.n_draft_passes == orc.n_draft_passes and c.n_verify_passes == orc.n_verify_passes
        e.close()


@pytest.mark.parametrize("V,n_rows", [(8, 6), (4096, 8), (1000, 32), (151936, 8), (157184, 16)])
def test_sample_from_logits_kernels_on_synthetic_logits(V, n_rows):
    """SampleFromLogits alone (s2d2_sample_logits): greedy proposals and, in sampling mode, inverse-CDF draws
    from pi_d with the draft-sampling Philox stream, against the oracle on the same fp32 logits.  The draw is
    an integer decided by a floating-point comparison; both sides take it in fp64, and a row whose target lies
    within 1e-9 of a cumulative-sum boundary (summation order differs) is exempt and counted."""
    from paper_2603_25702_b200 import Engine
    wl = get_config("t_f32", model_vocab=V)
    e = Engine(wl.model, block_size=min(n_rows, 32), max_batch=max(1, (n_rows + 31) // 32), max_seq_len=64, kv_page_tokens=8, seed=9,
               stream=torch.cuda.current_stream().cuda_stream)
    rng = np.random.default_rng(V + n_rows)
    exempt = 0
    for trial in range(3):
        x = (rng.standard_normal((n_rows, V)) * (0.5 + 1.5 * trial)).astype(np.float32)
        if trial == 2:
            x[:, V // 3] += 6.0                 # a peaked row: most draws land on one token
        pos = rng.integers(0, 5000, size=n_rows)
        streams = rng.integers(0, 100, size=n_rows)
        steps = rng.integers(0, 50, size=n_rows)
        tx = torch.from_numpy(x).cuda()
        gx, gc, gm, ge = e.sample_logits(tx.data_ptr(), n_rows, "greedy")
        sx, sc, sm_, se = e.sample_logits(tx.data_ptr(), n_rows, "sample", pos, streams, steps)
        for r in range(n_rows):
            og = A.sample_from_logits(x[r])
            assert og.xhat == gx[r] and abs(og.d - gc[r]) <= 1e-5 * og.d + 1e-9
            assert abs(og.margin - gm[r]) <= 1e-5 and abs(og.entropy - ge[r]) <= 1e-4 * max(1.0, og.entropy)
            u = philox.uniform(9, int(pos[r]), int(streams[r]), int(steps[r]), philox.STREAM_DRAFT)
            os_ = A.sample_from_logits(x[r], "sample", u)
            p = A.softmax(x[r])
            c = np.cumsum(p)
            near = np.abs(c - u * c[-1]).min() < 1e-9
            exempt += int(near)
            if not near:
                assert os_.xhat == sx[r], (trial, r)
                assert abs(os_.d - sc[r]) <= 1e-5 * os_.d + 1e-9
            assert abs(os_.margin - sm_[r]) <= 1e-5 and abs(os_.entropy - se[r]) <= 1e-4 * max(1.0, os_.entropy)
    assert exempt <= 1
    e.close()


def test_sampling_draft_mode_matches_oracle_end_to_end():
    """S2D2_DRAFT_SAMPLE through the decode loop on the fp32 workload: stage A with sampled proposals on the engine's
    logits, stage B, and the free-running token stream against the oracle in its sampling mode (the one
    configuration in which the speculative output law equals the verifier's)."""
    from tests.parity_util import run_steps
    wl = get_config("c1")
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.0)
    e, ids, prompts = _start(wl, W, draft_mode="sample")
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=80, logit_atol=0.0, logit_rtol=1e-4,
                    draft_mode="sample")
    print("sample", rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.n_committed == wl.gen_tokens
    e.close()
    e, ids, prompts = _start(wl, W, draft_mode="sample")
    e.generate(ids, wl.gen_tokens)
    got = e.get_tokens(ids[0])[len(prompts[0]):].tolist()
    orc = S.SequenceOracle(W, wl.model, wl.block_size, seed=wl.philox_seed, seq_stream=0, draft_mode="sample")
    want = orc.generate(prompts[0], wl.gen_tokens)
    greedy = S.SequenceOracle(W, wl.model, wl.block_size, seed=wl.philox_seed, seq_stream=0).generate(prompts[0], wl.gen_tokens)
    assert got == want and want != greedy          # and the sampled trajectory is a different one
    e.close()


@pytest.mark.parametrize("name,atol,rtol", [("c1", 0.0, 1e-4), ("t_f32", 0.0, 1e-4), ("t_bf16", 2e-2, 0.0), ("t_bf16_128", 2e-2, 0.0)])
def test_block_end_caching_matches_oracle(name, atol, rtol):
    """S2D2_CACHE_BLOCK_END (Algorithm "Block-wise autoregressive decoding", K^b, V^b <- x_theta(x^b)): whole-block draft
    rows that see each other, verifier rows that carry the block's committed prefix, nothing cached until the block is
    finished, then one pass over it with full attention inside the block.  Both parity stages over the whole generation,
    the cache against the oracle's block-causal passes, and for the fp32 workload the free-running token stream."""
    from tests.parity_util import check_kv, run_steps
    wl = get_config(name)
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.0 if name == "c1" else 0.1)
    e, ids, prompts = _start(wl, W, caching="block")
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_atol=atol, logit_rtol=rtol, caching="block")
    print(name, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.verified_steps > 0 and rep.n_committed == wl.gen_tokens * len(ids)
    assert e.get_counters().n_cache_passes >= wl.gen_tokens // wl.block_size
    for sid in ids:
        assert e.debug_seq_state(sid)["n_cached"] == e.debug_seq_state(sid)["block_start"]
        check_kv(e, W, wl.model, sid, atol=1e-5 if wl.model.dtype == "fp32" else 4e-2, block_size=wl.block_size)
    e.close()
    if name == "c1":
        e, ids, prompts = _start(wl, W, caching="block")
        e.generate(ids, wl.gen_tokens)
        got = e.get_tokens(ids[0])[len(prompts[0]):].tolist()
        orc = S.SequenceOracle(W, wl.model, wl.block_size, seed=wl.philox_seed, seq_stream=0, caching="block")
        assert got == orc.generate(prompts[0], wl.gen_tokens)
        c = e.get_counters()
        assert c.n_draft_passes == orc.n_draft_passes and c.n_verify_passes == orc.n_verify_passes and c.n_cache_passes == orc.n_cache_passes
        e.close()


@pytest.mark.parametrize("name,lens,passes", [
    ("t_bf16_128", [300, 40, 129, 24], 2),      # two long prompts share one wide pass (5 + 3 chunks); the short ones take one persistent pass
    ("t_bf16_128", [1500], 2),                  # 1024 rows (16 chunks of one prompt in one pass), then 476
    ("t_bf16", [65, 5, 9, 70, 3, 11, 2], 1),    # more than four short prompts ride the wide pass; 16-token pages
    ("t_f32", [150, 7], 1),                     # fp32 model: plain kernels, every prompt in wide passes
])
def test_prefill_in_wide_passes_matches_oracle(name, lens, passes):
    """Prefill (first line of the block-wise decoding algorithm: the prompt's K/V under the causal mask).  A prompt
    enters a pass as 64-row chunks, several chunks of one prompt in the same pass: chunk k reads chunks 0..k-1 of
    that pass from the cache pages they were written to a kernel earlier.  The cache of every sequence must equal
    the oracle's causal pass over its prompt."""
    from tests.parity_util import check_kv
    wl = get_config(name, batch=len(lens), prompt_len=(min(lens), max(lens)))
    W = generate_weights(wl.model, seed=3)
    rng = np.random.default_rng(11)
    prompts = [rng.integers(0, wl.model.vocab, size=n).tolist() for n in lens]
    e, ids, _ = _start(wl, W, prompts)
    cnt = e.get_counters()
    assert cnt.n_prefill_passes == passes and cnt.n_rows_prefill == sum(lens)
    for sid, n in zip(ids, lens):
        assert e.debug_seq_state(sid)["n_cached"] == n
        worst = check_kv(e, W, wl.model, sid, atol=1e-5 if wl.model.dtype == "fp32" else 4e-2)
        print(name, n, "KV off by", worst)
    e.close()
