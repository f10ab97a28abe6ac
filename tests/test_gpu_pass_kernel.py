"""The persistent pass kernel against the one-kernel-per-operation path of the same library
(both are separately checked against the oracle by the parity tests), and its phase trace."""
import numpy as np
import pytest

from s2d2_inputs import generate_prompts, generate_weights, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _run(wl, W, prompts, mode, n_steps):
    from paper_2603_25702_b200 import Engine
    e = Engine(wl.model, block_size=wl.block_size, max_batch=wl.batch, max_seq_len=wl.prompt_len[1] + wl.gen_tokens + wl.block_size,
               kv_page_tokens=wl.kv_page_tokens, seed=wl.philox_seed, stream=torch.cuda.current_stream().cuda_stream,
               use_tensor_cores=mode)
    e.load_weights(W)
    ids = e.prefill(prompts)
    for k, sid in enumerate(ids):
        e.seq_set_rng_stream(sid, k)
    out = []
    for _ in range(n_steps):
        st = e.draft_block(ids)
        fl = e.route(st)
        dl = e.debug_copy_logits(0, sum(s.n_masked for s in st))
        e.verify_block(ids, fl)
        vl = e.debug_copy_logits(1, sum(s.span_len for s in st))
        res = e.accept_and_commit(ids, fl)
        out.append((dl, vl, [(r.n_accepted, r.first_reject, r.resampled_id) for r in res]))
    launches = e.get_counters().n_kernel_launches
    e.close()
    return out, launches


@pytest.mark.parametrize("name", ["t_bf16", "t_bf16_128"])
def test_persistent_pass_matches_per_operation_path(name):
    wl = get_config(name)
    W = generate_weights(wl.model, seed=11, gain_jitter=0.1)
    prompts = generate_prompts(wl)
    a, launches_a = _run(wl, W, prompts, 1, 3)
    b, launches_b = _run(wl, W, prompts, 2, 3)
    assert launches_a < launches_b              # one launch per pass instead of one per operation (prefill chunks of more than 64 rows take the per-operation path in both)
    # step 0 starts from identical caches: logits agree to bf16 rounding of the two kernel orders
    for which in (0, 1):
        assert np.abs(a[0][which] - b[0][which]).max() < 2e-2


def test_pass_trace_is_monotone_and_complete():
    from paper_2603_25702_b200 import Engine, S2D2Error
    wl = get_config("t_bf16")
    W = generate_weights(wl.model, seed=11)
    e = Engine(wl.model, block_size=wl.block_size, max_batch=wl.batch, max_seq_len=128, kv_page_tokens=wl.kv_page_tokens,
               stream=torch.cuda.current_stream().cuda_stream)
    e.load_weights(W)
    ids = e.prefill(generate_prompts(wl))
    with pytest.raises(S2D2Error):
        e.debug_pass_trace()                     # nothing traced yet
    e.set_profiling(2)
    e.draft_block(ids)
    marks, sm = e.debug_pass_trace()
    e.set_profiling(0)
    n_ctas, n_marks = marks.shape
    L = wl.model.n_layers
    n_named = 3 + 12 * L + 2                             # embedding barrier, 12 marks per dense layer, the LM-head phase
    assert n_marks >= n_named + 6 * (4 * L + 1) and (n_marks - n_named) % 6 == 0 and n_ctas >= 1     # + two and four per sub-GEMM
    n_sub = (n_marks - n_named) // 6
    mma = marks[:, n_named:n_named + 2 * n_sub].reshape(n_ctas, n_sub, 2)
    assert (mma[:, :, 0] <= mma[:, :, 1]).all() and (mma > 0).any()
    names = Engine.TRACE_DENSE_MARKS
    used = [0, 1] + list(range(3, n_named))                # slot 2 is unused
    flat = marks[:, used]
    assert (flat > 0).all() and (np.diff(flat, axis=1) >= 0).all()    # every CTA passes its marks in slot order
    # nobody leaves a grid barrier before everybody has entered it (with one sequence in the pass the attention items hand over
    # to the combine through counters, not a barrier: this pass has several, so both are barriers)
    bars = [(0, 1)] + [(3 + 12 * l + names.index(n + "_entry"), 3 + 12 * l + names.index(n + "_exit"))
                       for l in range(L) for n in ("rope_barrier", "attn_barrier")]
    for ent, ex in bars:
        assert marks[:, ex].min() >= marks[:, ent].max() - 2000
    assert len(set(sm.tolist())) == n_ctas       # one CTA per SM
    prof = e.get_gemm_profile()
    assert prof["launches"] >= 1 and prof["bytes"] > 0
    e.close()


def test_full_shape_passes_repeat_bit_for_bit():
    """The pass kernel hands data from CTA to CTA through counters and grid barriers (split-K partials, GEMM
    inputs read by TMA, attention partials).  Its sums have a fixed order, so two runs of the same steps must
    agree bit for bit; a hand-over that let a reader run ahead of a writer would show up as a difference.
    1.7B-class shape, 30 decode steps (60 passes of 28 layers), two engines with the same seeds."""
    wl = get_config("c2", prompt_len=(200, 200), gen_tokens=30 * 4)
    W = generate_weights(wl.model, seed=wl.weight_seed)
    prompts = generate_prompts(wl)
    a, launches = _run(wl, W, prompts, 1, 30)
    b, _ = _run(wl, W, prompts, 1, 30)
    assert launches < 40 * 30                      # persistent passes
    for step, (x, y) in enumerate(zip(a, b)):
        assert x[2] == y[2], step
        assert np.array_equal(x[0], y[0]) and np.array_equal(x[1], y[1]), step


@pytest.mark.parametrize("name", ["t_bf16", "t_bf16_128"])
def test_sub_gemm_cuts_match_oracle_on_small_models(name):
    """use_tensor_cores = 3 cuts every GEMM of the persistent kernel into sub-GEMMs wherever the tile counts
    allow, so a small model runs the hand-overs a large one runs by default: output tiles reduced and turned
    into the next GEMM's input while the rest streams, the next GEMM starting on those k-blocks, and no grid
    barrier between the attention block of one layer and the next.  Both parity stages over the whole
    generation, then the cache against the oracle's causal pass."""
    from paper_2603_25702_b200 import Engine
    from tests.parity_util import check_kv, register_prompt_lens, run_steps
    wl = get_config(name)
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.1)
    e = Engine(wl.model, block_size=wl.block_size, max_batch=wl.batch, max_seq_len=wl.prompt_len[1] + wl.gen_tokens + wl.block_size,
               kv_page_tokens=wl.kv_page_tokens, seed=wl.philox_seed, stream=torch.cuda.current_stream().cuda_stream,
               use_tensor_cores=3)
    e.load_weights(W)
    prompts = generate_prompts(wl)
    ids = e.prefill(prompts)
    register_prompt_lens(ids, prompts)
    for k, sid in enumerate(ids):
        e.seq_set_rng_stream(sid, k)
    e.reset_counters()
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=200, logit_atol=2e-2)
    print(name, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.n_committed == wl.gen_tokens * len(ids)
    assert e.get_counters().n_kernel_launches < 12 * rep.steps     # persistent passes
    for sid in ids:
        check_kv(e, W, wl.model, sid, atol=4e-2)
    e.close()
