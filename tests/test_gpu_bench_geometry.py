"""Parity in the regime bench.py times, at a size the CPU side can afford.

The full-size parity tests run a handful of tokens of context (an fp64 prefill of a thousand tokens through
36 layers of width 4096 takes hours).  What the bench adds to that is geometry, not width: contexts of 1000 to
2000 tokens, i.e. about 18 to 33 pages of 64 tokens per (sequence, kv head), grouped-query attention with
32 query / 8 kv heads (16 / 4 for the mixture-of-experts workload), query tiles of 16 rows x 4 heads, key
splits sized to the SM count and their combine.  These tests keep exactly that geometry on a two-layer body of
width 1024 and run both parity stages through the persistent pass kernel, plus the mixture-of-experts layers at
the workload's block size of 32 (64-row verifier passes, spans of 32)."""
import pytest

from s2d2_inputs import generate_prompts, generate_weights, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _run(wl, n_steps, **engine_kw):
    from paper_2603_25702_b200 import Engine
    from tests.parity_util import register_prompt_lens, run_steps
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.1)
    e = Engine(wl.model, block_size=wl.block_size, max_batch=wl.batch, max_seq_len=wl.prompt_len[1] + wl.gen_tokens + wl.block_size,
               kv_page_tokens=wl.kv_page_tokens, seed=wl.philox_seed, stream=torch.cuda.current_stream().cuda_stream, **engine_kw)
    e.load_weights(W)
    prompts = generate_prompts(wl)
    ids = e.prefill(prompts)
    register_prompt_lens(ids, prompts)
    for k, sid in enumerate(ids):
        e.seq_set_rng_stream(sid, k)
    e.reset_counters()
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=n_steps, logit_atol=2e-2)
    launches = e.get_counters().n_kernel_launches
    return e, W, ids, rep, launches


@pytest.mark.parametrize("name,ctx", [("t_geo32", 1100), ("t_geo32", 2050), ("t_geo16", 1100)])
def test_bench_attention_geometry_matches_oracle(name, ctx):
    """Batch 1, block 8 (32 for the 16 / 4 head model), context 1100 and 2050: one sequence, so every attention item is
    one key split of one kv head over the full query tile, as in the default bench run."""
    from tests.parity_util import check_kv
    wl = get_config(name, prompt_len=(ctx, ctx))
    assert wl.kv_page_tokens == 64 and wl.model.head_dim == 128
    e, W, ids, rep, launches = _run(wl, n_steps=3)
    print(name, ctx, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.steps == 3 and rep.stage_b_passes == 6 and rep.verified_steps == 3
    assert launches < 12 * rep.steps                       # persistent passes
    assert rep.exempt_steps == 0
    if ctx == 1100:
        check_kv(e, W, wl.model, ids[0], atol=4e-2)
    e.close()


def test_bench_attention_geometry_with_sub_gemm_cuts():
    """The same, with every GEMM cut into sub-GEMMs (the tile-by-tile hand-overs of the large models)."""
    wl = get_config("t_geo32")
    e, W, ids, rep, launches = _run(wl, n_steps=3, use_tensor_cores=3)
    print("cuts", rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.stage_b_passes == 6 and launches < 12 * rep.steps
    e.close()


@pytest.mark.parametrize("name", ["t_moe128", "t_moe"])
def test_moe_block_32_matches_oracle(name):
    """Mixture-of-experts layers at the workload's block size: 64-row verifier passes (touched-expert lists built
    from 64 rows) and spans of up to 32 through the decode loop.  Expert choice is an integer decided by floating
    point: the oracle takes the engine's ids where they differ, every such difference must be a near tie of the
    oracle's router logits, and there may only be few of them."""
    from paper_2603_25702_b200 import Engine
    from tests.parity_util import ParityReport, moe_prefill_shadows, register_prompt_lens, run_steps
    wl = get_config(name, block_size=32, gen_tokens=64, batch=1, prompt_len=(9, 40))
    W = generate_weights(wl.model, seed=wl.weight_seed, gain_jitter=0.1)
    e = Engine(wl.model, block_size=32, max_batch=1, max_seq_len=160, kv_page_tokens=wl.kv_page_tokens, seed=wl.philox_seed,
               stream=torch.cuda.current_stream().cuda_stream)
    e.load_weights(W)
    prompts = generate_prompts(wl)
    ids = e.prefill(prompts)
    register_prompt_lens(ids, prompts)
    e.seq_set_rng_stream(ids[0], 0)
    shadows = moe_prefill_shadows(e, W, wl.model, ids, prompts)
    rep = run_steps(e, W, wl, ids, {ids[0]: 0}, n_steps=200, logit_atol=2e-2, shadows=shadows)
    print(name, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.n_committed == 64 and rep.steps >= 2
    assert rep.exempt_steps <= max(1, rep.steps // 100)
    assert rep.moe_rows_checked > 0 and rep.moe_forced_rows <= 0.03 * rep.moe_rows_checked, (rep.moe_forced_rows, rep.moe_rows_checked)
    e.close()
