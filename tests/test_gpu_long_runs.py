"""Long decode runs at the full model shapes and batch sizes of the workloads.

The oracle's forward at these sizes costs minutes per pass, so the forward stage (B) covers the first step only.
The acceptance stage (A) needs no oracle forward: proposals, acceptance scan, residual resampling and commit are
recomputed in fp64 from the engine's own logits at every step and must agree bit for bit (positions with
|u - a| < 1e-4 are counted, and there may only be few).  Over dozens to hundreds of steps this exercises what
the short full-size tests cannot: speculative K/V append and rollback over many blocks, page-boundary
crossings, multi-token pending rows, ragged batches whose sequences finish blocks at different steps, and the
routing rule of the 4B-class workload."""
import pytest

from s2d2_inputs import generate_prompts, generate_weights, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.mark.parametrize("name,batch,gen_tokens,max_steps", [
    ("c2", 1, 512, 600),          # the workload's full generation
    ("c3", 8, 96, 200),           # its batch of 8 with the mean-confidence router
    ("c4", 1, 96, 400),
    ("c4", 32, 16, 4),            # the batch-32 point: passes of 256 to 512 rows, one kernel per operation
    ("c5", 1, 64, 200),           # mixture of experts at block 32
])
def test_long_run_acceptance_stage_is_exact(name, batch, gen_tokens, max_steps):
    from paper_2603_25702_b200 import Engine, RoutePolicy
    from tests.parity_util import moe_prefill_shadows, register_prompt_lens, run_steps
    wl = get_config(name, prompt_len=(5, 9), gen_tokens=gen_tokens, batch=batch)
    W = generate_weights(wl.model, seed=wl.weight_seed)
    e = Engine(wl.model, block_size=wl.block_size, max_batch=batch, max_seq_len=16 + gen_tokens + wl.block_size, kv_page_tokens=wl.kv_page_tokens,
               seed=wl.philox_seed, tau_conf=wl.tau_conf, stream=torch.cuda.current_stream().cuda_stream)
    e.load_weights(W)
    if wl.route == "mean_conf":
        e.set_route_policy(RoutePolicy(RoutePolicy.MEAN_CONF, wl.tau_route, 0, 0, 0, 0, 0))
    prompts = generate_prompts(wl)
    ids = e.prefill(prompts)
    register_prompt_lens(ids, prompts)
    for k, sid in enumerate(ids):
        e.seq_set_rng_stream(sid, k)
    shadows = moe_prefill_shadows(e, W, wl.model, ids, prompts) if wl.model.is_moe else None
    rep = run_steps(e, W, wl, ids, {sid: k for k, sid in enumerate(ids)}, n_steps=max_steps, logit_atol=2e-2, tau_conf=wl.tau_conf,
                    stage_b_steps=1, stage_b_seqs={ids[0]}, shadows=shadows)
    print(name, batch, rep)
    assert not rep.mismatches, rep.mismatches[:5]
    assert rep.stage_b_passes >= 1
    if max_steps >= 100:
        assert rep.n_committed == gen_tokens * batch           # every sequence finished its generation
    assert rep.near_boundary <= max(1, rep.n_committed // 100) and rep.exempt_steps <= max(1, rep.steps * batch // 100)
    for sid in ids:                                            # the cache length follows the committed tokens
        st = e.debug_seq_state(sid)
        assert st["n_cached"] <= st["block_start"] + wl.block_size
    e.close()
