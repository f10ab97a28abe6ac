"""Drives the CUDA engine step by step next to the oracle.

Two-stage parity per step:
  A (acceptance stage): the oracle's SampleFromLogits / acceptance scan /
    residual resample / confidence branch run on the engine's own fp32 logits
    with the oracle's own Philox uniforms; proposals, accepted length, first
    rejection and committed token ids must be bit-exact, except at positions
    with |u - a| < 1e-4 (or a confidence within 1e-6 of the threshold), which
    are counted.
  B (forward stage): the oracle's fp64 forward over the same rows, on a cache
    the oracle computes itself from the committed tokens, must reproduce the
    engine's logits within the tolerance of the configuration.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

from oracle import accept as A
from oracle import model as M
from oracle import philox
from oracle import s2d2 as S


@dataclass
class ParityReport:
    steps: int = 0
    verified_steps: int = 0
    near_boundary: int = 0
    exempt_steps: int = 0
    mismatches: List[str] = field(default_factory=list)
    max_draft_err: float = 0.0
    max_verify_err: float = 0.0
    max_rel_err: float = 0.0
    logit_scale_seen: float = 0.0
    stage_b_passes: int = 0
    n_accepted: int = 0
    n_resampled: int = 0
    n_committed: int = 0
    moe_forced_rows: int = 0          # (row, layer) pairs whose expert set the oracle took from the engine (near ties)
    moe_rows_checked: int = 0         # (row, layer) pairs compared
    moe_max_forced_gap: float = 0.0   # largest distance of a swapped expert's router logit from the oracle's k-th
    err_without_kv_storage: float = 0.0   # probe: engine's draft logits of step 0 against an oracle that keeps K/V in fp64


class OracleShadow:
    """The oracle's own causal cache over the committed tokens of one sequence."""

    def __init__(self, W, cfg, kv_storage: bool = True):
        self.W, self.cfg, self.kv_storage = W, cfg, kv_storage
        self.cache: Optional[M.KV] = None
        self.n = 0

    def extend(self, all_tokens, upto: int):
        if upto <= self.n:
            return
        toks = [int(t) for t in all_tokens[self.n:upto]]
        _, kv = M.forward(self.W, self.cfg, toks, np.arange(self.n, upto), M.causal_mask(len(toks)), self.cache, need_logits=[],
                          kv_storage=self.kv_storage)
        self.cache = M.append_kv(self.cache, kv, np.arange(len(toks)))
        self.n = upto

    def extend_blocks(self, all_tokens, upto: int, prompt_len: int, B: int):
        """Block-end caching: causal over the prompt, then finished block by finished block with full attention
        inside the block (``upto`` is a block boundary)."""
        self.extend(all_tokens, min(upto, prompt_len))
        while self.n < upto:
            toks = [int(t) for t in all_tokens[self.n:self.n + B]]
            _, kv = M.forward(self.W, self.cfg, toks, np.arange(self.n, self.n + B), np.ones((B, B), dtype=bool), self.cache, need_logits=[],
                              kv_storage=self.kv_storage)
            self.cache = M.append_kv(self.cache, kv, np.arange(B))
            self.n += B


def run_steps(engine, W, wl, seq_ids, rng_streams, n_steps: int, stage_b_every: int = 1, seed: Optional[int] = None,
              gamma: float = 1.0, tau_conf: float = 0.9, logit_atol: float = 2e-2, logit_rtol: float = 0.0,
              route=None, shadows=None, stage_b_seqs=None, resample: bool = True, layout: str = "aligned",
              stage_b_steps: Optional[int] = None, draft_mode: str = "greedy", probe_kv_storage: bool = False,
              caching: str = "ar") -> ParityReport:
    """Run up to ``n_steps`` decode steps on all sequences (stops when every one has
    generated wl.gen_tokens) and check both parity stages.  ``stage_b_seqs``: restrict the
    oracle's forward (stage B) to these sequence ids (large batches at full model size); stage A
    always covers every sequence.  ``resample=False``: the reject-only variant (the first rejected position stays
    masked and is drafted again in the next step).  ``layout="shifted"``: the right-shifted verifier layout (L causal
    verifier rows, logits read one row to the left in both passes).  ``stage_b_steps``: run stage B on the first so many
    steps only (long runs at full model size).  ``draft_mode="sample"``: proposals drawn from pi_d with the
    draft-sampling uniforms."""
    shifted = layout == "shifted"
    block_cache = caching == "block"       # block-end caching: whole-block draft rows, verifier rows with the block's prefix
    cfg, B = wl.model, wl.block_size
    MASK = cfg.mask_id
    seed = wl.philox_seed if seed is None else seed
    rep = ParityReport()
    if shadows is None:
        assert not cfg.is_moe, "MoE parity mirrors the engine's passes: build the shadows with moe_prefill_shadows"
        shadows = {sid: OracleShadow(W, cfg) for sid in seq_ids}
    for step_no in range(n_steps):
        live = [sid for sid in seq_ids
                if engine.debug_seq_state(sid)["block_start"] - _prompt_len(engine, sid) < wl.gen_tokens]
        if not live:
            break
        before = {sid: engine.debug_seq_state(sid) for sid in live}
        final_toks = {sid: engine.get_tokens(sid) for sid in live}
        stats = engine.draft_block(live)
        flags = engine.route(stats) if route is None else np.array([int(route(s)) for s in stats], dtype=np.uint8)
        dlog = engine.debug_copy_logits(0, sum(s.n_masked for s in stats))
        eid_d = engine.debug_copy_expert_ids(64 * len(live)) if cfg.is_moe else None
        engine.verify_block(live, flags)
        eid_v = engine.debug_copy_expert_ids(64 * len(live)) if (cfg.is_moe and flags.any()) else None
        vlog = engine.debug_copy_logits(1, sum(s.span_len for s, f in zip(stats, flags) if f)) if flags.any() else None
        res = engine.accept_and_commit(live, flags)
        do_b = stage_b_every > 0 and step_no % stage_b_every == 0 and (stage_b_steps is None or step_no < stage_b_steps)
        drow = vrow = drow_all = vrow_all = 0
        for k, sid in enumerate(live):
            st, rs, bf = stats[k], res[k], before[sid]
            s0, j, nm, L = st.block_start, st.first_masked, st.n_masked, st.span_len
            blk = list(bf["block_tokens"])
            full = list(final_toks[sid]) + blk
            masked = [i for i in range(B) if blk[i] == MASK]
            tag = f"step {step_no} seq {sid}"
            if s0 != bf["block_start"] or masked != list(st.masked_idx[:nm]) or j != masked[0]:
                rep.mismatches.append(f"{tag}: block bookkeeping")
                continue
            my_d = dlog[drow:drow + nm]
            drow += nm
            # ---- stage A on the engine's logits ------------------------------------------------
            if draft_mode == "sample":
                o_stats = [A.sample_from_logits(my_d[r], "sample", philox.uniform(seed, s0 + masked[r], rng_streams[sid], bf["step"], philox.STREAM_DRAFT))
                           for r in range(nm)]
            else:
                o_stats = [A.sample_from_logits(my_d[r]) for r in range(nm)]
            xhat = [q.xhat for q in o_stats]
            exempt = False
            if xhat != list(st.xhat[:nm]):
                rep.mismatches.append(f"{tag}: proposals differ")
            for r in range(nm):
                if abs(o_stats[r].d - st.conf[r]) > 1e-5 * max(o_stats[r].d, 1e-30) + 1e-9:
                    rep.mismatches.append(f"{tag}: confidence {o_stats[r].d} vs {st.conf[r]}")
                if abs(o_stats[r].margin - st.margin[r]) > 1e-5 or abs(o_stats[r].entropy - st.entropy[r]) > 1e-4 * max(1, o_stats[r].entropy):
                    rep.mismatches.append(f"{tag}: margin/entropy")
            span_ok = 1
            while j + span_ok < B and blk[j + span_ok] == MASK:
                span_ok += 1
            if span_ok != L:
                rep.mismatches.append(f"{tag}: span length")
            committed = {}
            if flags[k]:
                my_v = vlog[vrow:vrow + L]
                vrow += L
                stream, stp = rng_streams[sid], bf["step"]
                u = [philox.uniform(seed, s0 + j + i, stream, stp, philox.STREAM_ACCEPT) for i in range(L)]
                u2 = [philox.uniform(seed, s0 + j + i, stream, stp, philox.STREAM_RESAMPLE) for i in range(L)]
                o = A.accept_scan(my_d[:L], my_v, xhat[:L], u, u2, gamma, resample=resample)
                near = sum(1 for m_ in o.margin_u if m_ < 1e-4)
                rep.near_boundary += near
                exempt = near > 0
                same = (o.n_accepted == rs.n_accepted and o.first_reject == rs.first_reject and o.resampled == rs.resampled_id)
                if not same and not exempt:
                    rep.mismatches.append(f"{tag}: accept n_acc {o.n_accepted}/{rs.n_accepted} rej {o.first_reject}/{rs.first_reject} "
                                          f"tok {o.resampled}/{rs.resampled_id}")
                for i in range(len(o.a)):
                    if i < (rs.first_reject + 1 if rs.first_reject >= 0 else rs.n_accepted):
                        if abs(o.a[i] - rs.a[i]) > 1e-5 or abs(u[i] - rs.u[i]) > 1e-7:
                            rep.mismatches.append(f"{tag}: a/u at {i}: {o.a[i]} {rs.a[i]} {u[i]} {rs.u[i]}")
                for i in range(rs.n_accepted):
                    committed[j + i] = int(st.xhat[i])
                if rs.first_reject >= 0 and resample:
                    committed[j + rs.first_reject] = rs.resampled_id
                rep.verified_steps += 1
                rep.n_accepted += rs.n_accepted
                rep.n_resampled += int(rs.first_reject >= 0)
            else:
                sel = A.threshold_select([q.d for q in o_stats], masked, tau_conf)
                edge = any(abs(q.d - tau_conf) < 1e-6 for q in o_stats)
                got = sorted(rs.committed_idx[:rs.n_committed])
                if sel != got and not edge:
                    rep.mismatches.append(f"{tag}: confidence branch {sel} vs {got}")
                exempt = edge
                for i in got:
                    committed[i] = int(st.xhat[masked.index(i)])
            if exempt:
                rep.exempt_steps += 1
            got_commit = {int(rs.committed_idx[i]): int(rs.committed_tok[i]) for i in range(rs.n_committed)}
            if got_commit != committed:
                rep.mismatches.append(f"{tag}: committed set {got_commit} vs {committed}")
            rep.n_committed += rs.n_committed
            # ---- stage B: the oracle's own forward ------------------------------------------------
            n_c0 = bf["n_cached"]
            q0 = min(n_c0, s0 + j - 1) if shifted else n_c0       # first row of the draft pass
            n_draft_rows = (s0 + j - q0) + (B - j)
            if block_cache and do_b and (stage_b_seqs is None or sid in stage_b_seqs):
                assert n_c0 == s0 and not cfg.is_moe
                sh = shadows[sid]
                sh.extend_blocks(full, s0, _prompt_len(engine, sid), B)
                toks, pos, mask = S.draft_pass_rows([], [], blk, list(range(s0, s0 + B)))
                ol, _ = M.forward(W, cfg, toks, pos, mask, sh.cache, need_logits=masked)
                _cmp(rep, "draft", tag, my_d, ol, logit_atol, logit_rtol)
                rep.stage_b_passes += 1
                if flags[k]:
                    vt, vp, vm = S.verify_pass_rows_with_prefix(blk[:j], list(st.xhat[:L]), s0, MASK)
                    ov, _ = M.forward(W, cfg, vt, vp, vm, sh.cache, need_logits=list(range(j + L, j + 2 * L)))
                    _cmp(rep, "verify", tag, my_v, ov, logit_atol, logit_rtol)
                    rep.stage_b_passes += 1
            elif do_b and (stage_b_seqs is None or sid in stage_b_seqs):
                sh = shadows[sid]
                if not cfg.is_moe:
                    sh.extend(full, n_c0)
                assert sh.n == n_c0 or not cfg.is_moe
                pend_pos = list(range(q0, s0 + j))
                toks, pos, mask = S.draft_pass_rows([full[p] for p in pend_pos], pend_pos, blk[j:], list(range(s0 + j, s0 + B)))
                need = [len(pend_pos) + (i - j) - (1 if shifted else 0) for i in masked]
                forced, tr = None, None
                visible = sh.cache if q0 == n_c0 else [(k_[:q0], v_[:q0]) for k_, v_ in sh.cache]
                if cfg.is_moe:
                    forced = [eid_d[l][drow_all:drow_all + n_draft_rows] for l in range(cfg.n_layers)]
                    tr = {}
                ol, kv = M.forward(W, cfg, toks, pos, mask, visible, need_logits=need, forced_expert_ids=forced, trace=tr)
                if cfg.is_moe:
                    _check_expert_choice(rep, tag + " draft", tr, forced, cfg.top_k)
                    if pend_pos:                       # mirror the engine: pending rows enter the cache
                        sh.cache = M.append_kv(sh.cache, kv, np.arange(len(pend_pos)))
                        sh.n = s0 + j
                _cmp(rep, "draft", tag, my_d, ol, logit_atol, logit_rtol)
                rep.stage_b_passes += 1
                if probe_kv_storage and step_no == 0 and not cfg.is_moe:
                    # the same draft pass by an oracle that keeps K and V in fp64 (cache and in-pass rows): how much of the
                    # engine's distance is the cache's storage format (recorded, not asserted)
                    sh2 = OracleShadow(W, cfg, kv_storage=False)
                    sh2.extend(full, n_c0)
                    vis2 = sh2.cache if q0 == n_c0 else [(k_[:q0], v_[:q0]) for k_, v_ in sh2.cache]
                    ol2, _ = M.forward(W, cfg, toks, pos, mask, vis2, need_logits=need, kv_storage=False)
                    rep.err_without_kv_storage = max(rep.err_without_kv_storage, float(np.abs(my_d.astype(np.float64) - ol2).max()))
                if flags[k]:
                    if not cfg.is_moe:
                        sh.extend(full, s0 + j)
                    if shifted:
                        assert not cfg.is_moe
                        vt, vp, vm = S.verify_pass_rows_shifted(full[s0 + j - 1], list(st.xhat[:L]), s0 + j)
                        vis = [(k_[:s0 + j - 1], v_[:s0 + j - 1]) for k_, v_ in sh.cache]
                        ov, vkv = M.forward(W, cfg, vt, vp, vm, vis, need_logits=list(range(L)))
                    else:
                        vt, vp, vm = S.verify_pass_rows(list(st.xhat[:L]), [s0 + j + i for i in range(L)], MASK)
                        if cfg.is_moe:
                            forced = [eid_v[l][vrow_all:vrow_all + 2 * L] for l in range(cfg.n_layers)]
                            tr = {}
                        ov, vkv = M.forward(W, cfg, vt, vp, vm, sh.cache, need_logits=list(range(L, 2 * L)),
                                            forced_expert_ids=forced, trace=tr)
                    if cfg.is_moe:
                        _check_expert_choice(rep, tag + " verify", tr, forced, cfg.top_k)
                        if rs.n_accepted:              # accepted drafted rows keep their K/V
                            sh.cache = M.append_kv(sh.cache, vkv, np.arange(rs.n_accepted))
                            sh.n += rs.n_accepted
                    _cmp(rep, "verify", tag, my_v, ov, logit_atol, logit_rtol)
                    rep.stage_b_passes += 1
            drow_all += n_draft_rows
            if flags[k]:
                vrow_all += L if shifted else 2 * L
        rep.steps += 1
    return rep


_PROMPT_LEN: Dict[int, int] = {}


def register_prompt_lens(seq_ids, prompts):
    for sid, p in zip(seq_ids, prompts):
        _PROMPT_LEN[sid] = len(p)


def _prompt_len(engine, sid):
    return _PROMPT_LEN[sid]


def _cmp(rep: ParityReport, which: str, tag: str, got: np.ndarray, want: np.ndarray, atol: float, rtol: float):
    err = np.abs(got.astype(np.float64) - want)
    mx = float(err.max())
    if which == "draft":
        rep.max_draft_err = max(rep.max_draft_err, mx)
    else:
        rep.max_verify_err = max(rep.max_verify_err, mx)
    scale = float(np.abs(want).max())
    rep.logit_scale_seen = max(rep.logit_scale_seen, scale)
    rep.max_rel_err = max(rep.max_rel_err, mx / scale)
    bound = atol + rtol * scale
    if mx > bound:
        rep.mismatches.append(f"{tag}: {which} logits off by {mx:.3e} (bound {bound:.3e}, scale {scale:.2f})")


def check_kv(engine, W, cfg, sid, atol: float, block_size: int = 0) -> float:
    """Cache contents of a sequence against the oracle's causal pass over the committed tokens (``block_size`` > 0:
    block-end caching, the oracle's block-causal passes)."""
    stt = engine.debug_seq_state(sid)
    n_c = stt["n_cached"]
    full = list(engine.get_tokens(sid)) + list(stt["block_tokens"])
    sh = OracleShadow(W, cfg)
    if block_size:
        sh.extend_blocks(full, n_c, _prompt_len(engine, sid), block_size)
    else:
        sh.extend(full, n_c)
    worst = 0.0
    for l in range(cfg.n_layers):
        k, v = engine.debug_copy_kv(sid, l, n_c)
        for got, want in ((k, sh.cache[l][0]), (v, sh.cache[l][1])):
            # the bound scales with the magnitude: the cache stores rounded values
            worst = max(worst, float((np.abs(got - want) / np.maximum(1.0, np.abs(want))).max()))
    assert worst <= atol, f"KV cache off by {worst} (relative to max(1, |value|))"
    return worst


def _check_expert_choice(rep: ParityReport, tag: str, trace: dict, forced, top_k: int, tie_tol: float = 5e-3):
    """Where the engine's expert set differs from the oracle's own top-k, every expert in
    the difference must sit within ``tie_tol`` of the oracle's k-th router logit (a near tie
    decided differently by the two precisions); anything else is a wrong selection."""
    for l, (logits, own) in enumerate(zip(trace["router_logits"], trace["expert_ids"])):
        # trace["expert_ids"] holds the ids used (the forced ones); recompute the oracle's own
        order = np.argsort(-logits, axis=-1, kind="stable")
        for r in range(logits.shape[0]):
            mine = set(order[r, :top_k].tolist())
            theirs = set(int(e) for e in forced[l][r])
            rep.moe_rows_checked += 1
            if len(theirs) != top_k:
                rep.mismatches.append(f"{tag}: layer {l} row {r}: duplicate expert ids")
            if mine == theirs:
                continue
            kth = logits[r, order[r, top_k - 1]]
            gap = max(abs(logits[r, e] - kth) for e in mine ^ theirs)
            if gap < tie_tol:
                rep.moe_forced_rows += 1
                rep.moe_max_forced_gap = max(rep.moe_max_forced_gap, float(gap))
            else:
                rep.mismatches.append(f"{tag}: layer {l} row {r}: expert set {sorted(theirs)} vs {sorted(mine)}")


def moe_prefill_shadows(engine, W, cfg, seq_ids, prompts, rep: Optional[ParityReport] = None):
    """Shadows for MoE models: the oracle's causal prefill with the engine's expert choice
    (every prompt must fit one prefill chunk so that the engine's last pass is the prefill)."""
    assert all(len(p) <= 64 for p in prompts)
    rep = rep or ParityReport()
    ids = engine.debug_copy_expert_ids(sum(len(p) for p in prompts))
    out, r0 = {}, 0
    for sid, p in zip(seq_ids, prompts):
        n = len(p)
        forced = [ids[l][r0:r0 + n] for l in range(cfg.n_layers)]
        tr = {}
        _, kv = M.forward(W, cfg, [int(t) for t in p], np.arange(n), M.causal_mask(n), None, need_logits=[],
                          forced_expert_ids=forced, trace=tr)
        _check_expert_choice(rep, f"prefill seq {sid}", tr, forced, cfg.top_k)
        sh = OracleShadow(W, cfg)
        sh.cache = M.append_kv(None, kv, np.arange(n))
        sh.n = n
        out[sid] = sh
        r0 += n
    assert not rep.mismatches, rep.mismatches[:3]
    return out
