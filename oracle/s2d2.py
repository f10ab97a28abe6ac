"""The S2D2 decode loop of the oracle, step by step (test infrastructure only).

Follows Algorithm "Block-wise autoregressive decoding" (outer loop) and
Algorithm "SampleBlock for S2D2" (inner loop), with the verifier mask of
Eq. (ver_mask) (the 2L construction for position-aligned models) and the
partially causal drafting/caching mask of Eq. (draft_mask).

Readings taken where the paper leaves a choice (each is restated in the
design notes of the repository):
  * Prefill is a causal pass over the prompt.
  * Caching is the AR-like variant: a committed token's K/V depends only on
    tokens at or before it.  Then the K/V that the verifier's drafted-token
    rows (top-left causal block of the 2L mask) produce for accepted tokens are
    final and enter the cache at once; the separate end-of-block cache pass of
    the outer loop becomes redundant (``literal_block_kv`` below restates it
    for a cross-check).
  * A committed token that has no K/V yet (a resampled token, or tokens
    committed by the confidence branch) is "pending": the next draft pass
    carries it as a causal row and appends its K/V.
  * T = B: every step commits at least one token, so a block always finishes.
  * No bonus token after an all-accept step (the 2L pass has no row L+1).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional

import numpy as np

from . import accept as A
from . import model as M
from . import philox


def draft_pass_rows(pending_tokens, pending_pos, block_tokens, block_pos):
    """Rows and in-pass mask of a draft pass.

    Pending rows (committed, not yet cached) are causal among themselves and
    see no block row; block rows (from the first masked position to the end of
    the block, MASK or already known) see every row of the pass: this is
    Eq. (draft_mask) restricted to the rows that are not in the cache."""
    P, Bn = len(pending_tokens), len(block_tokens)
    R = P + Bn
    mask = np.zeros((R, R), dtype=bool)
    mask[:P, :P] = M.causal_mask(P)
    mask[P:, :] = True
    tokens = np.concatenate([np.asarray(pending_tokens, dtype=np.int64), np.asarray(block_tokens, dtype=np.int64)])
    pos = np.concatenate([np.asarray(pending_pos, dtype=np.int64), np.asarray(block_pos, dtype=np.int64)])
    return tokens, pos, mask


def verify_pass_rows(xhat, positions, mask_id):
    """Rows and mask of the 2L verifier pass, Eq. (ver_mask):
    [[A_L, 0], [A_L^<, I_L]] over [drafted tokens ; MASK copies], both halves
    at the same position ids."""
    L = len(xhat)
    mask = np.zeros((2 * L, 2 * L), dtype=bool)
    mask[:L, :L] = M.causal_mask(L)
    mask[L:, :L] = np.tril(np.ones((L, L), dtype=bool), k=-1)
    mask[L:, L:] = np.eye(L, dtype=bool)
    tokens = np.concatenate([np.asarray(xhat, dtype=np.int64), np.full(L, mask_id, dtype=np.int64)])
    pos = np.concatenate([np.asarray(positions, dtype=np.int64)] * 2)
    return tokens, pos, mask


def verify_pass_rows_with_prefix(prefix_tokens, xhat, block_start, mask_id):
    """Verifier rows when the block's committed prefix x^b_{<j} has no K/V in the cache (block-end caching): the
    block-size-1 view needs those tokens as causal context, so they ride along as rows.  Rows: the j prefix tokens
    and the L drafted tokens (one causal run of j + L rows), then the L MASK copies of the span; the MASK copy of
    span position i sees the token rows strictly to its left and itself: Eq. (ver_mask) over the first j + L
    positions of the block, with the MASK copies of the prefix positions left out."""
    j, L = len(prefix_tokens), len(xhat)
    n = j + L
    tokens, pos, mask = verify_pass_rows(list(prefix_tokens) + list(xhat), list(range(block_start, block_start + n)), mask_id)
    keep = list(range(n)) + list(range(n + j, 2 * n))
    return tokens[keep], pos[keep], mask[np.ix_(keep, keep)]


def verify_pass_rows_shifted(prev_token, xhat, first_position):
    """Rows and mask of the verifier pass of a right-shifted model (Section "Self-Verification
    Mode", last sentence: there the plain causal mask already gives the verifier view).  In such a
    model the logits at position i - 1 score the token at position i, so the drafted span
    xhat_1..xhat_L at positions first_position.. is scored by L causal rows: the last committed
    token (position first_position - 1), whose logits score xhat_1, followed by xhat_1..xhat_{L-1};
    row k scores xhat_{k+1}.  xhat_L needs no row.  No MASK copies: L rows instead of 2L."""
    L = len(xhat)
    tokens = np.asarray([int(prev_token)] + [int(t) for t in xhat[:L - 1]], dtype=np.int64)
    pos = np.arange(first_position - 1, first_position - 1 + L, dtype=np.int64)
    return tokens, pos, M.causal_mask(L)


@dataclass
class StepTrace:
    block_start: int
    j: int                       # first masked index of the block at step start
    n_ctx: int                   # cache length after the draft pass appended pending rows
    masked: List[int]            # masked in-block indices M_t
    span: List[int]              # first contiguous masked span C_t (in-block indices)
    xhat: List[int]              # proposal per masked position (aligned with ``masked``)
    d: List[float]
    margin: List[float]
    entropy: List[float]
    verified: bool
    draft_logits: Optional[np.ndarray] = None     # [len(masked), V]
    verify_logits: Optional[np.ndarray] = None    # [L, V]
    u_accept: List[float] = field(default_factory=list)
    u_resample: List[float] = field(default_factory=list)
    result: Optional[A.AcceptResult] = None
    committed: List[int] = field(default_factory=list)   # in-block indices written this step
    committed_tokens: List[int] = field(default_factory=list)


class SequenceOracle:
    """One sequence decoded by S2D2; independent of every other sequence."""

    def __init__(self, W, cfg, block_size: int, seed: int, seq_stream: int,
                 route: Callable[[StepTrace], bool] = None, tau_conf: float = 0.9,
                 draft_mode: str = "greedy", gamma: float = 1.0, keep_logits: bool = False,
                 resample: bool = True, layout: str = "aligned", caching: str = "ar"):
        self.W, self.cfg, self.B = W, cfg, block_size
        self.seed, self.seq_stream = seed, seq_stream
        self.route = route or (lambda st: len(st.span) >= 1)      # minimum-span policy, tau_span = 1
        self.tau_conf, self.draft_mode, self.gamma = tau_conf, draft_mode, gamma
        self.keep_logits = keep_logits
        # False: the reject-only variant of the paper's failure-case study (Appendix, D2F LLaDA table): no residual
        # resampling, the first rejected position stays masked and is drafted again in the next step
        self.resample = resample
        # "aligned": logits of the row at position i score position i (the 2L verifier, Eq. (ver_mask)).
        # "shifted": right-shifted model, logits of the row at position i - 1 score position i, in the draft pass
        # and in the verifier pass alike; the verifier is L plain causal rows (verify_pass_rows_shifted).  Every
        # pass then starts with the row of the last committed token, whether its K/V is cached already or not:
        # the cache visible to the pass ends before that position and the row's K/V is written (again).
        assert layout in ("aligned", "shifted")
        self.layout = layout
        # "ar": the partially causal drafting/caching mask of Eq. (draft_mask) (K/V of committed tokens are causal and
        # enter the cache as they are committed).  "block": the standard block-diffusion pattern of Algorithm
        # "Block-wise autoregressive decoding": every row of the block sees the whole block in the draft pass
        # (Eq. (draft_mask) with j = 0), nothing of the block is cached while it is being decoded, and once it has no
        # MASK left one more pass over it (full attention inside the block) yields K^b, V^b, which are appended.
        assert caching in ("ar", "block") and not (caching == "block" and layout == "shifted")
        self.caching = caching
        self.n_cache_passes = 0
        self.tokens: List[int] = []       # finalised tokens before the current block
        self.cache: Optional[M.KV] = None
        self.n_c = 0                      # tokens whose K/V is cached
        self.xb: List[int] = []           # current block buffer (mask_id = masked)
        self.step_index = 0
        self.trace: List[StepTrace] = []
        self.n_draft_passes = 0
        self.n_verify_passes = 0

    # -- prefill: causal pass over the prompt -------------------------------------------------
    def prefill(self, prompt):
        prompt = [int(t) for t in prompt]
        n = len(prompt)
        _, kv = M.forward(self.W, self.cfg, prompt, np.arange(n), M.causal_mask(n), None, need_logits=[])
        self.cache = M.append_kv(None, kv, np.arange(n))
        self.tokens = prompt
        self.n_c = n
        self.xb = []

    def _all_tokens(self):
        return self.tokens + [t for t in self.xb]

    # -- one iteration of the SampleBlock loop -------------------------------------------------
    def step(self) -> StepTrace:
        cfg, B = self.cfg, self.B
        MASK = cfg.mask_id
        if not self.xb:
            self.xb = [MASK] * B                      # a new block of MASKs
        s = len(self.tokens)
        j = self.xb.index(MASK)
        if self.caching == "block":
            return self._step_block_caching(s, j)
        full = self._all_tokens()
        shifted = self.layout == "shifted"
        q0 = min(self.n_c, s + j - 1) if shifted else self.n_c       # first row of the pass
        if q0 < self.n_c:                                            # the last committed token is run again as a row
            self.cache = [(k[:q0], v[:q0]) for k, v in self.cache]
            self.n_c = q0
        pend_pos = list(range(q0, s + j))
        pend_tok = [full[p] for p in pend_pos]
        blk_pos = list(range(s + j, s + B))
        blk_tok = self.xb[j:]
        tokens, pos, mask = draft_pass_rows(pend_tok, pend_pos, blk_tok, blk_pos)
        P = len(pend_pos)
        masked = [i for i in range(B) if self.xb[i] == MASK]
        # the row whose logits score in-block position i: its own row, or the row one position to the left
        need = [P + (i - j) - (1 if shifted else 0) for i in masked]
        logits, kv = M.forward(self.W, cfg, tokens, pos, mask, self.cache, need_logits=need)
        self.n_draft_passes += 1
        if P:
            self.cache = M.append_kv(self.cache, kv, np.arange(P))
            self.n_c += P
        stats = []
        for r, i in enumerate(masked):
            u = philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_DRAFT)
            stats.append(A.sample_from_logits(logits[r], self.draft_mode, u))
        L = 1
        while j + L < B and self.xb[j + L] == MASK:
            L += 1
        span = list(range(j, j + L))
        st = StepTrace(s, j, self.n_c, masked, span, [q.xhat for q in stats], [q.d for q in stats],
                       [q.margin for q in stats], [q.entropy for q in stats], False)
        if self.keep_logits:
            st.draft_logits = logits
        st.verified = bool(self.route(st))
        if st.verified:
            xhat = st.xhat[:L]                       # masked[0:L] is exactly the span
            if shifted:
                vt, vp, vm = verify_pass_rows_shifted(full[s + j - 1], xhat, s + j)
                visible = [(k[:s + j - 1], v[:s + j - 1]) for k, v in self.cache]
                vlogits, vkv = M.forward(self.W, cfg, vt, vp, vm, visible, need_logits=list(range(L)))
                # vkv row 0 is the last committed token again, rows 1.. are xhat_1..xhat_{L-1}
                vkv = [(k[1:], v[1:]) for k, v in vkv]
            else:
                vt, vp, vm = verify_pass_rows(xhat, [s + i for i in span], MASK)
                vlogits, vkv = M.forward(self.W, cfg, vt, vp, vm, self.cache, need_logits=list(range(L, 2 * L)))
            self.n_verify_passes += 1
            st.u_accept = [philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_ACCEPT) for i in span]
            st.u_resample = [philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_RESAMPLE) for i in span]
            res = A.accept_scan(logits[:L], vlogits, xhat, st.u_accept, st.u_resample, self.gamma, resample=self.resample)
            st.result = res
            if self.keep_logits:
                st.verify_logits = vlogits
            for k in range(res.n_accepted):
                self.xb[j + k] = int(xhat[k])
                st.committed.append(j + k)
                st.committed_tokens.append(int(xhat[k]))
            # accepted drafted tokens keep the K/V their verifier rows produced (the shifted layout has no row for xhat_L)
            n_keep = min(res.n_accepted, L - 1) if shifted else res.n_accepted
            if n_keep:
                self.cache = M.append_kv(self.cache, vkv, np.arange(n_keep))
                self.n_c += n_keep
            if res.first_reject >= 0 and self.resample:
                self.xb[j + res.first_reject] = int(res.resampled)
                st.committed.append(j + res.first_reject)
                st.committed_tokens.append(int(res.resampled))
        else:
            for i in A.threshold_select(st.d, masked, self.tau_conf):
                self.xb[i] = int(st.xhat[masked.index(i)])
                st.committed.append(i)
                st.committed_tokens.append(self.xb[i])
        self.step_index += 1
        if MASK not in self.xb:
            self.tokens = self.tokens + self.xb
            self.xb = []
        self.trace.append(st)
        return st

    # -- the same iteration under block-end caching ---------------------------------------------------
    def _step_block_caching(self, s: int, j: int) -> StepTrace:
        cfg, B = self.cfg, self.B
        MASK = cfg.mask_id
        assert self.n_c == s
        blk_pos = list(range(s, s + B))
        tokens, pos, mask = draft_pass_rows([], [], self.xb, blk_pos)          # j = 0: every row sees the whole block
        masked = [i for i in range(B) if self.xb[i] == MASK]
        logits, _ = M.forward(self.W, cfg, tokens, pos, mask, self.cache, need_logits=masked)
        self.n_draft_passes += 1
        stats = []
        for r, i in enumerate(masked):
            u = philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_DRAFT)
            stats.append(A.sample_from_logits(logits[r], self.draft_mode, u))
        L = 1
        while j + L < B and self.xb[j + L] == MASK:
            L += 1
        span = list(range(j, j + L))
        st = StepTrace(s, j, self.n_c, masked, span, [q.xhat for q in stats], [q.d for q in stats],
                       [q.margin for q in stats], [q.entropy for q in stats], False)
        if self.keep_logits:
            st.draft_logits = logits
        st.verified = bool(self.route(st))
        if st.verified:
            xhat = st.xhat[:L]
            vt, vp, vm = verify_pass_rows_with_prefix(self.xb[:j], xhat, s, MASK)
            vlogits, _ = M.forward(self.W, cfg, vt, vp, vm, self.cache, need_logits=list(range(j + L, j + 2 * L)))
            self.n_verify_passes += 1
            st.u_accept = [philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_ACCEPT) for i in span]
            st.u_resample = [philox.uniform(self.seed, s + i, self.seq_stream, self.step_index, philox.STREAM_RESAMPLE) for i in span]
            res = A.accept_scan(logits[:L], vlogits, xhat, st.u_accept, st.u_resample, self.gamma, resample=self.resample)
            st.result = res
            if self.keep_logits:
                st.verify_logits = vlogits
            for k in range(res.n_accepted):
                self.xb[j + k] = int(xhat[k])
                st.committed.append(j + k)
                st.committed_tokens.append(int(xhat[k]))
            if res.first_reject >= 0 and self.resample:
                self.xb[j + res.first_reject] = int(res.resampled)
                st.committed.append(j + res.first_reject)
                st.committed_tokens.append(int(res.resampled))
        else:
            for i in A.threshold_select(st.d, masked, self.tau_conf):
                self.xb[i] = int(st.xhat[masked.index(i)])
                st.committed.append(i)
                st.committed_tokens.append(self.xb[i])
        self.step_index += 1
        if MASK not in self.xb:
            # K^b, V^b <- x_theta(x^b): one pass over the finished block, full attention inside it
            _, kv = M.forward(self.W, cfg, self.xb, blk_pos, np.ones((B, B), dtype=bool), self.cache, need_logits=[])
            self.cache = M.append_kv(self.cache, kv, np.arange(B))
            self.n_c += B
            self.n_cache_passes += 1
            self.tokens = self.tokens + self.xb
            self.xb = []
        self.trace.append(st)
        return st

    def generate(self, prompt, n_new: int):
        self.prefill(prompt)
        target = len(self.tokens) + n_new
        while len(self.tokens) < target:
            self.step()
        return self.tokens[len(prompt):]


def literal_block_kv(W, cfg, block_tokens, block_start, cache):
    """The end-of-block cache pass of the outer loop written literally under
    the fully causal drafting mask (j = B): K/V of a finished block from one
    causal pass over it on top of the cache."""
    n = len(block_tokens)
    _, kv = M.forward(W, cfg, block_tokens, np.arange(block_start, block_start + n),
                      M.causal_mask(n), cache, need_logits=[])
    return kv


def greedy_ar_decode(W, cfg, prompt, n_new: int):
    """Plain greedy decoding in block-size-1 mode: each new position is one
    MASK row on top of the causal cache (what B = 1 block diffusion reduces to)."""
    toks = [int(t) for t in prompt]
    n = len(toks)
    _, kv = M.forward(W, cfg, toks, np.arange(n), M.causal_mask(n), None, need_logits=[])
    cache = M.append_kv(None, kv, np.arange(n))
    pending: List[int] = []
    out = []
    for _ in range(n_new):
        pos0 = len(toks) - len(pending)
        tokens, pos, mask = draft_pass_rows(pending, list(range(pos0, len(toks))), [cfg.mask_id], [len(toks)])
        logits, kv = M.forward(W, cfg, tokens, pos, mask, cache, need_logits=[len(pending)])
        if pending:
            cache = M.append_kv(cache, kv, np.arange(len(pending)))
        t = int(np.argmax(logits[0]))
        out.append(t)
        toks.append(t)
        pending = [t]
    return out
