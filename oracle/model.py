"""fp64 transformer forward of the oracle (test infrastructure only).

The paper treats the network x_theta as given; the shapes come from the
synthetic workloads: a pre-norm decoder with RMSNorm, grouped-query attention
with rotate-half RoPE (optional per-head RMSNorm on q and k), SwiGLU feed-forward
or a softmax-top-k mixture of experts with a shared expert, an untied LM head
and a [MASK] embedding row past the vocabulary.

One function serves every pass of the decode step.  The caller gives the rows
of the pass (token or MASK, position id), a boolean rows-by-rows mask saying
which rows of the same pass a row may attend to (this is where the verifier
mask and the partially causal drafting mask of Section "Self-Verification Mode"
enter), and the cached prefix K/V, which every row sees in full.
Weights arrive as the stored values (bfloat16 bit patterns or fp32) and are
widened exactly to fp64; all arithmetic is fp64.  One storage format besides the weights'
enters: K and V of a bf16 model are bfloat16 values, as its KV cache stores them (as_stored_kv).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import numpy as np

KV = List[Tuple[np.ndarray, np.ndarray]]  # per layer: K [n, Hkv, hd], V [n, Hkv, hd]


def widen(w: np.ndarray) -> np.ndarray:
    """Stored tensor -> fp64 (exact)."""
    if w.dtype == np.uint16:
        return (w.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return w.astype(np.float64)


def as_stored_kv(x: np.ndarray, cfg) -> np.ndarray:
    """K and V as the cache holds them.  The cache of a bf16 model stores bfloat16 (the
    workloads name a "paged bf16 KV cache"), so for such a model K and V are bfloat16 values
    wherever they are used: rounded once, fp64 to the nearest bfloat16 with ties to even, where
    they are produced (after RoPE for K).  The rounding works on the fp64 bit pattern (bfloat16
    keeps 7 of the 52 fraction bits; a carry moves into the exponent by itself), so no fp32
    value lies in between; below bfloat16's normal range the spacing is the fixed 2^-133.
    fp32 models keep them unrounded in the oracle.  Returned as fp64."""
    if cfg.dtype != "bf16":
        return x
    x = np.ascontiguousarray(x, dtype=np.float64)
    u = x.view(np.uint64)
    drop = np.uint64(45)
    r = (u + (((u >> drop) & np.uint64(1)) + np.uint64((1 << 44) - 1))) & ~np.uint64((1 << 45) - 1)
    out = r.view(np.float64).copy()
    tiny = np.abs(x) < 2.0 ** -126
    if tiny.any():
        q = 2.0 ** -133
        out[tiny] = np.rint(x[tiny] / q) * q
    return out


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * gain over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotate-half RoPE. x: [R, H, hd]; pair i is (x[i], x[i + hd/2]), angle
    pos * base^(-2i/hd)."""
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = base ** (-np.arange(half, dtype=np.float64) * 2.0 / hd)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]        # [R, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def swiglu(x: np.ndarray, w_gate, w_up, w_down) -> np.ndarray:
    return (silu(x @ widen(w_gate).T) * (x @ widen(w_up).T)) @ widen(w_down).T


def moe_select(router_logits: np.ndarray, top_k: int):
    """Softmax over all experts, keep the top_k largest (ties -> lowest id),
    renormalise the kept gates to sum to one. Returns (ids [R,k], gates [R,k])."""
    z = router_logits - router_logits.max(axis=-1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=-1, keepdims=True)
    ids = np.argsort(-p, axis=-1, kind="stable")[:, :top_k]
    g = np.take_along_axis(p, ids, axis=-1)
    g = g / g.sum(axis=-1, keepdims=True)
    return ids, g


def moe_ffn(x: np.ndarray, W: Dict[str, np.ndarray], prefix: str, cfg,
            forced_ids: Optional[np.ndarray] = None, trace: Optional[dict] = None) -> np.ndarray:
    """Routed experts (top-k, renormalised gates) plus the shared expert.

    ``forced_ids`` [R, k] replaces the oracle's own expert choice (used when a
    comparison must take the integer decision in the other side's precision);
    the gates are still the oracle's softmax values renormalised over them."""
    logits = x @ widen(W[prefix + "router"]).T
    ids, gates = moe_select(logits, cfg.top_k)
    if forced_ids is not None:
        z = logits - logits.max(axis=-1, keepdims=True)
        p = np.exp(z)
        p /= p.sum(axis=-1, keepdims=True)
        ids = np.asarray(forced_ids)
        gates = np.take_along_axis(p, ids, axis=-1)
        gates = gates / gates.sum(axis=-1, keepdims=True)
    if trace is not None:
        trace.setdefault("router_logits", []).append(logits)
        trace.setdefault("expert_ids", []).append(ids)
    out = np.zeros_like(x)
    wg, wu, wd = W[prefix + "experts.w_gate"], W[prefix + "experts.w_up"], W[prefix + "experts.w_down"]
    for r in range(x.shape[0]):
        for e, g in zip(ids[r], gates[r]):
            out[r] += g * swiglu(x[r:r + 1], wg[e], wu[e], wd[e])[0]
    if cfg.n_shared:
        out += swiglu(x, W[prefix + "shared.w_gate"], W[prefix + "shared.w_up"], W[prefix + "shared.w_down"])
    return out


def forward(W: Dict[str, np.ndarray], cfg, tokens, positions, inblock_mask,
            kv_prefix: Optional[KV] = None, need_logits=None,
            forced_expert_ids: Optional[List[np.ndarray]] = None,
            trace: Optional[dict] = None, kv_storage: bool = True):
    """One pass of the network over R rows.

    tokens [R] (cfg.mask_id = MASK), positions [R], inblock_mask [R, R] bool
    (row r attends row c of this pass iff mask[r, c]); every row attends all of
    kv_prefix.  Returns (logits [R or len(need_logits), V], kv_rows) where
    kv_rows[l] = (K [R, Hkv, hd], V [R, Hkv, hd]) are this pass's own K/V.
    kv_storage=False keeps K and V in fp64 even for a bf16 model (used only to measure how much
    of a logit difference is the cache's storage format).
    """
    tokens = np.asarray(tokens, dtype=np.int64)
    positions = np.asarray(positions, dtype=np.int64)
    mask = np.asarray(inblock_mask, dtype=bool)
    R = tokens.shape[0]
    Hq, Hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    group = Hq // Hkv
    h = widen(W["embed"][tokens])
    kv_rows: KV = []
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        x = rmsnorm(h, widen(W[p + "attn_norm"]), cfg.rms_eps)
        q = (x @ widen(W[p + "wq"]).T).reshape(R, Hq, hd)
        k = (x @ widen(W[p + "wk"]).T).reshape(R, Hkv, hd)
        v = (x @ widen(W[p + "wv"]).T).reshape(R, Hkv, hd)
        if cfg.qk_norm:
            q = rmsnorm(q, widen(W[p + "q_norm"]), cfg.rms_eps)
            k = rmsnorm(k, widen(W[p + "k_norm"]), cfg.rms_eps)
        q = rope(q, positions, cfg.rope_base)
        k = rope(k, positions, cfg.rope_base)
        if kv_storage:
            k, v = as_stored_kv(k, cfg), as_stored_kv(v, cfg)
        kv_rows.append((k, v))
        if kv_prefix is not None and kv_prefix[l][0].shape[0] > 0:
            K_all = np.concatenate([kv_prefix[l][0], k], axis=0)
            V_all = np.concatenate([kv_prefix[l][1], v], axis=0)
            n_pre = kv_prefix[l][0].shape[0]
        else:
            K_all, V_all, n_pre = k, v, 0
        allow = np.concatenate([np.ones((R, n_pre), dtype=bool), mask], axis=1)
        attn = np.empty((R, Hq, hd))
        for hq in range(Hq):
            s = q[:, hq, :] @ K_all[:, hq // group, :].T / np.sqrt(float(hd))
            s = np.where(allow, s, -np.inf)
            s = s - s.max(axis=-1, keepdims=True)
            e = np.exp(s)
            attn[:, hq, :] = (e / e.sum(axis=-1, keepdims=True)) @ V_all[:, hq // group, :]
        h = h + attn.reshape(R, Hq * hd) @ widen(W[p + "wo"]).T
        x = rmsnorm(h, widen(W[p + "ffn_norm"]), cfg.rms_eps)
        if cfg.is_moe:
            forced = None if forced_expert_ids is None else forced_expert_ids[l]
            h = h + moe_ffn(x, W, p, cfg, forced, trace)
        else:
            h = h + swiglu(x, W[p + "w_gate"], W[p + "w_up"], W[p + "w_down"])
    if need_logits is not None:
        h = h[np.asarray(need_logits, dtype=np.int64)]
    if h.shape[0] == 0:
        return np.zeros((0, cfg.vocab)), kv_rows
    hn = rmsnorm(h, widen(W["final_norm"]), cfg.rms_eps)
    lm = W["lm_head"]
    logits = np.empty((hn.shape[0], cfg.vocab))
    step = 16384                      # widen the head in slabs to bound memory
    for lo in range(0, cfg.vocab, step):
        logits[:, lo:lo + step] = hn @ widen(lm[lo:lo + step]).T
    return logits * cfg.logit_scale, kv_rows


def causal_mask(n: int) -> np.ndarray:
    return np.tril(np.ones((n, n), dtype=bool))


def append_kv(cache: Optional[KV], rows: KV, idx) -> KV:
    """cache ⊕ rows[idx] per layer (the K ⊕ K^b update of the decoding loop)."""
    idx = np.asarray(idx, dtype=np.int64)
    out: KV = []
    for l, (k, v) in enumerate(rows):
        if cache is None:
            out.append((k[idx].copy(), v[idx].copy()))
        else:
            out.append((np.concatenate([cache[l][0], k[idx]], axis=0),
                        np.concatenate([cache[l][1], v[idx]], axis=0)))
    return out
