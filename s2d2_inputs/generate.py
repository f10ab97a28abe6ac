"""Seeded generators for weights and prompts (no method arithmetic here).

Weights are i.i.d. N(0, init_std^2), drawn per tensor in fixed-size chunks from
numpy's Philox bit generator keyed by (seed, crc32(tensor name), chunk), so a
tensor's values do not depend on which other tensors exist or on the number of
worker threads.  For "bf16" models the matrices are rounded to bfloat16
(round-to-nearest-even) and returned as uint16 bit patterns; both the oracle
and the CUDA path start from exactly these bits.  Norm gains are fp32 and equal
to 1 unless ``gain_jitter`` is given (tests use it so that a dropped gain shows).
"""
from __future__ import annotations

import zlib
from concurrent.futures import ThreadPoolExecutor
from typing import Dict, List, Tuple

import numpy as np

from .configs import ModelConfig, WorkloadConfig

_CHUNK = 1 << 22  # elements per independently seeded chunk


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (nearest, ties to even); returns uint16 bits."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounding = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + rounding) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to fp32 exactly."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def weight_shapes(m: ModelConfig) -> List[Tuple[str, Tuple[int, ...], str]]:
    """(name, shape, kind) for every tensor; kind is "matrix" or "gain".

    Matrices are stored [out_features, in_features] (y = x @ W.T)."""
    d, hd = m.d_model, m.head_dim
    out: List[Tuple[str, Tuple[int, ...], str]] = [("embed", (m.vocab + 1, d), "matrix")]
    for l in range(m.n_layers):
        p = f"layers.{l}."
        out.append((p + "attn_norm", (d,), "gain"))
        out.append((p + "wq", (m.n_q_heads * hd, d), "matrix"))
        out.append((p + "wk", (m.n_kv_heads * hd, d), "matrix"))
        out.append((p + "wv", (m.n_kv_heads * hd, d), "matrix"))
        out.append((p + "wo", (d, m.n_q_heads * hd), "matrix"))
        if m.qk_norm:
            out.append((p + "q_norm", (hd,), "gain"))
            out.append((p + "k_norm", (hd,), "gain"))
        out.append((p + "ffn_norm", (d,), "gain"))
        if m.is_moe:
            f = m.expert_ffn
            out.append((p + "router", (m.n_experts, d), "matrix"))
            out.append((p + "experts.w_gate", (m.n_experts, f, d), "matrix"))
            out.append((p + "experts.w_up", (m.n_experts, f, d), "matrix"))
            out.append((p + "experts.w_down", (m.n_experts, d, f), "matrix"))
            if m.n_shared:
                fs = f * m.n_shared
                out.append((p + "shared.w_gate", (fs, d), "matrix"))
                out.append((p + "shared.w_up", (fs, d), "matrix"))
                out.append((p + "shared.w_down", (d, fs), "matrix"))
        else:
            out.append((p + "w_gate", (m.ffn, d), "matrix"))
            out.append((p + "w_up", (m.ffn, d), "matrix"))
            out.append((p + "w_down", (d, m.ffn), "matrix"))
    out.append(("final_norm", (d,), "gain"))
    out.append(("lm_head", (m.vocab, d), "matrix"))
    return out


def _fill_chunk(dst: np.ndarray, lo: int, hi: int, seed: int, name_key: int,
                chunk: int, std: float, as_bf16: bool) -> None:
    ss = np.random.SeedSequence([seed, name_key, chunk])
    rng = np.random.Generator(np.random.Philox(ss))
    x = rng.standard_normal(hi - lo, dtype=np.float32)
    x *= np.float32(std)
    if as_bf16:
        dst[lo:hi] = f32_to_bf16_bits(x)
    else:
        dst[lo:hi] = x


def generate_weights(m: ModelConfig, seed: int = 0, gain_jitter: float = 0.0,
                     threads: int = 0) -> Dict[str, np.ndarray]:
    """All tensors of the model as numpy arrays (uint16 bf16 bits or fp32)."""
    import os
    threads = threads or min(32, os.cpu_count() or 1)
    as_bf16 = m.dtype == "bf16"
    out: Dict[str, np.ndarray] = {}
    jobs = []
    for name, shape, kind in weight_shapes(m):
        key = zlib.crc32(name.encode())
        n = int(np.prod(shape))
        if kind == "gain":
            g = np.ones(n, dtype=np.float32)
            if gain_jitter:
                rng = np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, key, 0])))
                g += np.float32(gain_jitter) * rng.standard_normal(n, dtype=np.float32)
            out[name] = g.reshape(shape)
            continue
        flat = np.empty(n, dtype=np.uint16 if as_bf16 else np.float32)
        out[name] = flat.reshape(shape)
        for c, lo in enumerate(range(0, n, _CHUNK)):
            jobs.append((flat, lo, min(n, lo + _CHUNK), seed, key, c, m.init_std, as_bf16))
    if threads > 1 and len(jobs) > 1:
        with ThreadPoolExecutor(threads) as ex:
            list(ex.map(lambda a: _fill_chunk(*a), jobs))
    else:
        for a in jobs:
            _fill_chunk(*a)
    return out


def generate_prompts(wl: WorkloadConfig, seed: int | None = None) -> List[np.ndarray]:
    """``wl.batch`` prompts of token ids uniform in [0, vocab), lengths uniform
    in the workload's inclusive range."""
    seed = wl.prompt_seed if seed is None else seed
    rng = np.random.Generator(np.random.Philox(np.random.SeedSequence([seed, 0x70726F6D])))
    lo, hi = wl.prompt_len
    prompts = []
    for _ in range(wl.batch):
        n = int(rng.integers(lo, hi + 1))
        prompts.append(rng.integers(0, wl.model.vocab, size=n, dtype=np.int64).astype(np.int32))
    return prompts
