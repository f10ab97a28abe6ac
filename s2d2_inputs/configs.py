"""Model and workload shapes of the synthetic configurations.

The five named workloads mirror the shapes the method was evaluated on
(1.7B/4B/8B-class dense block-diffusion decoders and a Mini-class MoE), with
random-init weights standing in for trained ones.  The extra "t_*" entries are
small shapes used by tests so that every code path (GQA, QK-norm, MoE, bf16,
paging) is exercised at a size a CPU finishes in seconds.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Tuple


@dataclass(frozen=True)
class ModelConfig:
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int                      # dense SwiGLU width (0 for MoE models)
    vocab: int
    dtype: str = "bf16"           # "bf16" | "fp32": storage type of the matrices
    rope_base: float = 1.0e6
    rms_eps: float = 1.0e-6
    qk_norm: bool = True
    logit_scale: float = 1.0
    n_experts: int = 0            # routed experts (0 = dense FFN)
    top_k: int = 0
    expert_ffn: int = 0
    n_shared: int = 0             # shared experts (each of width expert_ffn)
    init_std: float = 0.02

    @property
    def mask_id(self) -> int:
        """Token id of [MASK]: one extra embedding row past the vocabulary."""
        return self.vocab

    @property
    def is_moe(self) -> bool:
        return self.n_experts > 0


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    model: ModelConfig
    batch: int
    prompt_len: Tuple[int, int]   # inclusive range; equal ends = fixed length
    block_size: int
    gen_tokens: int
    kv_page_tokens: int = 64
    route: str = "always"         # "always" | "mean_conf" (verify iff mean draft confidence < tau_route)
    tau_route: float = 0.9
    tau_conf: float = 0.9         # confidence threshold of the non-verified branch
    weight_seed: int = 0
    prompt_seed: int = 0
    philox_seed: int = 1


_c1 = ModelConfig("tiny-fp32", 2, 256, 4, 4, 64, 704, 4096, dtype="fp32",
                  rope_base=1.0e4, qk_norm=False, logit_scale=4.0)
_c2 = ModelConfig("dense-1.7b", 28, 2048, 16, 8, 128, 6144, 151936)
_c3 = ModelConfig("dense-4b", 36, 2560, 32, 8, 128, 9728, 151936)
_c4 = ModelConfig("dense-8b", 36, 4096, 32, 8, 128, 12288, 151936)
_c5 = ModelConfig("moe-mini", 20, 2048, 16, 4, 128, 0, 157184,
                  n_experts=256, top_k=8, expert_ffn=512, n_shared=1)

# small shapes for tests
_t_bf16 = ModelConfig("t-dense-bf16", 2, 256, 4, 2, 64, 512, 1000)
_t_bf16_128 = ModelConfig("t-dense-bf16-hd128", 2, 512, 4, 2, 128, 768, 2000)
_t_moe = ModelConfig("t-moe-bf16", 2, 256, 4, 2, 64, 0, 1000,
                     n_experts=16, top_k=4, expert_ffn=128, n_shared=1)
_t_moe128 = ModelConfig("t-moe128-bf16", 2, 256, 4, 2, 64, 0, 1000,
                        n_experts=128, top_k=8, expert_ffn=128, n_shared=1)
# the attention geometry of the 8B-/4B-class and of the MoE workloads (query / kv heads, head_dim, 64-token pages)
# on a narrow two-layer body, so that the CPU side can afford contexts of one to two thousand tokens
_t_geo32 = ModelConfig("t-geo-32q8kv", 2, 1024, 32, 8, 128, 2048, 2000)
_t_geo16 = ModelConfig("t-geo-16q4kv", 2, 1024, 16, 4, 128, 2048, 2000)
_t_f32 = ModelConfig("t-dense-fp32", 2, 64, 2, 1, 32, 96, 50, dtype="fp32",
                     rope_base=1.0e4, qk_norm=True, logit_scale=3.0)

CONFIGS = {
    "c1": WorkloadConfig("c1", _c1, 1, (64, 64), 4, 32),
    "c2": WorkloadConfig("c2", _c2, 1, (256, 256), 4, 512),
    "c3": WorkloadConfig("c3", _c3, 8, (128, 512), 4, 512, route="mean_conf"),
    "c4": WorkloadConfig("c4", _c4, 1, (1024, 1024), 8, 1024),
    "c4b32": WorkloadConfig("c4b32", _c4, 32, (1024, 1024), 8, 1024),
    # the paper's batched runs on the 8B-class model use block size 16 and batch sizes up to 64 (its table of batched
    # throughput): draft passes of 1024 rows, verifier passes of 2048 rows (the 2L construction)
    "c4b64": WorkloadConfig("c4b64", _c4, 64, (1024, 1024), 16, 1024),
    "c5": WorkloadConfig("c5", _c5, 1, (512, 512), 32, 1024),
    "t_bf16": WorkloadConfig("t_bf16", _t_bf16, 3, (5, 70), 4, 16, kv_page_tokens=16),
    "t_bf16_128": WorkloadConfig("t_bf16_128", _t_bf16_128, 2, (60, 130), 8, 24),
    "t_moe": WorkloadConfig("t_moe", _t_moe, 2, (9, 40), 8, 16, kv_page_tokens=16),
    "t_moe128": WorkloadConfig("t_moe128", _t_moe128, 2, (9, 40), 8, 16, kv_page_tokens=16),
    "t_f32": WorkloadConfig("t_f32", _t_f32, 2, (3, 20), 4, 12, kv_page_tokens=8),
    "t_geo32": WorkloadConfig("t_geo32", _t_geo32, 1, (1100, 1100), 8, 24),
    "t_geo16": WorkloadConfig("t_geo16", _t_geo16, 1, (1100, 1100), 32, 64),
}


def get_config(name: str, **overrides) -> WorkloadConfig:
    """Look up a workload; keyword overrides replace WorkloadConfig fields
    (prefix ``model_`` to replace a ModelConfig field)."""
    wl = CONFIGS[name]
    m_over = {k[6:]: v for k, v in overrides.items() if k.startswith("model_")}
    w_over = {k: v for k, v in overrides.items() if not k.startswith("model_")}
    if m_over:
        w_over["model"] = replace(wl.model, **m_over)
    return replace(wl, **w_over) if w_over else wl
