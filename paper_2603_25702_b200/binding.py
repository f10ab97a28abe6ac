"""ctypes binding of include/s2d2.h: same names, argument marshalling only.

Every numerical step runs inside the CUDA library.  There is no CPU path: if
``libs2d2.so`` is missing or no CUDA device is present the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

MAX_BLOCK = 32

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB: Optional[C.CDLL] = None


class S2D2Error(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"s2d2 error {code}: {msg}")
        self.code = code


class ModelConfigC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab",
                                         "dtype", "qk_norm", "n_experts", "top_k", "expert_ffn", "n_shared")] + \
               [(n, C.c_float) for n in ("rope_base", "rms_eps", "logit_scale")]


class DecodeConfigC(C.Structure):
    _fields_ = [("block_size", C.c_int32), ("max_batch", C.c_int32), ("max_seq_len", C.c_int32),
                ("kv_page_tokens", C.c_int32), ("n_kv_pages", C.c_int32), ("draft_mode", C.c_int32),
                ("resample", C.c_int32), ("tau_conf", C.c_float), ("ratio_gamma", C.c_float), ("seed", C.c_uint32),
                ("use_tensor_cores", C.c_int32), ("verifier_layout", C.c_int32), ("caching", C.c_int32)]


class TensorDesc(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dtype", C.c_int32), ("ndim", C.c_int32), ("shape", C.c_int64 * 4),
                ("data", C.c_void_p)]


class DraftStats(C.Structure):
    _fields_ = [("seq_id", C.c_int32), ("block_start", C.c_int32), ("first_masked", C.c_int32),
                ("n_masked", C.c_int32), ("span_len", C.c_int32), ("n_hi", C.c_int32), ("mean_conf", C.c_float),
                ("masked_idx", C.c_int32 * MAX_BLOCK), ("xhat", C.c_int32 * MAX_BLOCK),
                ("conf", C.c_float * MAX_BLOCK), ("margin", C.c_float * MAX_BLOCK), ("entropy", C.c_float * MAX_BLOCK)]


class StepResult(C.Structure):
    _fields_ = [("seq_id", C.c_int32), ("verified", C.c_int32), ("n_accepted", C.c_int32),
                ("first_reject", C.c_int32), ("resampled_id", C.c_int32), ("n_committed", C.c_int32),
                ("block_done", C.c_int32), ("n_near_boundary", C.c_int32),
                ("committed_idx", C.c_int32 * MAX_BLOCK), ("committed_tok", C.c_int32 * MAX_BLOCK),
                ("u", C.c_float * MAX_BLOCK), ("a", C.c_float * MAX_BLOCK), ("v", C.c_float * MAX_BLOCK)]


class Counters(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("n_draft_passes", "n_verify_passes", "n_prefill_passes", "n_steps",
                                         "n_committed_tokens", "n_accepted_tokens", "n_resampled", "n_near_boundary",
                                         "n_kernel_launches")] + \
               [("accepted_len_hist", C.c_int64 * (MAX_BLOCK + 1))] + \
               [(n, C.c_double) for n in ("ms_draft", "ms_verify", "ms_accept", "ms_prefill")] + \
               [(n, C.c_int64) for n in ("kv_pages_in_use", "kv_pages_total", "moe_expert_tiles_touched", "h2d_bytes", "d2h_bytes",
                                         "n_rows_draft", "n_rows_verify", "n_rows_prefill", "n_cache_passes")]


class RoutePolicy(C.Structure):
    MIN_SPAN, SCORE, HYSTERESIS, MEAN_CONF, NEVER, UCB = range(6)
    _fields_ = [("policy", C.c_int32), ("p0", C.c_float), ("p1", C.c_float), ("cost", C.c_float),
                ("dynamic_cost", C.c_int32), ("alpha_entropy", C.c_int32), ("alpha_param", C.c_float)]


ROUTE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.POINTER(DraftStats))

EXPORTS = [
    "s2d2_create", "s2d2_destroy", "s2d2_last_error", "s2d2_load_weights", "s2d2_prefill",
    "s2d2_seq_set_rng_stream", "s2d2_draft_block", "s2d2_set_router", "s2d2_set_route_policy", "s2d2_route",
    "s2d2_verify_block", "s2d2_accept_and_commit", "s2d2_generate", "s2d2_get_tokens", "s2d2_release_seq",
    "s2d2_get_counters", "s2d2_reset_counters", "s2d2_set_profiling", "s2d2_set_accept_override", "s2d2_get_gemm_profile", "s2d2_accept_logits", "s2d2_sample_logits", "s2d2_debug_copy_logits",
    "s2d2_debug_copy_kv", "s2d2_debug_seq_state", "s2d2_debug_gemm", "s2d2_debug_gemm2", "s2d2_debug_gemm_swiglu", "s2d2_debug_copy_expert_ids", "s2d2_debug_pass_trace", "s2d2_debug_wait_timeout",
    "s2d2_gemm_bf16_noalloc", "s2d2_noalloc_last_error",
]


def library_path() -> str:
    return os.path.join(_HERE, "libs2d2.so")


def load_library() -> C.CDLL:
    """Load libs2d2.so (built in-tree by ``paper_2603_25702_b200.build``)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        raise S2D2Error(-2, f"{path} is missing: run `python -m paper_2603_25702_b200.build` (there is no CPU fallback)")
    lib = C.CDLL(path)
    lib.s2d2_last_error.restype = C.c_char_p
    lib.s2d2_last_error.argtypes = [C.c_void_p]
    lib.s2d2_noalloc_last_error.restype = C.c_char_p
    lib.s2d2_noalloc_last_error.argtypes = []
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("s2d2_last_error", "s2d2_noalloc_last_error"):
            fn.restype = C.c_int
    lib.s2d2_gemm_bf16_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.s2d2_create.argtypes = [C.POINTER(ModelConfigC), C.POINTER(DecodeConfigC), C.c_void_p, C.POINTER(C.c_void_p)]
    lib.s2d2_destroy.argtypes = [C.c_void_p]
    lib.s2d2_load_weights.argtypes = [C.c_void_p, C.POINTER(TensorDesc), C.c_int32]
    lib.s2d2_prefill.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.POINTER(C.c_int32)), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.s2d2_seq_set_rng_stream.argtypes = [C.c_void_p, C.c_int32, C.c_uint32]
    lib.s2d2_draft_block.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(DraftStats)]
    lib.s2d2_set_router.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.s2d2_set_route_policy.argtypes = [C.c_void_p, C.POINTER(RoutePolicy)]
    lib.s2d2_route.argtypes = [C.c_void_p, C.c_int32, C.POINTER(DraftStats), C.POINTER(C.c_uint8)]
    lib.s2d2_verify_block.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_uint8)]
    lib.s2d2_accept_and_commit.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_uint8), C.POINTER(StepResult)]
    lib.s2d2_generate.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_int32]
    lib.s2d2_get_tokens.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.POINTER(C.c_int32)]
    lib.s2d2_release_seq.argtypes = [C.c_void_p, C.c_int32]
    lib.s2d2_get_counters.argtypes = [C.c_void_p, C.POINTER(Counters)]
    lib.s2d2_reset_counters.argtypes = [C.c_void_p]
    lib.s2d2_set_profiling.argtypes = [C.c_void_p, C.c_int32]
    lib.s2d2_set_accept_override.argtypes = [C.c_void_p, C.c_float]
    lib.s2d2_get_gemm_profile.argtypes = [C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.s2d2_accept_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32),
                                       C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_uint32),
                                       C.POINTER(C.c_int32), C.POINTER(StepResult)]
    lib.s2d2_sample_logits.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_uint32),
                                       C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_float), C.POINTER(C.c_float),
                                       C.POINTER(C.c_float)]
    lib.s2d2_debug_copy_logits.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.POINTER(C.c_int64)]
    lib.s2d2_debug_copy_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.s2d2_debug_seq_state.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    lib.s2d2_debug_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
    lib.s2d2_debug_gemm_swiglu.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.s2d2_debug_gemm2.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_int32, C.c_void_p]
    lib.s2d2_debug_copy_expert_ids.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_int64, C.POINTER(C.c_int32)]
    lib.s2d2_debug_wait_timeout.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32]
    lib.s2d2_debug_pass_trace.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
    _LIB = lib
    return lib


def _i32(a: Sequence[int]):
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data_as(C.POINTER(C.c_int32))


def gemm_bf16_noalloc(d_x: int, d_w: int, d_y: int, M: int, N: int, K: int, stream: int = 0) -> None:
    """y[M, N] = x[M, K] w[N, K]^T on caller-owned device buffers (raw device pointers),
    for hosts that must not allocate device memory: nothing is allocated, the scratch is a
    fixed region inside the library.  Synchronous; calls that overlap on the GPU race on
    that shared scratch.  Make the first call on a device outside any stream capture."""
    lib = load_library()
    rc = lib.s2d2_gemm_bf16_noalloc(C.c_void_p(d_x), C.c_void_p(d_w), C.c_void_p(d_y), M, N, K, C.c_void_p(stream))
    if rc != 0:
        raise S2D2Error(rc, lib.s2d2_noalloc_last_error().decode())


class Engine:
    """One S2D2 context.  ``model`` needs the attributes of s2d2_model_config
    (``dtype`` as "fp32"/"bf16"); ``stream`` is a raw cudaStream_t value
    (e.g. ``torch.cuda.current_stream().cuda_stream``) or 0."""

    def __init__(self, model, block_size: int, max_batch: int, max_seq_len: int, kv_page_tokens: int = 64,
                 n_kv_pages: int = 0, seed: int = 1, tau_conf: float = 0.9, ratio_gamma: float = 1.0,
                 resample: bool = True, stream: int = 0, use_tensor_cores: int = 1, verifier_layout: str = "aligned",
                 draft_mode: str = "greedy", caching: str = "ar"):
        self.lib = load_library()
        self.model = model
        self.block_size = block_size
        self.vocab = model.vocab
        mc = ModelConfigC(model.n_layers, model.d_model, model.n_q_heads, model.n_kv_heads, model.head_dim, model.ffn,
                          model.vocab, 1 if model.dtype == "bf16" else 0, int(model.qk_norm), model.n_experts,
                          model.top_k, model.expert_ffn, model.n_shared, model.rope_base, model.rms_eps,
                          model.logit_scale)
        dc = DecodeConfigC(block_size, max_batch, max_seq_len, kv_page_tokens, n_kv_pages,
                           {"greedy": 0, "sample": 1}[draft_mode], int(resample), tau_conf,
                           ratio_gamma, seed, int(use_tensor_cores), {"aligned": 0, "shifted": 1}[verifier_layout],
                           {"ar": 0, "block": 1}[caching])
        self._h = C.c_void_p()
        rc = self.lib.s2d2_create(C.byref(mc), C.byref(dc), C.c_void_p(stream), C.byref(self._h))
        if rc != 0:
            msg = self.lib.s2d2_last_error(self._h).decode() if self._h else "s2d2_create failed"
            if self._h:
                self.lib.s2d2_destroy(self._h)
                self._h = C.c_void_p()
            raise S2D2Error(rc, msg)
        self._router_ref = None

    # -- helpers ------------------------------------------------------------------------------
    def _check(self, rc: int):
        if rc != 0:
            raise S2D2Error(rc, self.lib.s2d2_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            self.lib.s2d2_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the calls of the header, same names --------------------------------------------------------
    def load_weights(self, tensors: Dict[str, np.ndarray]):
        """uint16 arrays are bfloat16 bit patterns, float32 arrays fp32."""
        descs = (TensorDesc * len(tensors))()
        keep = []
        for i, (name, arr) in enumerate(tensors.items()):
            arr = np.ascontiguousarray(arr)
            keep.append(arr)
            descs[i].name = name.encode()
            descs[i].dtype = 1 if arr.dtype == np.uint16 else 0
            if arr.dtype not in (np.uint16, np.float32):
                raise TypeError(f"{name}: dtype {arr.dtype}")
            descs[i].ndim = arr.ndim
            for k, s in enumerate(arr.shape):
                descs[i].shape[k] = s
            descs[i].data = arr.ctypes.data
        self._check(self.lib.s2d2_load_weights(self._h, descs, len(tensors)))

    def prefill(self, prompts: Sequence[Sequence[int]]) -> List[int]:
        n = len(prompts)
        arrs = [np.ascontiguousarray(p, dtype=np.int32) for p in prompts]
        ptrs = (C.POINTER(C.c_int32) * n)(*[a.ctypes.data_as(C.POINTER(C.c_int32)) for a in arrs])
        lens, lens_p = _i32([len(a) for a in arrs])
        out = np.zeros(n, dtype=np.int32)
        self._check(self.lib.s2d2_prefill(self._h, n, ptrs, lens_p, out.ctypes.data_as(C.POINTER(C.c_int32))))
        return out.tolist()

    def seq_set_rng_stream(self, seq_id: int, stream: int):
        self._check(self.lib.s2d2_seq_set_rng_stream(self._h, seq_id, stream))

    def draft_block(self, seq_ids: Sequence[int]):
        ids, ids_p = _i32(seq_ids)
        out = (DraftStats * len(ids))()
        self._check(self.lib.s2d2_draft_block(self._h, len(ids), ids_p, out))
        return out

    def set_router(self, fn):
        """fn(stats: DraftStats) -> bool, or None for the built-in policy."""
        if fn is None:
            self._router_ref = None
            self._check(self.lib.s2d2_set_router(self._h, None, None))
            return
        cb = ROUTE_FN(lambda user, st: int(bool(fn(st.contents))))
        self._router_ref = cb
        self._check(self.lib.s2d2_set_router(self._h, C.cast(cb, C.c_void_p), None))

    def set_route_policy(self, policy: RoutePolicy):
        self._check(self.lib.s2d2_set_route_policy(self._h, C.byref(policy)))

    def route(self, stats) -> np.ndarray:
        n = len(stats)
        flags = np.zeros(n, dtype=np.uint8)
        self._check(self.lib.s2d2_route(self._h, n, stats, flags.ctypes.data_as(C.POINTER(C.c_uint8))))
        return flags

    def verify_block(self, seq_ids: Sequence[int], flags: Sequence[int]):
        ids, ids_p = _i32(seq_ids)
        fl = np.ascontiguousarray(flags, dtype=np.uint8)
        self._check(self.lib.s2d2_verify_block(self._h, len(ids), ids_p, fl.ctypes.data_as(C.POINTER(C.c_uint8))))

    def accept_and_commit(self, seq_ids: Sequence[int], flags: Sequence[int]):
        ids, ids_p = _i32(seq_ids)
        fl = np.ascontiguousarray(flags, dtype=np.uint8)
        out = (StepResult * len(ids))()
        self._check(self.lib.s2d2_accept_and_commit(self._h, len(ids), ids_p, fl.ctypes.data_as(C.POINTER(C.c_uint8)), out))
        return out

    def generate(self, seq_ids: Sequence[int], n_new_tokens: int):
        ids, ids_p = _i32(seq_ids)
        self._check(self.lib.s2d2_generate(self._h, len(ids), ids_p, n_new_tokens))

    def get_tokens(self, seq_id: int) -> np.ndarray:
        n = C.c_int32()
        self._check(self.lib.s2d2_get_tokens(self._h, seq_id, None, 0, C.byref(n)))
        out = np.zeros(n.value, dtype=np.int32)
        self._check(self.lib.s2d2_get_tokens(self._h, seq_id, out.ctypes.data_as(C.POINTER(C.c_int32)), n.value, C.byref(n)))
        return out

    def release_seq(self, seq_id: int):
        self._check(self.lib.s2d2_release_seq(self._h, seq_id))

    def get_counters(self) -> Counters:
        c = Counters()
        self._check(self.lib.s2d2_get_counters(self._h, C.byref(c)))
        return c

    def reset_counters(self):
        self._check(self.lib.s2d2_reset_counters(self._h))

    def set_accept_override(self, prob: float):
        """prob in (0, 1]: accept test u < prob for every scanned position (speed studies only); 0: the paper's rule."""
        self._check(self.lib.s2d2_set_accept_override(self._h, float(prob)))

    def set_profiling(self, on):
        """0: off; 1: event pairs around the dominant kernels; 2: also the persistent kernel's phase marks."""
        self._check(self.lib.s2d2_set_profiling(self._h, int(on)))

    def get_gemm_profile(self):
        n, ms, b = C.c_int64(), C.c_double(), C.c_double()
        self._check(self.lib.s2d2_get_gemm_profile(self._h, C.byref(n), C.byref(ms), C.byref(b)))
        return {"launches": n.value, "ms": ms.value, "bytes": b.value}

    def accept_logits(self, d_draft_logits: int, d_verify_logits: int, n_seqs: int, l_max: int, span_len, xhat,
                      position0, rng_stream, step):
        """Device pointers (ints) to fp32 [n_seqs*l_max, vocab] logits; host arrays for the rest."""
        sl, sl_p = _i32(span_len)
        xh, xh_p = _i32(np.asarray(xhat).reshape(-1))
        p0, p0_p = _i32(position0)
        rs = np.ascontiguousarray(rng_stream, dtype=np.uint32)
        stp, stp_p = _i32(step)
        out = (StepResult * n_seqs)()
        self._check(self.lib.s2d2_accept_logits(self._h, C.c_void_p(d_draft_logits), C.c_void_p(d_verify_logits), n_seqs,
                                                l_max, sl_p, xh_p, p0_p, rs.ctypes.data_as(C.POINTER(C.c_uint32)), stp_p, out))
        return out

    def sample_logits(self, d_logits: int, n_rows: int, draft_mode: str = "greedy", position=None, rng_stream=None, step=None):
        """SampleFromLogits on device logits (pointer as int, fp32 [n_rows, vocab]): (xhat, conf, margin, entropy)."""
        pos, pos_p = _i32(position if position is not None else [0] * n_rows)
        rs = np.ascontiguousarray(rng_stream if rng_stream is not None else [0] * n_rows, dtype=np.uint32)
        stp, stp_p = _i32(step if step is not None else [0] * n_rows)
        xh = np.zeros(n_rows, dtype=np.int32)
        cf, mg, en = (np.zeros(n_rows, dtype=np.float32) for _ in range(3))
        fp = lambda a: a.ctypes.data_as(C.POINTER(C.c_float))
        self._check(self.lib.s2d2_sample_logits(self._h, C.c_void_p(d_logits), n_rows, {"greedy": 0, "sample": 1}[draft_mode], pos_p,
                                                rs.ctypes.data_as(C.POINTER(C.c_uint32)), stp_p,
                                                xh.ctypes.data_as(C.POINTER(C.c_int32)), fp(cf), fp(mg), fp(en)))
        return xh, cf, mg, en

    def debug_copy_logits(self, which: int, max_rows: int) -> np.ndarray:
        buf = np.empty((max_rows, self.vocab), dtype=np.float32)
        n = C.c_int64()
        self._check(self.lib.s2d2_debug_copy_logits(self._h, which, buf.ctypes.data, buf.size, C.byref(n)))
        return buf[: n.value]

    def debug_copy_kv(self, seq_id: int, layer: int, n_tokens: int):
        shape = (n_tokens, self.model.n_kv_heads, self.model.head_dim)
        k, v = np.empty(shape, dtype=np.float32), np.empty(shape, dtype=np.float32)
        self._check(self.lib.s2d2_debug_copy_kv(self._h, seq_id, layer, n_tokens, k.ctypes.data, v.ctypes.data))
        return k, v

    def debug_seq_state(self, seq_id: int):
        nc, bs, st = C.c_int32(), C.c_int32(), C.c_int32()
        blk = np.zeros(self.block_size, dtype=np.int32)
        self._check(self.lib.s2d2_debug_seq_state(self._h, seq_id, C.byref(nc), C.byref(bs),
                                                  blk.ctypes.data_as(C.POINTER(C.c_int32)), C.byref(st)))
        return {"n_cached": nc.value, "block_start": bs.value, "block_tokens": blk.tolist(), "step": st.value}

    def debug_gemm(self, x: np.ndarray, w: np.ndarray) -> np.ndarray:
        """x [M, K], w [N, K] in the model's storage type (uint16 = bf16 bits, or float32)."""
        x, w = np.ascontiguousarray(x), np.ascontiguousarray(w)
        M, K = x.shape
        N = w.shape[0]
        y = np.empty((M, N), dtype=np.float32)
        self._check(self.lib.s2d2_debug_gemm(self._h, x.ctypes.data, w.ctypes.data, M, N, K, y.ctypes.data))
        return y

    def debug_gemm2(self, x_hi: np.ndarray, x_lo, w: np.ndarray, y: np.ndarray, scale: float = 1.0, accumulate: bool = False) -> np.ndarray:
        """Two-term token operand (bf16 bits; ``x_lo`` may be None): returns scale * (x_hi + x_lo) w^T, added to ``y`` when accumulating."""
        x_hi, w = np.ascontiguousarray(x_hi), np.ascontiguousarray(w)
        x_lo = None if x_lo is None else np.ascontiguousarray(x_lo)
        M, K = x_hi.shape
        N = w.shape[0]
        y = np.ascontiguousarray(y, dtype=np.float32).copy()
        assert y.shape == (M, N)
        self._check(self.lib.s2d2_debug_gemm2(self._h, x_hi.ctypes.data, None if x_lo is None else x_lo.ctypes.data, w.ctypes.data,
                                              M, N, K, C.c_float(scale), int(accumulate), y.ctypes.data))
        return y

    def debug_gemm_swiglu(self, x_hi: np.ndarray, x_lo: np.ndarray, w: np.ndarray):
        """w [2f, K] (gate rows, then up rows), bf16 bits: (act_hi, act_lo) of silu(x w_g^T) * (x w_u^T), bf16 bits [M, f]."""
        x_hi, x_lo, w = np.ascontiguousarray(x_hi), np.ascontiguousarray(x_lo), np.ascontiguousarray(w)
        M, K = x_hi.shape
        f = w.shape[0] // 2
        hi = np.empty((M, f), dtype=np.uint16)
        lo = np.empty((M, f), dtype=np.uint16)
        self._check(self.lib.s2d2_debug_gemm_swiglu(self._h, x_hi.ctypes.data, x_lo.ctypes.data, w.ctypes.data, M, f, K,
                                                    hi.ctypes.data, lo.ctypes.data))
        return hi, lo

    def debug_wait_timeout(self, target: int, limit_polls: int = 1000):
        """Runs the bounded-wait pattern on a word nothing sets; raises S2D2Error(-5) when target > 0."""
        self._check(self.lib.s2d2_debug_wait_timeout(self._h, target, limit_polls))

    # names of the 12 marks a dense layer records, in slot order (see s2d2_debug_pass_trace)
    TRACE_DENSE_MARKS = ("qkv_drained", "rope_barrier_entry", "rope_barrier_exit", "attn_barrier_entry", "attn_barrier_exit",
                         "combine_done", "o_drained", "o_residual_done", "gu_drained", "swiglu_done", "down_drained",
                         "down_residual_done")

    def debug_pass_trace(self):
        """(marks [n_ctas, n_marks], sm_ids [n_ctas]): global-timer ns of the named points of the last persistent pass
        (slot layout in include/s2d2.h: 3 slots of the embedding barrier, 12 marks per dense layer or 9 barrier
        triples per mixture-of-experts layer, 2 marks of the LM-head phase, 2 per sub-GEMM) and the SM each CTA ran on."""
        buf = np.zeros(256 * (3 + (27 + 6 * 21) * self.model.n_layers + 2 + 6 + 1), dtype=np.uint64)
        nc, nm = C.c_int32(), C.c_int32()
        self._check(self.lib.s2d2_debug_pass_trace(self._h, buf.ctypes.data, buf.size, C.byref(nc), C.byref(nm)))
        rows = buf[: nc.value * (nm.value + 1)].reshape(nc.value, nm.value + 1)
        return rows[:, :nm.value].astype(np.int64), rows[:, nm.value].astype(np.int64)

    def debug_copy_expert_ids(self, max_rows: int) -> np.ndarray:
        k, nl = self.model.top_k, self.model.n_layers
        buf = np.zeros(nl * max_rows * k, dtype=np.int32)
        n = C.c_int32()
        self._check(self.lib.s2d2_debug_copy_expert_ids(self._h, buf.ctypes.data_as(C.POINTER(C.c_int32)), buf.size, C.byref(n)))
        return buf[: nl * n.value * k].reshape(nl, n.value, k)
