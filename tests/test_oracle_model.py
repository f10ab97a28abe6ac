"""Pins the oracle's transformer forward to things other than itself:
a separately written composition of torch fp64 library routines for the plain
causal case, structural invariants (RoPE depends on relative positions only;
a cached pass equals a recomputed one), and the MoE top-k path against a dense
evaluation of every expert with zeroed gates."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import model as M
from s2d2_inputs import bf16_bits_to_f32, generate_weights, get_config


def _t(w):
    if w.dtype == np.uint16:
        w = bf16_bits_to_f32(w)
    return torch.from_numpy(np.ascontiguousarray(w)).double()


def _torch_rope_complex(x, pos, base):
    """RoPE as a complex rotation of the pairs (x[i], x[i+hd/2])."""
    hd = x.shape[-1]
    half = hd // 2
    inv = torch.tensor([base ** (-(2.0 * i) / hd) for i in range(half)], dtype=torch.float64)
    ang = pos.double()[:, None] * inv[None, :]
    rot = torch.polar(torch.ones_like(ang), ang)[:, None, :]
    z = torch.complex(x[..., :half], x[..., half:]) * rot
    return torch.cat([z.real, z.imag], dim=-1)


def _torch_causal_forward(W, cfg, tokens):
    """Library-op composition of one causal pass (dense or MoE-free models)."""
    R = len(tokens)
    pos = torch.arange(R)
    h = F.embedding(torch.tensor(tokens), _t(W["embed"]))
    Hq, Hkv, hd = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    for l in range(cfg.n_layers):
        p = f"layers.{l}."
        x = F.rms_norm(h, (cfg.d_model,), _t(W[p + "attn_norm"]), cfg.rms_eps)
        q = F.linear(x, _t(W[p + "wq"])).view(R, Hq, hd)
        k = F.linear(x, _t(W[p + "wk"])).view(R, Hkv, hd)
        v = F.linear(x, _t(W[p + "wv"])).view(R, Hkv, hd)
        if cfg.qk_norm:
            q = F.rms_norm(q, (hd,), _t(W[p + "q_norm"]), cfg.rms_eps)
            k = F.rms_norm(k, (hd,), _t(W[p + "k_norm"]), cfg.rms_eps)
        q, k = _torch_rope_complex(q, pos, cfg.rope_base), _torch_rope_complex(k, pos, cfg.rope_base)
        if cfg.dtype == "bf16":      # K and V are held as the cache stores them: torch's own bfloat16 rounding
            k, v = k.float().bfloat16().double(), v.float().bfloat16().double()
        o = F.scaled_dot_product_attention(q.transpose(0, 1)[None], k.transpose(0, 1)[None], v.transpose(0, 1)[None],
                                           is_causal=True, enable_gqa=True)[0]
        h = h + F.linear(o.transpose(0, 1).reshape(R, Hq * hd), _t(W[p + "wo"]))
        x = F.rms_norm(h, (cfg.d_model,), _t(W[p + "ffn_norm"]), cfg.rms_eps)
        h = h + F.linear(F.silu(F.linear(x, _t(W[p + "w_gate"]))) * F.linear(x, _t(W[p + "w_up"])), _t(W[p + "w_down"]))
    hn = F.rms_norm(h, (cfg.d_model,), _t(W["final_norm"]), cfg.rms_eps)
    return (F.linear(hn, _t(W["lm_head"])) * cfg.logit_scale).numpy()


@pytest.mark.parametrize("name", ["t_f32", "t_bf16"])
def test_causal_pass_matches_library_composition(name):
    wl = get_config(name)
    cfg = wl.model
    W = generate_weights(cfg, seed=11, gain_jitter=0.3)
    rng = np.random.default_rng(0)
    toks = rng.integers(0, cfg.vocab + 1, size=13).tolist()      # includes the chance of a MASK row
    toks[4] = cfg.mask_id
    got, _ = M.forward(W, cfg, toks, np.arange(13), M.causal_mask(13))
    want = _torch_causal_forward(W, cfg, toks)
    assert got.shape == (13, cfg.vocab)
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-11)
    assert np.abs(want).max() > 0.1          # the comparison is not vacuous


def test_rope_depends_on_relative_position_only(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    toks = [3, 7, cfg.mask_id, 9, 1, 0]
    a, _ = M.forward(W, cfg, toks, np.arange(6), M.causal_mask(6))
    b, _ = M.forward(W, cfg, toks, np.arange(6) + 37, M.causal_mask(6))
    np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-11)
    c, _ = M.forward(W, cfg, toks, np.array([0, 1, 2, 4, 5, 6]), M.causal_mask(6))
    assert np.abs(a - c).max() > 1e-6        # positions do matter


def test_cached_pass_equals_recomputed(tiny_f32):
    wl, W = tiny_f32
    cfg = wl.model
    rng = np.random.default_rng(1)
    toks = rng.integers(0, cfg.vocab, size=11).tolist()
    full, kv_full = M.forward(W, cfg, toks, np.arange(11), M.causal_mask(11))
    _, kv_a = M.forward(W, cfg, toks[:6], np.arange(6), M.causal_mask(6), need_logits=[])
    cache = M.append_kv(None, kv_a, np.arange(6))
    tail, kv_b = M.forward(W, cfg, toks[6:], np.arange(6, 11), M.causal_mask(5), cache)
    np.testing.assert_allclose(tail, full[6:], rtol=1e-9, atol=1e-12)
    for l in range(cfg.n_layers):
        np.testing.assert_allclose(kv_b[l][0], kv_full[l][0][6:], rtol=1e-9, atol=1e-13)
        np.testing.assert_allclose(kv_b[l][1], kv_full[l][1][6:], rtol=1e-9, atol=1e-13)


def test_inblock_mask_blocks_information(tiny_f32):
    """A row that may not attend another row does not change when that row's token changes."""
    wl, W = tiny_f32
    cfg = wl.model
    mask = np.array([[1, 0, 0], [1, 1, 0], [1, 0, 1]], dtype=bool)
    a, _ = M.forward(W, cfg, [1, 2, 3], [0, 1, 1], mask)
    b, _ = M.forward(W, cfg, [1, 9, 3], [0, 1, 1], mask)
    np.testing.assert_array_equal(a[0], b[0])
    np.testing.assert_array_equal(a[2], b[2])
    assert np.abs(a[1] - b[1]).max() > 1e-6
    full = np.ones((3, 3), dtype=bool)
    c, _ = M.forward(W, cfg, [1, 2, 3], [0, 1, 1], full)
    d, _ = M.forward(W, cfg, [1, 9, 3], [0, 1, 1], full)
    assert np.abs(c[0] - d[0]).max() > 1e-6   # bidirectional rows do see it


def test_moe_topk_equals_dense_with_zeroed_gates(tiny_moe):
    wl, W = tiny_moe
    cfg = wl.model
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, cfg.d_model))
    got = M.moe_ffn(x, W, "layers.0.", cfg)
    # dense restatement: every expert evaluated, gates zero outside the top-k
    R = _t(W["layers.0.router"]).numpy()
    p = torch.softmax(torch.from_numpy(x @ R.T), dim=-1).numpy()
    want = np.zeros_like(x)
    for r in range(5):
        keep = sorted(range(cfg.n_experts), key=lambda e: (-p[r, e], e))[: cfg.top_k]
        g = np.zeros(cfg.n_experts)
        g[keep] = p[r, keep] / p[r, keep].sum()
        assert abs(g.sum() - 1) < 1e-12
        for e in range(cfg.n_experts):
            wg, wu, wd = (_t(W[f"layers.0.experts.{n}"][e]).numpy() for n in ("w_gate", "w_up", "w_down"))
            a = x[r] @ wg.T
            want[r] += g[e] * (((a / (1 + np.exp(-a))) * (x[r] @ wu.T)) @ wd.T)
    sg, su, sd = (_t(W[f"layers.0.shared.{n}"]).numpy() for n in ("w_gate", "w_up", "w_down"))
    a = x @ sg.T
    want += ((a / (1 + np.exp(-a))) * (x @ su.T)) @ sd.T
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-13)


def test_moe_model_forward_runs_and_is_finite(tiny_moe):
    wl, W = tiny_moe
    cfg = wl.model
    logits, kv = M.forward(W, cfg, [1, 2, cfg.mask_id], [0, 1, 2], M.causal_mask(3))
    assert logits.shape == (3, cfg.vocab) and np.isfinite(logits).all()
    assert kv[0][0].shape == (3, cfg.n_kv_heads, cfg.head_dim)


def test_kv_is_held_as_the_cache_stores_it():
    """bf16 models: every K/V value the oracle hands out is a bfloat16 number (low 16 bits of
    its fp32 pattern are zero), is the bfloat16 nearest to the fp64 value (ties to even, one
    rounding), and equals torch's conversion wherever that is a single rounding too (inputs that
    are fp32 numbers); fp32 models keep fp64 K/V."""
    class Cfg:
        dtype = "bf16"
    x = np.random.default_rng(5).standard_normal(4096) * np.logspace(-6, 3, 4096)
    got = M.as_stored_kv(x, Cfg)
    assert (got.astype(np.float32).view(np.uint32) & 0xFFFF == 0).all() and (got.astype(np.float32) == got).all()
    # nearest: within half a unit in the last place of the result's binade (8 significant bits)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(got))) - 7)
    assert (np.abs(x - got) <= ulp / 2).all()
    # torch converts fp64 through fp32; on fp32 inputs that is one rounding and must agree exactly
    x32 = x.astype(np.float32).astype(np.float64)
    assert (M.as_stored_kv(x32, Cfg) == torch.from_numpy(x32).float().bfloat16().double().numpy()).all()
    # where the two-step conversion differs on fp64 inputs, the single rounding is strictly closer
    two_step = torch.from_numpy(x).float().bfloat16().double().numpy()
    differ = got != two_step
    assert (np.abs(x - got)[differ] < np.abs(x - two_step)[differ]).all()
    ties = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8])      # exactly between two bfloat16 neighbours: to even
    assert M.as_stored_kv(ties, Cfg).tolist() == [1.0, 1.0 + 2.0 ** -6]
    # a value that the fp32 detour rounds the wrong way: just above a tie in fp64, exactly the tie in fp32
    sneaky = np.array([1.0 + 2.0 ** -8 + 2.0 ** -40])
    assert M.as_stored_kv(sneaky, Cfg).tolist() == [1.0 + 2.0 ** -7]
    assert M.as_stored_kv(np.array([0.0, -0.0, 2.0 ** -130, 1e-45]), Cfg).tolist() == [0.0, -0.0, 2.0 ** -130, 0.0]
    Cfg.dtype = "fp32"
    assert M.as_stored_kv(x, Cfg) is x
    wl = get_config("t_bf16")
    W = generate_weights(wl.model, seed=2)
    _, kv = M.forward(W, wl.model, [1, 2, 3], np.arange(3), M.causal_mask(3), need_logits=[])
    for k, v in kv:
        for a in (k, v):
            assert (a.astype(np.float32).view(np.uint32) & 0xFFFF == 0).all() and (a.astype(np.float32) == a).all()
