"""The tensor-core weight-streaming GEMM against a float64 matmul of the same bf16 inputs."""
import numpy as np
import pytest

from s2d2_inputs import bf16_bits_to_f32, f32_to_bf16_bits, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module")
def engine():
    from paper_2603_25702_b200 import Engine
    wl = get_config("t_bf16")
    e = Engine(wl.model, block_size=4, max_batch=1, max_seq_len=64, kv_page_tokens=16,
               stream=torch.cuda.current_stream().cuda_stream)
    yield e
    e.close()


@pytest.mark.parametrize("M,N,K", [(1, 128, 64), (4, 256, 256), (8, 384, 128), (16, 128, 4096), (16, 6144, 4096),
                                   (5, 200, 192), (33, 1000, 512), (64, 4096, 1024), (100, 640, 2048), (257, 300, 320),
                                   (512, 1024, 512), (16, 151936, 256), (3, 64, 704),
                                   (342, 6144, 1024), (200, 384, 512), (160, 4096, 12288)])   # two weight sub-tiles per CTA
def test_gemm_matches_float64(engine, M, N, K):
    rng = np.random.default_rng(M * 1000003 + N * 101 + K)
    x = f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
    w = f32_to_bf16_bits((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
    got = engine.debug_gemm(x, w)
    want = bf16_bits_to_f32(x).astype(np.float64) @ bf16_bits_to_f32(w).astype(np.float64).T
    err = np.abs(got - want).max()
    # fp32 accumulation of exact bf16 products: error ~ K * eps_fp32 * |terms|
    bound = 2e-6 * np.sqrt(K) * np.abs(want).max() + 1e-6
    assert err <= bound, (err, bound)
    # twice the same launch: bitwise identical (split-K partials are summed in a fixed order)
    again = engine.debug_gemm(x, w)
    assert np.array_equal(got, again)


@pytest.mark.parametrize("M,N,K,acc,scale", [
    (65, 256, 256, False, 1.0), (100, 640, 2048, True, 1.0), (181, 6144, 4096, False, 1.0), (265, 4096, 4096, True, 1.0),
    (312, 4096, 12288, True, 1.0), (312, 24576, 4096, False, 1.0), (512, 6144, 4096, False, 0.5), (1024, 4096, 4096, True, 1.0),
    (130, 300, 320, True, 2.0), (96, 151936, 256, False, 4.0), (700, 1000, 128, True, 1.0), (129, 128, 64, False, 1.0),
])
def test_wide_gemm_with_two_term_rows_matches_float64(engine, M, N, K, acc, scale):
    """Passes of more than 64 rows (large batches, prefill): token operand x = hi + lo as two bf16 terms, results that
    leave the CTA as bulk copies (plain, or added to the residual), K splits summed by the CTA that takes a tile's
    last ticket.  Against float64 on the same inputs; the right and bottom edges of the matrix are ragged in some cases."""
    rng = np.random.default_rng(M * 7919 + N * 31 + K)
    x = rng.standard_normal((M, K)).astype(np.float32)
    hi = f32_to_bf16_bits(x)
    lo = f32_to_bf16_bits(x - bf16_bits_to_f32(hi))
    w = f32_to_bf16_bits((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
    y0 = rng.standard_normal((M, N)).astype(np.float32)
    got = engine.debug_gemm2(hi, lo, w, y0, scale=scale, accumulate=acc)
    xs = bf16_bits_to_f32(hi).astype(np.float64) + bf16_bits_to_f32(lo).astype(np.float64)
    want = scale * (xs @ bf16_bits_to_f32(w).astype(np.float64).T) + (y0.astype(np.float64) if acc else 0.0)
    err = np.abs(got - want).max()
    bound = 2e-6 * np.sqrt(K) * np.abs(want).max() + 1e-6
    assert err <= bound, (err, bound)
    again = engine.debug_gemm2(hi, lo, w, y0, scale=scale, accumulate=acc)
    assert np.array_equal(got, again)


@pytest.mark.parametrize("M,f,K", [(65, 128, 64), (181, 768, 512), (312, 12288, 4096), (1024, 1024, 2048), (200, 384, 320)])
def test_gate_up_gemm_with_swiglu_epilogue_matches_float64(engine, M, f, K):
    """Wide passes compute act = silu(x Wg^T) * (x Wu^T) inside the gate/up GEMM (a CTA holds the same 128 rows of the gate
    and of the up half) and write it as two bf16 terms.  Against float64 of the same inputs: the sum of the two terms is
    within two-term bf16 rounding (2^-16 relative) plus the fp32 accumulation error of the GEMM."""
    rng = np.random.default_rng(M * 131 + f * 7 + K)
    x = rng.standard_normal((M, K)).astype(np.float32)
    hi = f32_to_bf16_bits(x)
    lo = f32_to_bf16_bits(x - bf16_bits_to_f32(hi))
    w = f32_to_bf16_bits((rng.standard_normal((2 * f, K)) * (1.0 / np.sqrt(K))).astype(np.float32))
    a_hi, a_lo = engine.debug_gemm_swiglu(hi, lo, w)
    got = bf16_bits_to_f32(a_hi).astype(np.float64) + bf16_bits_to_f32(a_lo).astype(np.float64)
    xs = bf16_bits_to_f32(hi).astype(np.float64) + bf16_bits_to_f32(lo).astype(np.float64)
    y = xs @ bf16_bits_to_f32(w).astype(np.float64).T
    g, u = y[:, :f], y[:, f:]
    want = g / (1.0 + np.exp(-g)) * u
    err = np.abs(got - want).max()
    bound = 2.0 ** -15 * np.abs(want).max() + 4e-6 * np.sqrt(K) * np.abs(y).max() ** 2 + 1e-6
    assert err <= bound, (err, bound)
    # the low term is the rounding remainder of the high one
    assert np.all(np.abs(bf16_bits_to_f32(a_lo)) <= np.abs(bf16_bits_to_f32(a_hi)) * 2.0 ** -7 + 1e-30)
