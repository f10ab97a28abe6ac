"""The allocation-free GEMM entry point, through the C ABI.

It serves hosts that may not allocate device memory while they run (the GPU is fully
reserved by a framework's own arena, or a cudaMalloc would stall a latency-critical
loop), so its scratch is a fixed region inside the library.  Here it must reproduce the
regular GEMM entry on two calls in a row: the second call finds the scratch as the first
one left it.  The file name sorts last so that a run that stops at the first failure has
already run every other test."""
import numpy as np
import pytest

from s2d2_inputs import f32_to_bf16_bits, get_config

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


def _bf16_dev(a: np.ndarray):
    """bf16 bit patterns -> device tensor holding the same bits."""
    return torch.from_numpy(a.view(np.int16)).cuda()


@pytest.mark.parametrize("M,N,K", [(16, 4096, 4096), (5, 1000, 512), (200, 640, 1024)])
def test_noalloc_gemm_matches_regular_entry_twice(M, N, K):
    from paper_2603_25702_b200 import Engine, S2D2Error, gemm_bf16_noalloc
    wl = get_config("t_bf16")
    eng = Engine(wl.model, block_size=4, max_batch=1, max_seq_len=64, kv_page_tokens=16,
                 stream=torch.cuda.current_stream().cuda_stream)
    rng = np.random.default_rng(7 + M)
    stream = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        x = f32_to_bf16_bits(rng.standard_normal((M, K)).astype(np.float32))
        w = f32_to_bf16_bits((rng.standard_normal((N, K)) * 0.05).astype(np.float32))
        want = eng.debug_gemm(x, w)
        dx, dw = _bf16_dev(x), _bf16_dev(w)
        dy = torch.full((M, N), float("nan"), device="cuda", dtype=torch.float32)
        torch.cuda.synchronize()
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), M, N, K, stream)
        got = dy.cpu().numpy()
        bound = 2e-6 * np.sqrt(K) * np.abs(want).max() + 1e-6     # the tolerance of the GEMM parity test
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= bound, (call, np.abs(got - want).max(), bound)
    with pytest.raises(S2D2Error):           # beyond the stated maximum: a clear error, nothing runs
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), 257, N, K, stream)
    with pytest.raises(S2D2Error):
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), M, N, 100, stream)
    eng.close()
