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


def _widen(a: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> fp64 (exact)."""
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def _bf16_dev(a: np.ndarray):
    """bf16 bit patterns -> device tensor holding the same bits."""
    return torch.from_numpy(a.view(np.int16)).cuda()


@pytest.mark.parametrize("M,N,K", [(16, 4096, 4096), (5, 1000, 512), (200, 640, 1024), (256, 512, 2048), (33, 384, 64),
                                   (256, 8192, 4096)])
def test_noalloc_gemm_matches_regular_entry_twice(M, N, K):
    """(256, ...): the stated maximum of rows; K = 64: a single k-block; (256, 8192, 4096): partial tiles of a K
    split would not fit the fixed scratch, so the split is lowered to one."""
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
        exact = _widen(x) @ _widen(w).T                              # fp64 product of the same bf16 inputs
        dx, dw = _bf16_dev(x), _bf16_dev(w)
        dy = torch.full((M, N), float("nan"), device="cuda", dtype=torch.float32)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), M, N, K, stream)
        if call == 1:                                                # the first call on a device may load the module's kernels
            assert torch.cuda.mem_get_info()[0] == free_before       # nothing was allocated on the device
        got = dy.cpu().numpy()
        bound = 2e-6 * np.sqrt(K) * np.abs(want).max() + 1e-6     # the tolerance of the GEMM parity test
        assert np.isfinite(got).all()
        assert np.abs(got - want).max() <= bound, (call, np.abs(got - want).max(), bound)
        assert np.abs(got - exact).max() <= 2e-6 * np.sqrt(K) * np.abs(exact).max() + 1e-6, (call, np.abs(got - exact).max())
    with pytest.raises(S2D2Error):           # beyond the stated maximum: a clear error, nothing runs
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), 257, N, K, stream)
    with pytest.raises(S2D2Error):
        gemm_bf16_noalloc(dx.data_ptr(), dw.data_ptr(), dy.data_ptr(), M, N, 100, stream)
    eng.close()
