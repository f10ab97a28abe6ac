// GEMM dispatch of the forward pass.
#include "gemm.h"

#include "context.h"
#include "kernels_simt.cuh"

using namespace s2d2;

int gemm_init(s2d2_ctx*) { return S2D2_OK; }
void gemm_destroy(s2d2_ctx*) {}

template <typename TW, typename TX>
static void gemm_simt(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale,
                      int accumulate) {
    constexpr int ROWS = 8;
    dim3 grid((N + 3) / 4, (M + ROWS - 1) / ROWS);
    gemm_simt_kernel<TW, TX, ROWS><<<grid, 128, 0, c->stream>>>((const TX*)X, (const TW*)W, Y, M, N, K, ldy, scale, accumulate);
    c->cnt.n_kernel_launches++;
}

int gemm(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale, int accumulate) {
    if (c->m.dtype == S2D2_DTYPE_F32) gemm_simt<float, float>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
    else gemm_simt<bf16, bf16>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
    return S2D2_OK;
}
