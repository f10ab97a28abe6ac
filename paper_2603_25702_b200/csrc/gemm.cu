// GEMM dispatch of the forward pass.
#include "gemm.h"

#include "context.h"
#include "kernels_simt.cuh"

using namespace s2d2;

int gemm_init(s2d2_ctx*) { return S2D2_OK; }
void gemm_destroy(s2d2_ctx* c) {
    for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
    c->prof_events.clear();
}

template <typename TW, typename TX>
static void gemm_simt(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale,
                      int accumulate) {
    constexpr int ROWS = 8;
    dim3 grid((N + 3) / 4, (M + ROWS - 1) / ROWS);
    gemm_simt_kernel<TW, TX, ROWS><<<grid, 128, 0, c->stream>>>((const TX*)X, (const TW*)W, Y, M, N, K, ldy, scale, accumulate);
    c->cnt.n_kernel_launches++;
}

void gemm_prof_begin(s2d2_ctx* c) {
    if (!c->profiling) return;
    if (c->prof_used + 2 > c->prof_events.size()) {
        for (int i = 0; i < 512; ++i) {
            cudaEvent_t e;
            cudaEventCreate(&e);
            c->prof_events.push_back(e);
        }
    }
    cudaEventRecord(c->prof_events[c->prof_used], c->stream);
}
void gemm_prof_end(s2d2_ctx* c, double bytes) {
    if (!c->profiling) return;
    cudaEventRecord(c->prof_events[c->prof_used + 1], c->stream);
    c->prof_used += 2;
    c->prof_bytes += bytes;
    c->prof_launches++;
}
int gemm_prof_collect(s2d2_ctx* c) {
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return S2D2_ERR_CUDA;
    for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
        float ms = 0;
        cudaEventElapsedTime(&ms, c->prof_events[i], c->prof_events[i + 1]);
        c->prof_ms_done += ms;
    }
    c->prof_used = 0;
    return S2D2_OK;
}

int gemm(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale, int accumulate) {
    size_t es = c->m.dtype == S2D2_DTYPE_F32 ? 4 : 2;
    gemm_prof_begin(c);
    struct End {
        s2d2_ctx* c;
        double b;
        ~End() { gemm_prof_end(c, b); }
    } end{c, (double)N * K * es + (double)M * K * es + (double)M * N * 4 * (accumulate ? 2 : 1)};
    if (c->m.dtype == S2D2_DTYPE_F32) gemm_simt<float, float>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
    else gemm_simt<bf16, bf16>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
    return S2D2_OK;
}
