// Y[M, N] (+)= scale * X[M, K] * W[N, K]^T for the model's storage type.
// X is fp32 (fp32 model) or bf16 (bf16 model); W is the stored matrix; Y is fp32.
// X_lo (bf16 models, may be null): the low halves of a two-term input, X = X + X_lo.
#pragma once
struct s2d2_ctx;
int gemm_init(s2d2_ctx* c);
void gemm_destroy(s2d2_ctx* c);
int gemm(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale, int accumulate,
         const void* X_lo = nullptr);
// act[M, f] = silu(X Wg^T) * (X Wu^T) with W = [Wg; Wu] ([2f, K]), written as two bf16 terms (act, act_lo), in one kernel.
// Returns -1 when the shape or the model takes the separate GEMM and SwiGLU kernels instead (nothing was launched).
int gemm_swiglu(s2d2_ctx* c, const void* X, const void* X_lo, const void* W, int M, int f, int K, void* act, void* act_lo);
// Profiling helpers: bracket a launch with an event pair while profiling is on.
void gemm_prof_begin(s2d2_ctx* c);
void gemm_prof_end(s2d2_ctx* c, double algorithmic_bytes);
int gemm_prof_collect(s2d2_ctx* c);   // synchronises, folds finished pairs into the totals
// Drops cached tensor maps of a buffer that is about to be freed.
void gemm_forget(s2d2_ctx* c, const void* ptr);
// 2D bf16 tensor map [rows, cols] with boxes of box_rows x 64 columns and the 128-byte swizzle.
// `out` points to a CUtensorMap (128 bytes). Returns 0 on success.
int gemm_encode_map(s2d2_ctx* c, void* out, const void* ptr, unsigned long long rows, int cols, int box_rows);
// 3D bf16 tensor map [rows, mid, cols] (cols contiguous) with boxes of box_rows x box_mid x 64 columns, 128-byte swizzle.
int gemm_encode_map3(s2d2_ctx* c, void* out, const void* ptr, int cols, int mid, unsigned long long rows, int box_mid, int box_rows);
bool gemm_tc_available(s2d2_ctx* c);
// After a kernel gave up on a bounded wait: a split-K CTA that left early took no ticket, so the tile counters no
// longer return to zero by themselves; clear them (enqueued on the context's stream).
void gemm_reset_tickets(s2d2_ctx* c);
