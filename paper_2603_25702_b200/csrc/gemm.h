// Y[M, N] (+)= scale * X[M, K] * W[N, K]^T for the model's storage type.
// X is fp32 (fp32 model) or bf16 (bf16 model); W is the stored matrix; Y is fp32.
#pragma once
struct s2d2_ctx;
int gemm_init(s2d2_ctx* c);
void gemm_destroy(s2d2_ctx* c);
int gemm(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale, int accumulate);
