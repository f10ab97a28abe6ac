// Host side of the persistent pass kernel (pass_kernel.cuh): one cooperative launch runs a
// whole draft pass, verifier pass or prefill chunk of a bf16 dense model with at most 64 rows.
#pragma once
#include "common.cuh"
struct s2d2_ctx;
int pass_init(s2d2_ctx* c);      // after gemm_init and attention_init
void pass_destroy(s2d2_ctx* c);
// Runs the pass described by the uploaded row tables if the persistent kernel takes it.
// *taken = false: nothing was launched and the caller runs the one-kernel-per-operation path.
// sum_ctx: cached tokens visible to the pass, summed over its sequences (for byte accounting).
int pass_run(s2d2_ctx* c, const s2d2::PassView& pv, int max_ctx, int max_rows, long long sum_ctx, float* logits_out,
             bool* taken);
// Timestamps of the last persistent pass (see s2d2_debug_pass_trace).
int pass_copy_trace(s2d2_ctx* c, unsigned long long* out, long long cap, int* n_ctas, int* n_marks);
// Most rows the persistent kernel takes in one pass on this context (0: it is not available).
int pass_max_rows(s2d2_ctx* c);
