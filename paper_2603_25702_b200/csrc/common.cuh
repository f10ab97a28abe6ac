// Shared device-side types and small helpers of the S2D2 kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace s2d2 {

typedef __nv_bfloat16 bf16;

// Row flags of a pass.
enum : int {
    ROW_WRITE_KV = 1,   // this row's K/V is written to the sequence's cache page at its position
};

// Device view of one pass (prefill chunk, draft pass or verifier pass).
// Rows of one sequence are contiguous; bit b of row_mask[r] says that row r may
// attend row (seq_row0[row_seq[r]] + b) of the same pass.  Every row attends the
// whole cached prefix [0, seq_nctx) of its sequence.
struct PassView {
    int n_rows;
    int n_seqs;
    int n_logit_rows;
    const int* row_token;
    const int* row_pos;
    const int* row_seq;          // index into the seq_* arrays of this pass
    const int* row_flags;
    const unsigned long long* row_mask;
    const int* logit_rows;       // rows whose logits are needed
    const int* seq_nctx;         // cached tokens visible to the pass
    const int* seq_row0;
    const int* seq_nrows;
    const int* seq_pages;        // [n_seqs, max_pages] page ids of the sequence
    int max_pages;
};

// Paged KV pool: [layer][page][K|V][kv_head][token_in_page][head_dim].
template <typename T>
struct KvPool {
    T* base;
    int page_tokens, page_shift;
    int n_kv_heads, head_dim;
    size_t page_stride;      // elements per page = 2 * Hkv * page_tokens * hd
    size_t layer_stride;     // elements per layer = n_pages * page_stride

    __device__ __forceinline__ T* ptr(int layer, int page, int kv, int head, int tok) const {
        return base + (size_t)layer * layer_stride + (size_t)page * page_stride +
               ((size_t)(kv * n_kv_heads + head) * page_tokens + tok) * head_dim;
    }
};

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Philox4x32-10 (Salmon et al. 2011) and the uniform convention of the decode
// step: counter = (absolute position, sequence stream, step, stream id),
// key = (seed, 0), u = ((x0 >> 8) + 0.5) * 2^-24 in (0, 1).
__host__ __device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                               uint32_t k0, uint32_t k1) {
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c0;
}
enum : uint32_t { STREAM_ACCEPT = 0, STREAM_RESAMPLE = 1, STREAM_DRAFT = 2 };
__host__ __device__ __forceinline__ double philox_uniform(uint32_t seed, uint32_t position, uint32_t seq_stream,
                                                          uint32_t step, uint32_t stream) {
    uint32_t x = philox_first_word(position, seq_stream, step, stream, seed, 0u);
    return ((double)(x >> 8) + 0.5) * (1.0 / 16777216.0);
}

}  // namespace s2d2
