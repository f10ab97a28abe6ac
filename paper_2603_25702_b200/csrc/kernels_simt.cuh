// Portable SIMT kernels of the forward pass: every op of the pass in its plain
// form.  They serve the fp32 model (whose tolerance forbids tensor-core input
// rounding), all the small glue ops of the bf16 path, and act as the in-library
// fallback for shapes the tensor-core kernels do not take.
#pragma once
#include "common.cuh"

namespace s2d2 {

// h[r, :] = embed[token[r], :]  (token == vocab selects the [MASK] row)
template <typename TW>
__global__ void embed_kernel(const TW* __restrict__ embed, const int* __restrict__ row_token, float* __restrict__ h,
                             int d) {
    int r = blockIdx.x;
    const TW* src = embed + (size_t)row_token[r] * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) h[(size_t)r * d + i] = to_f32(src[i]);
}

__device__ __forceinline__ float block_sum(float v, float* sh) {
    v = warp_sum(v);
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sh[w] = v;
    __syncthreads();
    int nw = (blockDim.x + 31) >> 5;
    float t = (threadIdx.x < nw) ? sh[threadIdx.x] : 0.f;
    if (w == 0) {
        t = warp_sum(t);
        if (lane == 0) sh[0] = t;
    }
    __syncthreads();
    return sh[0];
}

// Stores v as hi = T(v) and, when a second buffer is given, lo = T(v - hi): the GEMMs and the
// attention of bf16 models take such two-term inputs (16 significant bits instead of 8).
template <typename T>
__device__ __forceinline__ void store_two_term(T* hi, T* lo, size_t i, float v) {
    const T h = from_f32<T>(v);
    hi[i] = h;
    if (lo) lo[i] = from_f32<T>(v - to_f32(h));
}
// Four consecutive values at once (i a multiple of 4): one 8- or 16-byte store per buffer.
__device__ __forceinline__ void store_two_term_x4(float* hi, float*, size_t i, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(hi + i) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store_two_term_x4(bf16* hi, bf16* lo, size_t i, float a, float b, float c, float d) {
    const __nv_bfloat162 h0 = __floats2bfloat162_rn(a, b), h1 = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&h0);
    u.y = *reinterpret_cast<const uint32_t*>(&h1);
    *reinterpret_cast<uint2*>(hi + i) = u;
    if (lo) {
        const __nv_bfloat162 l0 = __floats2bfloat162_rn(a - __low2float(h0), b - __high2float(h0));
        const __nv_bfloat162 l1 = __floats2bfloat162_rn(c - __low2float(h1), d - __high2float(h1));
        u.x = *reinterpret_cast<const uint32_t*>(&l0);
        u.y = *reinterpret_cast<const uint32_t*>(&l1);
        *reinterpret_cast<uint2*>(lo + i) = u;
    }
}
// out[i, :] = rmsnorm(h[rows ? rows[i] : i, :]) * gain, written as TO (out_lo: low halves, may be null).
template <typename TO>
__global__ void rmsnorm_kernel(const float* __restrict__ h, const int* __restrict__ rows, const float* __restrict__ gain,
                               TO* __restrict__ out, TO* __restrict__ out_lo, int d, float eps) {
    __shared__ float sh[32];
    int i = blockIdx.x;
    const float* x = h + (size_t)(rows ? rows[i] : i) * d;
    const bool vec = (d & 3) == 0;
    float ss = 0.f;
    if (vec) {
        for (int c = threadIdx.x; c < d / 4; c += blockDim.x) {
            const float4 v = reinterpret_cast<const float4*>(x)[c];
            ss += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) ss += x[c] * x[c];
    }
    ss = block_sum(ss, sh);
    float inv = rsqrtf(ss / (float)d + eps);
    // rsqrtf is approximate (2 ulp); refine once so the fp32 model stays within 1e-4 relative
    float m = ss / (float)d + eps;
    inv = inv * (1.5f - 0.5f * m * inv * inv);
    if (vec) {
        for (int c = threadIdx.x; c < d / 4; c += blockDim.x) {
            const float4 v = reinterpret_cast<const float4*>(x)[c], g = reinterpret_cast<const float4*>(gain)[c];
            store_two_term_x4(out, out_lo, (size_t)i * d + 4 * c, v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
        }
    } else {
        for (int c = threadIdx.x; c < d; c += blockDim.x) store_two_term(out, out_lo, (size_t)i * d + c, x[c] * inv * gain[c]);
    }
}

// Y[m, n] (+)= scale * sum_k X[m, k] * W[n, k].  One warp per output column and
// tile of ROWS rows.  ldy: row stride of Y.
template <typename TW, typename TX, int ROWS>
__global__ void gemm_simt_kernel(const TX* __restrict__ X, const TW* __restrict__ W, float* __restrict__ Y, int M,
                                 int N, int K, int ldy, float scale, int accumulate) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (warp >= N) return;
    int m0 = blockIdx.y * ROWS;
    const TW* w = W + (size_t)warp * K;
    float acc[ROWS];
#pragma unroll
    for (int r = 0; r < ROWS; ++r) acc[r] = 0.f;
    for (int k = lane; k < K; k += 32) {
        float wv = to_f32(w[k]);
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
            if (m0 + r < M) acc[r] += wv * to_f32(X[(size_t)(m0 + r) * K + k]);
    }
#pragma unroll
    for (int r = 0; r < ROWS; ++r) {
        float s = warp_sum(acc[r]);
        if (lane == 0 && m0 + r < M) {
            float* y = Y + (size_t)(m0 + r) * ldy + warp;
            *y = accumulate ? (*y + scale * s) : scale * s;
        }
    }
}

// Per (row, head) of the fused QKV output: optional per-head RMSNorm (q and k),
// rotate-half RoPE from a host-built fp64->fp32 table, then
//   q -> q_out [M, Hq, hd];  k, v -> this pass's K/V rows [M, Hkv, hd]
//   and, for rows flagged ROW_WRITE_KV, into the sequence's cache page.
template <typename TA, typename TKV>
__global__ void qk_rope_kv_kernel(const float* __restrict__ qkv, PassView pv, const float* __restrict__ q_gain,
                                  const float* __restrict__ k_gain, const float* __restrict__ rope_cos,
                                  const float* __restrict__ rope_sin, TA* __restrict__ q_out, TA* __restrict__ q_lo, TKV* __restrict__ k_rows,
                                  TKV* __restrict__ v_rows, KvPool<TKV> pool, int layer, int Hq, int Hkv, int hd,
                                  float eps, int qk_norm) {
    __shared__ float sh[32];
    int r = blockIdx.x, head = blockIdx.y;
    int half = hd >> 1;
    int i = threadIdx.x;  // pair index, blockDim.x == half
    const float* src = qkv + (size_t)r * (Hq + 2 * Hkv) * hd + (size_t)head * hd;
    float x1 = src[i], x2 = src[i + half];
    bool is_q = head < Hq, is_k = !is_q && head < Hq + Hkv;
    if (is_q || is_k) {
        if (qk_norm) {
            float ss = block_sum(x1 * x1 + x2 * x2, sh);
            float m = ss / (float)hd + eps;
            float inv = rsqrtf(m);
            inv = inv * (1.5f - 0.5f * m * inv * inv);
            const float* g = is_q ? q_gain : k_gain;
            x1 = x1 * inv * g[i];
            x2 = x2 * inv * g[i + half];
        }
        int pos = pv.row_pos[r];
        float c = rope_cos[(size_t)pos * half + i], s = rope_sin[(size_t)pos * half + i];
        float y1 = x1 * c - x2 * s, y2 = x2 * c + x1 * s;
        x1 = y1;
        x2 = y2;
    }
    if (is_q) {
        const size_t o = ((size_t)r * Hq + head) * hd;
        store_two_term(q_out, q_lo, o + i, x1);
        store_two_term(q_out, q_lo, o + i + half, x2);
        return;
    }
    int kvh = is_k ? head - Hq : head - Hq - Hkv;
    TKV* rows = is_k ? k_rows : v_rows;
    TKV a = from_f32<TKV>(x1), b = from_f32<TKV>(x2);
    TKV* dst = rows + ((size_t)r * Hkv + kvh) * hd;
    dst[i] = a;
    dst[i + half] = b;
    if (pv.row_flags[r] & ROW_WRITE_KV) {
        int sq = pv.row_seq[r];
        int pos = pv.row_pos[r];
        int page = pv.seq_pages[(size_t)sq * pv.max_pages + (pos >> pool.page_shift)];
        TKV* c = pool.ptr(layer, page, is_k ? 0 : 1, kvh, pos & (pool.page_tokens - 1));
        c[i] = a;
        c[i + half] = b;
    }
}

// The same for wide passes: a warp per (row, head), eight heads per block, the per-head sum of squares by warp
// shuffles (head_dim up to 256: a lane holds up to four rotation pairs).
template <typename TA, typename TKV>
__global__ void __launch_bounds__(256) qk_rope_kv_rows_kernel(const float* __restrict__ qkv, PassView pv, const float* __restrict__ q_gain,
                                       const float* __restrict__ k_gain, const float* __restrict__ rope_cos,
                                       const float* __restrict__ rope_sin, TA* __restrict__ q_out, TA* __restrict__ q_lo,
                                       TKV* __restrict__ k_rows, TKV* __restrict__ v_rows, KvPool<TKV> pool, int layer, int Hq,
                                       int Hkv, int hd, float eps, int qk_norm) {
    const int r = blockIdx.x, head = blockIdx.y * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (head >= Hq + 2 * Hkv) return;
    const int half = hd >> 1;
    const float* src = qkv + (size_t)r * (Hq + 2 * Hkv) * hd + (size_t)head * hd;
    float x1[4], x2[4];
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = lane + 32 * j;
        x1[j] = x2[j] = 0.f;
        if (i < half) {
            x1[j] = src[i];
            x2[j] = src[i + half];
            ss += x1[j] * x1[j] + x2[j] * x2[j];
        }
    }
    const bool is_q = head < Hq, is_k = !is_q && head < Hq + Hkv;
    const int pos = pv.row_pos[r];
    if (is_q || is_k) {
        float inv = 1.f;
        if (qk_norm) {
            ss = warp_sum(ss);
            const float m = ss / (float)hd + eps;
            inv = rsqrtf(m);
            inv = inv * (1.5f - 0.5f * m * inv * inv);
        }
        const float* g = is_q ? q_gain : k_gain;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = lane + 32 * j;
            if (i < half) {
                float a = x1[j], b = x2[j];
                if (qk_norm) {
                    a = a * inv * g[i];
                    b = b * inv * g[i + half];
                }
                const float c = rope_cos[(size_t)pos * half + i], s = rope_sin[(size_t)pos * half + i];
                x1[j] = a * c - b * s;
                x2[j] = b * c + a * s;
            }
        }
    }
    if (is_q) {
        const size_t o = ((size_t)r * Hq + head) * hd;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = lane + 32 * j;
            if (i < half) {
                store_two_term(q_out, q_lo, o + i, x1[j]);
                store_two_term(q_out, q_lo, o + i + half, x2[j]);
            }
        }
        return;
    }
    const int kvh = is_k ? head - Hq : head - Hq - Hkv;
    TKV* dst = (is_k ? k_rows : v_rows) + ((size_t)r * Hkv + kvh) * hd;
    TKV* cache = nullptr;
    if (pv.row_flags[r] & ROW_WRITE_KV) {
        const int page = pv.seq_pages[(size_t)pv.row_seq[r] * pv.max_pages + (pos >> pool.page_shift)];
        cache = pool.ptr(layer, page, is_k ? 0 : 1, kvh, pos & (pool.page_tokens - 1));
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int i = lane + 32 * j;
        if (i < half) {
            const TKV a = from_f32<TKV>(x1[j]), b = from_f32<TKV>(x2[j]);
            dst[i] = a;
            dst[i + half] = b;
            if (cache) {
                cache[i] = a;
                cache[i + half] = b;
            }
        }
    }
}

// Two-part attention, plain form: one warp per (row, query head).  Part 1: all
// cached tokens [0, n_ctx) of the row's sequence, read from the pages.  Part 2:
// the rows of this pass the row's bitmask allows, read from the pass's K/V rows.
// Online softmax in fp32; the output is normalised at the end.
template <typename TA, typename TKV, int HD>
__global__ void attention_simt_kernel(const TA* __restrict__ q, const TKV* __restrict__ k_rows,
                                      const TKV* __restrict__ v_rows, PassView pv, KvPool<TKV> pool, int layer, int Hq,
                                      int Hkv, TA* __restrict__ out, float scale) {
    constexpr int E = HD / 32;
    int lane = threadIdx.x & 31;
    int wid = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (wid >= pv.n_rows * Hq) return;
    int r = wid / Hq, hq = wid % Hq;
    int kvh = hq / (Hq / Hkv);
    int sq = pv.row_seq[r];
    float qv[E], acc[E];
    const TA* qp = q + ((size_t)r * Hq + hq) * HD;
#pragma unroll
    for (int e = 0; e < E; ++e) {
        qv[e] = to_f32(qp[lane + 32 * e]) * scale;
        acc[e] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    auto visit = [&](const TKV* kp, const TKV* vp) {
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) s += qv[e] * to_f32(kp[lane + 32 * e]);
        s = warp_sum(s);
        float mn = fmaxf(m, s);
        float corr = expf(m - mn), p = expf(s - mn);
        l = l * corr + p;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = acc[e] * corr + p * to_f32(vp[lane + 32 * e]);
        m = mn;
    };
    int n_ctx = pv.seq_nctx[sq];
    const int* pages = pv.seq_pages + (size_t)sq * pv.max_pages;
    for (int t = 0; t < n_ctx; ++t) {
        int page = pages[t >> pool.page_shift], o = t & (pool.page_tokens - 1);
        visit(pool.ptr(layer, page, 0, kvh, o), pool.ptr(layer, page, 1, kvh, o));
    }
    unsigned long long mask = pv.row_mask[r];
    int r0 = pv.seq_row0[sq];
    while (mask) {
        int b = __ffsll((long long)mask) - 1;
        mask &= mask - 1;
        size_t o = ((size_t)(r0 + b) * Hkv + kvh) * HD;
        visit(k_rows + o, v_rows + o);
    }
    float inv = 1.f / l;
    TA* op = out + ((size_t)r * Hq + hq) * HD;
#pragma unroll
    for (int e = 0; e < E; ++e) op[lane + 32 * e] = from_f32<TA>(acc[e] * inv);
}

// act[m, i] = silu(gu[m, i]) * gu[m, f + i]
template <typename TA>
__global__ void swiglu_kernel(const float* __restrict__ gu, TA* __restrict__ act, TA* __restrict__ act_lo, int M, int f) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if ((f & 3) == 0) {       // four consecutive columns per thread; the grid has a thread per element, the rest leave
        if (idx >= (size_t)M * (f / 4)) return;
        const size_t m = idx / (f / 4), i = (idx % (f / 4)) * 4;
        const float4 g = *reinterpret_cast<const float4*>(gu + m * 2 * f + i), u = *reinterpret_cast<const float4*>(gu + m * 2 * f + f + i);
        store_two_term_x4(act, act_lo, m * f + i, g.x / (1.f + expf(-g.x)) * u.x, g.y / (1.f + expf(-g.y)) * u.y,
                          g.z / (1.f + expf(-g.z)) * u.z, g.w / (1.f + expf(-g.w)) * u.w);
        return;
    }
    if (idx >= (size_t)M * f) return;
    size_t m = idx / f, i = idx % f;
    float g = gu[m * 2 * f + i], u = gu[m * 2 * f + f + i];
    store_two_term(act, act_lo, idx, g / (1.f + expf(-g)) * u);
}

// ---- mixture of experts, plain form -------------------------------------------------------------

// Per row: softmax over the router logits, top_k largest (ties -> lowest id),
// gates renormalised over the kept experts.  One warp per row.
static __global__ void moe_topk_kernel(const float* __restrict__ logits, int M, int E, int top_k, int* __restrict__ ids,
                                float* __restrict__ gates) {
    int r = blockIdx.x, lane = threadIdx.x;
    const float* x = logits + (size_t)r * E;
    float mx = -INFINITY;
    for (int e = lane; e < E; e += 32) mx = fmaxf(mx, x[e]);
    mx = warp_max(mx);
    float sum = 0.f;
    for (int e = lane; e < E; e += 32) sum += expf(x[e] - mx);
    sum = warp_sum(sum);
    // top-k by repeated arg-max on the logits (softmax is monotone); taken ids are skipped
    float kept = 0.f;
    float last_v = INFINITY;
    int last_i = -1;
    for (int k = 0; k < top_k; ++k) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int e = lane; e < E; e += 32) {
            float v = x[e];
            // candidates strictly after (last_v, last_i) in the order (value desc, id asc)
            bool after = (v < last_v) || (v == last_v && e > last_i);
            if (after && (v > bv || (v == bv && e < bi))) {
                bv = v;
                bi = e;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) {
                bv = ov;
                bi = oi;
            }
        }
        last_v = bv;
        last_i = bi;
        float p = expf(bv - mx) / sum;
        kept += p;
        if (lane == 0) {
            ids[(size_t)r * top_k + k] = bi;
            gates[(size_t)r * top_k + k] = p;
        }
    }
    __syncwarp();
    if (lane < top_k) gates[(size_t)r * top_k + lane] /= kept;
}

// Expert gate/up: for pair p = (row, slot) with expert e = ids[p]:
//   out[p, n] = sum_k X[row, k] * W[e, n, k]   for both w_gate (n < f) and w_up (n >= f).
template <typename TW, typename TX>
__global__ void moe_gateup_kernel(const TX* __restrict__ X, const TW* __restrict__ Wg, const TW* __restrict__ Wu,
                                  const int* __restrict__ ids, float* __restrict__ out, int top_k, int f, int d) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= 2 * f) return;
    int p = blockIdx.y, row = p / top_k, e = ids[p];
    const TW* w = (warp < f ? Wg : Wu) + ((size_t)e * f + (warp < f ? warp : warp - f)) * d;
    const TX* x = X + (size_t)row * d;
    float acc = 0.f;
    for (int k = lane; k < d; k += 32) acc += to_f32(w[k]) * to_f32(x[k]);
    acc = warp_sum(acc);
    if (lane == 0) out[(size_t)p * 2 * f + warp] = acc;
}

// Expert down projection per pair: out[p, n] = sum_k act[p, k] * Wd[e, n, k].
template <typename TW, typename TX>
__global__ void moe_down_kernel(const TX* __restrict__ act, const TW* __restrict__ Wd, const int* __restrict__ ids,
                                float* __restrict__ out, int f, int d) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= d) return;
    int p = blockIdx.y, e = ids[p];
    const TW* w = Wd + ((size_t)e * d + warp) * f;
    const TX* x = act + (size_t)p * f;
    float acc = 0.f;
    for (int k = lane; k < f; k += 32) acc += to_f32(w[k]) * to_f32(x[k]);
    acc = warp_sum(acc);
    if (lane == 0) out[(size_t)p * d + warp] = acc;
}

// h[row, :] += sum_slot gates[row, slot] * pair_out[row*top_k + slot, :]  (fixed slot order)
static __global__ void moe_combine_kernel(const float* __restrict__ pair_out, const float* __restrict__ gates,
                                   float* __restrict__ h, int M, int top_k, int d) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)M * d) return;
    size_t row = idx / d, c = idx % d;
    float acc = 0.f;
    for (int s = 0; s < top_k; ++s) acc += gates[row * top_k + s] * pair_out[(row * top_k + s) * d + c];
    h[idx] += acc;
}

// The bounded-wait pattern of the tensor-core kernels in isolation (test tap): poll a word that is
// expected to reach `target`; after `limit` polls raise the status word and return normally.
static __global__ void bounded_wait_probe_kernel(const unsigned* __restrict__ word, unsigned target, unsigned limit, int* status) {
    for (unsigned it = 0; it < limit; ++it) {
        unsigned v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
        if (v >= target) return;
        __nanosleep(100);
    }
    atomicCAS(status, 0, 10);
}

// Copy K/V of cache positions [0, n) of one layer to fp32 (test tap).
template <typename TKV>
__global__ void kv_export_kernel(KvPool<TKV> pool, const int* __restrict__ pages, int layer, int n, float* __restrict__ k,
                                 float* __restrict__ v) {
    int t = blockIdx.x, head = blockIdx.y;
    int page = pages[t >> pool.page_shift], o = t & (pool.page_tokens - 1);
    const TKV* kp = pool.ptr(layer, page, 0, head, o);
    const TKV* vp = pool.ptr(layer, page, 1, head, o);
    size_t dst = ((size_t)t * pool.n_kv_heads + head) * pool.head_dim;
    for (int i = threadIdx.x; i < pool.head_dim; i += blockDim.x) {
        k[dst + i] = to_f32(kp[i]);
        v[dst + i] = to_f32(vp[i]);
    }
}

}  // namespace s2d2
