// One persistent kernel per network pass (draft pass, verifier pass or prefill chunk) for bf16
// dense models with at most 64 rows.
//
// At batch 1 a pass multiplies 4..64 token rows by every weight matrix once: the weights are the
// only large stream (15 GB for the 8B-class shape) and each single operation lasts 5-30 us at HBM
// rate, so a kernel per operation spends more time starting and draining than streaming.  Here
// one cooperative grid of one CTA per SM runs the whole pass and the weight stream never stops:
//
//   warp 0    W producer: walks the static list of every GEMM of the pass (QKV, O, gate/up, down
//             per layer, then the LM head) and TMA-loads this CTA's 128-row x 64-column weight
//             tiles into a ring of stages, limited only by ring space.  It does not wait for any
//             other operation, so while the CTA sits in a grid barrier, an element-wise phase or
//             attention, the next GEMM's weights are already arriving.
//   warp 1    X producer: TMA-loads the matching 64-column slices of the token rows into the same
//             stages once the grid barrier that publishes them has been passed.
//   warp 2    issues tcgen05.mma (weight tile = M operand, token rows = N operand, fp32
//             accumulators double-buffered in tensor memory).
//   warps 4-7 everything else: drain accumulators to split-K partials, then between grid barriers
//             the element-wise phases (partial sums + RMSNorm scale, q/k norm + RoPE + K/V write,
//             residual adds, SwiGLU, logits), the two-mask attention items and their combine.
//
// Work split of a GEMM (stream-K): its (weight tile, k-block) units, tile-major, are cut into
// gridDim equal contiguous ranges; a CTA's range yields one partial accumulator per tile it
// touches.  The phase after the barrier sums the partials of a tile in CTA order, so results do
// not depend on timing.  RMSNorm is folded around the GEMM: the GEMM input is bf16(h * gain) and
// the per-row 1/rms (from per-tile sums of squares written by the phase that produced h) scales
// the summed output.
//
// Every wait (mbarrier, grid barrier) is bounded; on time-out the kernel raises the status word,
// which makes every other wait in the grid give up too, and leaves normally.
#pragma once
#include <cuda.h>

#include "attention_tc.cuh"
#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace s2d2 {
namespace pp {

constexpr int THREADS = 256;
constexpr int CTHREADS = 128;        // compute warps 4..7
constexpr int BAR_COMPUTE = 1;       // named barrier of the compute warps
constexpr int ACC_STRIDE = 64;       // tensor-memory columns per accumulator buffer
constexpr int MAX_T = 64;            // most token rows of a pass
constexpr int W_TILE_BYTES = tc::BLOCK_N * 128;
constexpr uint32_t SPIN_LIMIT = 1u << 24;

struct LayerGains {
    const float *attn_norm, *ffn_norm, *q_norm, *k_norm;
};

struct PassParams {
    int n_layers, d, Hq, Hkv, hd, f, V;
    int qk_norm;
    float eps, logit_scale;
    PassView pv;
    int M, T, n_logit;
    const bf16* embed;
    const LayerGains* gains;
    const float* final_norm;
    float* h;                 // [M, d] residual stream
    bf16 *xn, *q, *k_rows, *v_rows, *attn, *act;
    float* ws;                // split-K partials [grid][max_segs][T][128]
    int max_segs;
    float *ssq_a, *ssq_b;     // per-tile sums of squares of h rows [d/128][MAX_T]
    float* logits;            // [n_logit, V]
    const float *rope_cos, *rope_sin;
    KvPool<bf16> pool;
    const CUtensorMap* maps;  // device array: weights [n_layers*4 + 1], then the entries below
    int map_xn, map_attn, map_act, map_kv;
    att::AttnParams ap;       // attention geometry of this pass (layer filled in per layer)
    unsigned* barrier;        // grid barrier counter, zero at launch
    int* status;
    int S;                    // ring stages
};

__host__ __device__ inline size_t stage_bytes(int T) { return (size_t)W_TILE_BYTES + (size_t)T * 128; }
__host__ __device__ inline size_t misc_bytes() { return 2048; }
__host__ __device__ inline size_t smem_bytes(int T, int S, int hd) {
    return 1024 + (size_t)S * stage_bytes(T) + att::attn_tiles_bytes(hd) + misc_bytes();
}

struct GemmShape {
    int n_tiles, kbt, map_w, map_x;
    long long U;
};
// kind 0: QKV, 1: O, 2: gate/up, 3: down (layer l), 4: LM head.
__device__ __forceinline__ GemmShape gemm_shape(const PassParams& p, int l, int kind) {
    int N, K, mx;
    switch (kind) {
        case 0: N = (p.Hq + 2 * p.Hkv) * p.hd; K = p.d; mx = p.map_xn; break;
        case 1: N = p.d; K = p.Hq * p.hd; mx = p.map_attn; break;
        case 2: N = 2 * p.f; K = p.d; mx = p.map_xn; break;
        case 3: N = p.d; K = p.f; mx = p.map_act; break;
        default: N = p.V; K = p.d; mx = p.map_xn; break;
    }
    GemmShape g;
    g.n_tiles = (N + tc::BLOCK_N - 1) / tc::BLOCK_N;
    g.kbt = K / tc::BLOCK_K;
    g.map_w = kind == 4 ? p.n_layers * 4 : l * 4 + kind;
    g.map_x = mx;
    g.U = (long long)g.n_tiles * g.kbt;
    return g;
}
// Grid barriers passed before the inputs of a GEMM are published.
__device__ __forceinline__ unsigned gemm_epoch(const PassParams& p, int l, int kind) {
    const unsigned off[5] = {1u, 5u, 7u, 9u, 1u};
    return off[kind] + 10u * (unsigned)(kind == 4 ? p.n_layers : l);
}
__device__ __forceinline__ long long unit_begin(long long U, int c, int G) { return U * c / G; }

// Calls f(tile, kb0, kb1, local_segment) for the segments of this CTA's unit range.
template <class F>
__device__ __forceinline__ void for_each_segment(const GemmShape& g, int cta, int G, F f) {
    long long u = unit_begin(g.U, cta, G), u1 = unit_begin(g.U, cta + 1, G);
    const int first_tile = (int)(u / g.kbt);
    while (u < u1) {
        int tile = (int)(u / g.kbt);
        int kb0 = (int)(u - (long long)tile * g.kbt);
        int kb1 = (int)min((long long)g.kbt, kb0 + (u1 - u));
        if (!f(tile, kb0, kb1, tile - first_tile)) return;
        u += kb1 - kb0;
    }
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc::smem_u32(bar)) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait until the grid barrier counter reaches `target`; gives up early when any CTA has
// raised the status word.
__device__ __forceinline__ bool wait_counter(const PassParams& p, unsigned target, volatile int* abort_flag) {
    for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
        if (ld_acquire(p.barrier) >= target) return true;
        if ((it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) return false;
        __nanosleep(20);
    }
    return false;
}

// Sum of the split-K partials of (tile, row m, column n) in CTA order.
struct TileParts {
    int c_lo, c_hi;
};
__device__ __forceinline__ TileParts tile_parts(const GemmShape& g, int tile, int G) {
    long long ua = (long long)tile * g.kbt, ub = ua + g.kbt - 1;
    TileParts t;
    int c = (int)(ua * G / g.U);
    while (unit_begin(g.U, c + 1, G) <= ua) ++c;
    t.c_lo = c;
    c = (int)(ub * G / g.U);
    while (unit_begin(g.U, c + 1, G) <= ub) ++c;
    t.c_hi = c;
    return t;
}
constexpr int RC = 8;   // rows handled together so that their loads are in flight at once
// acc[j] = sum of the split-K partials of (tile, row rows[j], column n), parts in CTA order.
__device__ __forceinline__ void tile_sum_rows(const PassParams& p, const GemmShape& g, const TileParts& tp, int tile, int G,
                                              const int (&rows)[RC], int n, float (&acc)[RC]) {
#pragma unroll
    for (int j = 0; j < RC; ++j) acc[j] = 0.f;
    for (int c = tp.c_lo; c <= tp.c_hi; ++c) {
        long long b0 = unit_begin(g.U, c, G), b1 = unit_begin(g.U, c + 1, G);
        if (b1 <= b0) continue;
        int local = tile - (int)(b0 / g.kbt);
        const float* part = p.ws + ((size_t)c * p.max_segs + local) * (size_t)p.T * tc::BLOCK_N + n;
        float v[RC];
#pragma unroll
        for (int j = 0; j < RC; ++j) v[j] = __ldcg(part + (size_t)rows[j] * tc::BLOCK_N);
#pragma unroll
        for (int j = 0; j < RC; ++j) acc[j] += v[j];
    }
}
// rows m0 .. m0+RC-1, clamped to the last valid row (duplicates are computed and dropped)
__device__ __forceinline__ void chunk_rows(int m0, int M, int (&rows)[RC]) {
#pragma unroll
    for (int j = 0; j < RC; ++j) rows[j] = min(m0 + j, M - 1);
}

template <int HD>
__global__ void __launch_bounds__(THREADS, 1) pass_kernel(const __grid_constant__ PassParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int S = p.S, T = p.T, G = gridDim.x, cta = blockIdx.x;
    const size_t sbytes = stage_bytes(T);
    uint8_t* ring = base;
    uint8_t* attn_s = ring + (size_t)S * sbytes;
    uint8_t* misc = attn_s + att::attn_tiles_bytes(HD);
    uint64_t* full = (uint64_t*)misc;
    uint64_t* empty = full + S;
    uint64_t* acc_full = empty + S;
    uint64_t* acc_empty = acc_full + 2;
    uint64_t* kv_full = acc_empty + 2;
    uint32_t* tmem_slot = (uint32_t*)(kv_full + att::STAGES);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    volatile int* w_issued = abort_flag + 1;
    volatile int* x_issued = w_issued + 1;
    volatile int* consumed = x_issued + 1;
    float* red = (float*)(misc + 512);        // [4][MAX_T]
    float* inv_s = red + 4 * MAX_T;           // [MAX_T]
    float* stage_f = (float*)attn_s;          // [MAX_T][128] staging of the QKV phase (aliases the attention tiles)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_gemms = p.n_layers * 4 + (p.n_logit > 0 ? 1 : 0);

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc::mbar_init(&full[s], 2);
            tc::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            tc::mbar_init(&acc_full[b], 1);
            tc::mbar_init(&acc_empty[b], 4);
        }
        for (int s = 0; s < att::STAGES; ++s) tc::mbar_init(&kv_full[s], 1);
        *abort_flag = 0;
        *w_issued = 0;
        *x_issued = 0;
        *consumed = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        tc::tmem_alloc(tmem_slot, 2 * ACC_STRIDE);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- W producer: free-running over every GEMM of the pass ----------------
            uint64_t policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
            uint32_t i = 0;
            bool ok = true;
            for (int gi = 0; gi < n_gemms && ok; ++gi) {
                const int l = gi >> 2, kind = gi < p.n_layers * 4 ? (gi & 3) : 4;
                const GemmShape g = gemm_shape(p, l, kind);
                const CUtensorMap* mw = p.maps + g.map_w;
                for_each_segment(g, cta, G, [&](int tile, int kb0, int kb1, int) {
                    for (int kb = kb0; kb < kb1; ++kb, ++i) {
                        int s = (int)(i % (uint32_t)S);
                        if (i >= (uint32_t)S && !tc::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) return ok = false;
                        if (*abort_flag) return ok = false;
                        tc::mbar_expect_tx(&full[s], W_TILE_BYTES);
                        tc::tma_load_2d_hint(ring + s * sbytes, mw, kb * tc::BLOCK_K, tile * tc::BLOCK_N, &full[s], policy);
                        *w_issued = (int)i + 1;
                    }
                    return true;
                });
            }
            if (!ok) {
                atomicCAS(p.status, 0, 7);
                *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------- X producer: token-row slices, after their grid barrier ----------------
            uint32_t i = 0;
            bool ok = true;
            for (int gi = 0; gi < n_gemms && ok; ++gi) {
                const int l = gi >> 2, kind = gi < p.n_layers * 4 ? (gi & 3) : 4;
                const GemmShape g = gemm_shape(p, l, kind);
                const CUtensorMap* mx = p.maps + g.map_x;
                if (unit_begin(g.U, cta + 1, G) > unit_begin(g.U, cta, G)) {
                    if (!wait_counter(p, gemm_epoch(p, l, kind) * (unsigned)G, abort_flag)) {
                        ok = false;
                        break;
                    }
                    asm volatile("fence.proxy.async;" ::: "memory");
                }
                for_each_segment(g, cta, G, [&](int, int kb0, int kb1, int) {
                    for (int kb = kb0; kb < kb1; ++kb, ++i) {
                        int s = (int)(i % (uint32_t)S);
                        if (i >= (uint32_t)S && !tc::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) return ok = false;
                        if (*abort_flag) return ok = false;
                        tc::mbar_expect_tx(&full[s], (uint32_t)T * 128u);
                        tc::tma_load_2d(ring + s * sbytes + W_TILE_BYTES, mx, kb * tc::BLOCK_K, 0, &full[s]);
                        *x_issued = (int)i + 1;
                    }
                    return true;
                });
            }
            if (!ok) {
                atomicCAS(p.status, 0, 3);
                *abort_flag = 1;
            }
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = tc::instr_desc_bf16(T);
            uint32_t i = 0, seg = 0;
            bool ok = true;
            for (int gi = 0; gi < n_gemms && ok; ++gi) {
                const int l = gi >> 2, kind = gi < p.n_layers * 4 ? (gi & 3) : 4;
                const GemmShape g = gemm_shape(p, l, kind);
                for_each_segment(g, cta, G, [&](int, int kb0, int kb1, int) {
                    const uint32_t b = seg & 1u;
                    if (seg >= 2 && !tc::mbar_wait(&acc_empty[b], ((seg >> 1) - 1) & 1, abort_flag)) return ok = false;
                    tc::tc_fence_after();
                    const uint32_t d_tmem = tmem_base + b * ACC_STRIDE;
                    for (int kb = kb0; kb < kb1; ++kb, ++i) {
                        int s = (int)(i % (uint32_t)S);
                        if (!tc::mbar_wait(&full[s], (i / S) & 1, abort_flag)) return ok = false;
                        tc::tc_fence_after();
                        uint32_t a_addr = tc::smem_u32(ring + s * sbytes);
                        uint64_t a_desc = tc::smem_desc_sw128(a_addr), b_desc = tc::smem_desc_sw128(a_addr + W_TILE_BYTES);
#pragma unroll
                        for (int k = 0; k < tc::BLOCK_K / tc::UMMA_K; ++k)
                            tc::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                        tc::umma_commit(&empty[s]);
                        *consumed = (int)i + 1;
                    }
                    tc::umma_commit(&acc_full[b]);
                    ++seg;
                    return true;
                });
            }
            if (!ok) {
                atomicCAS(p.status, 0, 4);
                *abort_flag = 1;
            }
        }
    } else if (warp >= 4) {
        // ---------------- compute warps ----------------
        const int tid = threadIdx.x - (THREADS - CTHREADS), cw = tid >> 5;
        unsigned epoch = 0;
        uint32_t seg = 0, kv_ring = 0;
        bool ok = true;
        const int M = p.M, d = p.d;
        const int d_tiles = d / tc::BLOCK_N;

        auto grid_sync = [&]() {
            ++epoch;
            asm volatile("fence.proxy.async;" ::: "memory");
            __threadfence();
            att::group_sync(BAR_COMPUTE, CTHREADS);
            if (tid == 0) {
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
                if (!wait_counter(p, epoch * (unsigned)G, abort_flag)) {
                    atomicCAS(p.status, 0, 5);
                    *abort_flag = 1;
                }
                __threadfence();
            }
            att::group_sync(BAR_COMPUTE, CTHREADS);
            asm volatile("fence.proxy.async;" ::: "memory");
            if (*abort_flag) ok = false;
        };
        // accumulators of this CTA's segments of one GEMM -> split-K partials
        auto drain = [&](int l, int kind) {
            const GemmShape g = gemm_shape(p, l, kind);
            for_each_segment(g, cta, G, [&](int, int, int, int local) {
                const uint32_t b = seg & 1u;
                if (!tc::mbar_wait(&acc_full[b], (seg >> 1) & 1, abort_flag)) return ok = false;
                tc::tc_fence_after();
                float* mine = p.ws + ((size_t)cta * p.max_segs + local) * (size_t)T * tc::BLOCK_N + tid;
                const uint32_t taddr = tmem_base + ((uint32_t)(cw * 32) << 16) + b * ACC_STRIDE;
                for (int c0 = 0; c0 < T; c0 += 16) {
                    float v[16];
                    tc::tmem_ld16(taddr + c0, v);
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < M) mine[(size_t)(c0 + j) * tc::BLOCK_N] = v[j];
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[b]);
                ++seg;
                return true;
            });
            if (!ok) {
                atomicCAS(p.status, 0, 6);
                *abort_flag = 1;
            }
        };
        // 1/rms of every row from the per-tile sums of squares
        auto compute_inv = [&](const float* ssq) {
            if (tid < M) {
                float s = 0.f;
#pragma unroll 8
                for (int t = 0; t < d_tiles; ++t) s += __ldcg(ssq + (size_t)t * MAX_T + tid);
                inv_s[tid] = 1.0f / sqrtf(s / (float)d + p.eps);
            }
            att::group_sync(BAR_COMPUTE, CTHREADS);
        };
        // h tile update shared by the embedding and the two residual phases: value(rows, x) gives the
        // new h of RC rows of this thread's column; writes h, the next GEMM's input bf16(h * gain)
        // and the tile's per-row sums of squares
        auto h_tile = [&](int t, const float* gain, float* ssq, auto&& value) {
            const int col = t * tc::BLOCK_N + tid;
            const float gn = gain[col];
            for (int m0 = 0; m0 < M; m0 += RC) {
                int rows[RC];
                chunk_rows(m0, M, rows);
                float x[RC];
                value(rows, col, x);
#pragma unroll
                for (int j = 0; j < RC; ++j) {
                    if (m0 + j < M) {
                        p.h[(size_t)rows[j] * d + col] = x[j];
                        p.xn[(size_t)rows[j] * d + col] = __float2bfloat16_rn(x[j] * gn);
                    }
                    float sq = warp_sum(x[j] * x[j]);
                    if (lane == 0 && m0 + j < M) red[cw * MAX_T + m0 + j] = sq;
                }
            }
            att::group_sync(BAR_COMPUTE, CTHREADS);
            if (tid < M) ssq[(size_t)t * MAX_T + tid] = red[tid] + red[MAX_T + tid] + red[2 * MAX_T + tid] + red[3 * MAX_T + tid];
            att::group_sync(BAR_COMPUTE, CTHREADS);
        };
        auto residual_phase = [&](int l, int kind, const float* gain, float* ssq) {
            const GemmShape g = gemm_shape(p, l, kind);
            for (int t = cta; t < d_tiles; t += G) {
                const TileParts tp = tile_parts(g, t, G);
                h_tile(t, gain, ssq, [&](const int (&rows)[RC], int col, float (&x)[RC]) {
                    float hv[RC];
#pragma unroll
                    for (int j = 0; j < RC; ++j) hv[j] = __ldcg(p.h + (size_t)rows[j] * d + col);
                    tile_sum_rows(p, g, tp, t, G, rows, tid, x);
#pragma unroll
                    for (int j = 0; j < RC; ++j) x[j] += hv[j];
                });
            }
        };

        // ---- embedding ----
        for (int t = cta; t < d_tiles; t += G)
            h_tile(t, p.gains[0].attn_norm, p.ssq_a, [&](const int (&rows)[RC], int col, float (&x)[RC]) {
#pragma unroll
                for (int j = 0; j < RC; ++j) x[j] = __bfloat162float(p.embed[(size_t)p.pv.row_token[rows[j]] * d + col]);
            });
        grid_sync();

        for (int l = 0; l < p.n_layers && ok; ++l) {
            const LayerGains lg = p.gains[l];
            // ---- QKV GEMM ----
            drain(l, 0);
            if (!ok) break;
            grid_sync();
            if (!ok) break;
            // ---- 1/rms, q/k norm, RoPE, K/V write ----
            compute_inv(p.ssq_a);
            {
                const GemmShape g = gemm_shape(p, l, 0);
                constexpr int HIT = tc::BLOCK_N / HD;      // heads per tile
                constexpr int E = HD / 32, half = HD / 2;
                for (int t = cta; t < g.n_tiles; t += G) {
                    const TileParts tp = tile_parts(g, t, G);
                    for (int m0 = 0; m0 < M; m0 += RC) {
                        int rows[RC];
                        chunk_rows(m0, M, rows);
                        float x[RC];
                        tile_sum_rows(p, g, tp, t, G, rows, tid, x);
#pragma unroll
                        for (int j = 0; j < RC; ++j)
                            if (m0 + j < M) stage_f[(m0 + j) * tc::BLOCK_N + tid] = inv_s[m0 + j] * x[j];
                    }
                    att::group_sync(BAR_COMPUTE, CTHREADS);
                    for (int pair = cw; pair < M * HIT; pair += 4) {
                        const int m = pair / HIT, head = t * HIT + pair % HIT;
                        const float* src = stage_f + m * tc::BLOCK_N + (pair % HIT) * HD;
                        float x[E];
#pragma unroll
                        for (int e = 0; e < E; ++e) x[e] = src[lane + 32 * e];
                        const bool is_q = head < p.Hq, is_k = !is_q && head < p.Hq + p.Hkv;
                        const int pos = p.pv.row_pos[m];
                        if (is_q || is_k) {
                            if (p.qk_norm) {
                                float ss = 0.f;
#pragma unroll
                                for (int e = 0; e < E; ++e) ss += x[e] * x[e];
                                ss = warp_sum(ss);
                                const float inv = 1.0f / sqrtf(ss / (float)HD + p.eps);
                                const float* gq = is_q ? lg.q_norm : lg.k_norm;
#pragma unroll
                                for (int e = 0; e < E; ++e) x[e] = x[e] * inv * gq[lane + 32 * e];
                            }
#pragma unroll
                            for (int e = 0; e < E / 2; ++e) {
                                const int i = lane + 32 * e;
                                const float c = p.rope_cos[(size_t)pos * half + i], s = p.rope_sin[(size_t)pos * half + i];
                                const float x1 = x[e], x2 = x[e + E / 2];
                                x[e] = x1 * c - x2 * s;
                                x[e + E / 2] = x2 * c + x1 * s;
                            }
                        }
                        if (is_q) {
                            bf16* dst = p.q + ((size_t)m * p.Hq + head) * HD;
#pragma unroll
                            for (int e = 0; e < E; ++e) dst[lane + 32 * e] = __float2bfloat16_rn(x[e]);
                        } else {
                            const int kvh = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
                            bf16* dst = (is_k ? p.k_rows : p.v_rows) + ((size_t)m * p.Hkv + kvh) * HD;
                            bf16* cdst = nullptr;
                            if (p.pv.row_flags[m] & ROW_WRITE_KV) {
                                const int sq = p.pv.row_seq[m];
                                const int page = p.pv.seq_pages[(size_t)sq * p.pv.max_pages + (pos >> p.pool.page_shift)];
                                cdst = p.pool.ptr(l, page, is_k ? 0 : 1, kvh, pos & (p.pool.page_tokens - 1));
                            }
#pragma unroll
                            for (int e = 0; e < E; ++e) {
                                const bf16 v = __float2bfloat16_rn(x[e]);
                                dst[lane + 32 * e] = v;
                                if (cdst) cdst[lane + 32 * e] = v;
                            }
                        }
                    }
                    att::group_sync(BAR_COMPUTE, CTHREADS);
                }
            }
            grid_sync();
            if (!ok) break;
            // ---- attention items ----
            {
                att::AttnParams ap = p.ap;
                ap.layer = l;
                const int n_splits = ap.n_cache_splits + 1;
                const int total = ap.pv.n_seqs * ap.Hkv * ap.n_qtiles * n_splits;
                // plain stores of the previous phases into the tile region precede TMA writes
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                att::group_sync(BAR_COMPUTE, CTHREADS);
                for (int idx = cta; idx < total && ok; idx += G) {
                    const int split = idx % n_splits, r = idx / n_splits;
                    if (!att::attn_item<HD>(p.maps + p.map_kv, ap, split, r % ap.n_qtiles, r / ap.n_qtiles, attn_s, kv_full,
                                            kv_ring, tid, BAR_COMPUTE)) {
                        ok = false;
                        *abort_flag = 1;
                    }
                }
                if (!ok) break;
                grid_sync();
                if (!ok) break;
                // ---- combine the key splits of every (row, query head) ----
                for (int pair = cta * 4 + cw; pair < M * p.Hq; pair += G * 4) {
                    const int r = pair / p.Hq, hq = pair % p.Hq;
                    const int seq = p.pv.row_seq[r], kvh = hq / ap.group;
                    const int qv = (r - p.pv.seq_row0[seq]) * ap.group + hq % ap.group;
                    const int qt = qv / att::QT, qi = qv % att::QT;
                    const int n_ctx = p.pv.seq_nctx[seq];
                    const int n_pages = (n_ctx + ap.page_tokens - 1) >> ap.page_shift;
                    const size_t item0 = ((size_t)(seq * ap.Hkv + kvh) * ap.n_qtiles + qt) * n_splits;
                    // lanes take the splits for the maxima and weights, then the columns for the sums
                    float mx = -INFINITY;
                    for (int s0 = 0; s0 < n_splits; s0 += 32) {
                        const int s = s0 + lane;
                        const bool used = s < n_splits && (s == ap.n_cache_splits || s * ap.pages_per_split < n_pages);
                        const float ms = used ? __ldcg(ap.part_ml + (item0 + s) * att::QT * 2 + qi * 2) : -INFINITY;
                        mx = fmaxf(mx, warp_max(ms));
                    }
                    float acc[HD / 32], lsum = 0.f;
#pragma unroll
                    for (int e = 0; e < HD / 32; ++e) acc[e] = 0.f;
                    for (int s0 = 0; s0 < n_splits; s0 += 32) {
                        const int s = s0 + lane;
                        const bool used = s < n_splits && (s == ap.n_cache_splits || s * ap.pages_per_split < n_pages);
                        float w_l = 0.f, l_l = 0.f;
                        if (used) {
                            const float ms = __ldcg(ap.part_ml + (item0 + s) * att::QT * 2 + qi * 2);
                            if (ms != -INFINITY) {
                                w_l = exp2f(ms - mx);
                                l_l = __ldcg(ap.part_ml + (item0 + s) * att::QT * 2 + qi * 2 + 1);
                            }
                        }
                        const int cnt = min(32, n_splits - s0);
#pragma unroll 4
                        for (int k = 0; k < cnt; ++k) {
                            const float w = __shfl_sync(0xffffffffu, w_l, k);
                            lsum += w * __shfl_sync(0xffffffffu, l_l, k);
                            const float* po = ap.part_o + ((item0 + s0 + k) * att::QT + qi) * HD + lane;
#pragma unroll
                            for (int e = 0; e < HD / 32; ++e) {
                                const float v = w != 0.f ? __ldcg(po + 32 * e) : 0.f;
                                acc[e] += w * v;
                            }
                        }
                    }
#pragma unroll
                    for (int e = 0; e < HD / 32; ++e)
                        p.attn[((size_t)r * p.Hq + hq) * HD + lane + 32 * e] = __float2bfloat16_rn(acc[e] / lsum);
                }
            }
            grid_sync();
            if (!ok) break;
            // ---- O GEMM, residual ----
            drain(l, 1);
            if (!ok) break;
            grid_sync();
            if (!ok) break;
            residual_phase(l, 1, lg.ffn_norm, p.ssq_b);
            grid_sync();
            if (!ok) break;
            // ---- gate/up GEMM, SwiGLU ----
            drain(l, 2);
            if (!ok) break;
            grid_sync();
            if (!ok) break;
            compute_inv(p.ssq_b);
            {
                const GemmShape g = gemm_shape(p, l, 2);
                const int f_tiles = p.f / tc::BLOCK_N;
                for (int t = cta; t < f_tiles; t += G) {
                    const TileParts tg = tile_parts(g, t, G), tu = tile_parts(g, t + f_tiles, G);
                    for (int m0 = 0; m0 < M; m0 += RC) {
                        int rows[RC];
                        chunk_rows(m0, M, rows);
                        float gs[RC], us[RC];
                        tile_sum_rows(p, g, tg, t, G, rows, tid, gs);
                        tile_sum_rows(p, g, tu, t + f_tiles, G, rows, tid, us);
#pragma unroll
                        for (int j = 0; j < RC; ++j) {
                            if (m0 + j >= M) continue;
                            const float gv = inv_s[m0 + j] * gs[j], uv = inv_s[m0 + j] * us[j];
                            p.act[(size_t)(m0 + j) * p.f + t * tc::BLOCK_N + tid] = __float2bfloat16_rn(gv / (1.f + expf(-gv)) * uv);
                        }
                    }
                }
            }
            grid_sync();
            if (!ok) break;
            // ---- down GEMM, residual; prepares the next layer's (or the head's) input ----
            drain(l, 3);
            if (!ok) break;
            grid_sync();
            if (!ok) break;
            residual_phase(l, 3, l + 1 < p.n_layers ? p.gains[l + 1].attn_norm : p.final_norm, p.ssq_a);
            grid_sync();
        }
        if (ok && p.n_logit > 0) {
            // ---- LM head on the rows that need logits ----
            drain(p.n_layers, 4);
            if (ok) grid_sync();
            if (ok) {
                compute_inv(p.ssq_a);
                const GemmShape g = gemm_shape(p, p.n_layers, 4);
                for (int t = cta; t < g.n_tiles; t += G) {
                    const TileParts tp = tile_parts(g, t, G);
                    const int col = t * tc::BLOCK_N + tid;
                    for (int r0 = 0; r0 < p.n_logit; r0 += RC) {
                        int rows[RC];
#pragma unroll
                        for (int j = 0; j < RC; ++j) rows[j] = p.pv.logit_rows[min(r0 + j, p.n_logit - 1)];
                        float x[RC];
                        tile_sum_rows(p, g, tp, t, G, rows, tid, x);
#pragma unroll
                        for (int j = 0; j < RC; ++j)
                            if (r0 + j < p.n_logit && col < p.V)
                                p.logits[(size_t)(r0 + j) * p.V + col] = p.logit_scale * inv_s[rows[j]] * x[j];
                    }
                }
            }
        }
    }
    __syncwarp();
    tc::tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) {
        // every role has stopped: give the copies already issued into this CTA's shared memory a
        // bounded wait before the CTA leaves
        const int issued = min(*w_issued, *x_issued);
        for (int i = *consumed; i < issued; ++i) tc::mbar_wait(&full[i % S], (i / S) & 1);
        for (int k = 0; k < 1000; ++k) __nanosleep(1000);   // copies whose partner never came have no barrier to wait on
    }
    __syncthreads();
    if (warp == 2) tc::tmem_dealloc(tmem_base, 2 * ACC_STRIDE);
}

}  // namespace pp
}  // namespace s2d2
