// Skinny weight-streaming GEMM on the 5th-generation tensor cores (sm_100a).
//
//   Y[m, n] (+)= scale * sum_k X[m, k] * W[n, k]      X bf16 [M, K], W bf16 [N, K], Y fp32
//
// The decode step multiplies a few token rows (M = block x batch, 4..512) by every
// weight matrix of the network, so the weights are the stream and the tokens are
// the small operand.  The roles are therefore swapped with respect to a square
// GEMM: a tile of 128 weight rows is the MMA "M" operand (A, K-major, staged by
// TMA with the 128-byte swizzle), the token rows are the MMA "N" operand
// (B, K-major, T = 16..256 rows), and the fp32 accumulator D[128 x T] lives in
// tensor memory.  With two-term inputs (x = hi + lo, both bf16: 16 significant bits, which a
// network of 30 and more layers needs to keep its logits within 2e-2) the low halves are T more
// token rows of the same MMA and the epilogue adds the two accumulator halves.  One CTA owns one (weight tile, token tile, K split):
//   warp 0 / lane 0   TMA producer: W and X K-blocks of 64 into a ring of stages
//   warp 1 / lane 0   tcgen05.mma issuer, 4 MMAs (K = 16 each) per stage;
//                     tcgen05.commit frees the stage and finally signals the epilogue
//   warps 0..3        epilogue: tcgen05.ld of the 128 accumulator lanes, then either
//                     the final store or, with split K, a partial tile to a workspace;
//                     the last CTA to arrive for a tile (ticket counter) sums the
//                     partials in split order, so the result does not depend on timing.
// Two CTAs fit on one SM, so one CTA's set-up and epilogue overlap the other's stream.
// With more than about 128 token rows the kernel is bound by what enters shared memory, and most of
// that is the token block, re-read for every weight tile: a CTA then takes two weight sub-tiles
// (256 rows, one accumulator each) per token block.
// Every wait on an mbarrier is bounded; on time-out the kernel raises a status word
// that the host turns into S2D2_ERR_TIMEOUT, drains its copies and frees its TMEM.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace s2d2 {
namespace tc {

constexpr int BLOCK_N = 128;   // weight rows per tile (MMA M)
constexpr int BLOCK_K = 64;    // bf16 elements per K-block = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int THREADS = 128;

struct GemmParams {
    float* Y;
    int M, N, K;
    int ldy;
    float scale;
    int accumulate;      // Y += result
    int T;               // token rows per tile (multiple of 16, <= 256)
    int stages;
    int splits;          // K splits per tile
    int kb_total;        // K / 64
    int n_tiles, m_tiles;
    float* ws;           // split-K partial tiles [(tile * splits + split)][T][128]
    unsigned* tickets;   // one counter per (n_tile, m_tile), zero between launches
    int* status;         // device status word (0 = ok)
    int evict_first;     // stream W with an evict-first L2 policy
    int wtiles;          // 128-row weight sub-tiles per CTA (1 or 2): two halve the re-reads of the token block
    int hilo;            // X arrives as two bf16 terms (X = X_hi + X_lo): both are token rows of one MMA (N = 2T, T <= 128)
    // gemm_wide_kernel only: the GEMM is gate/up of a SwiGLU layer (W = [gate rows; up rows], f rows each).  A CTA takes the
    // same 128 rows of both halves as its two sub-tiles and writes act = silu(gate) * up as two bf16 terms instead of Y.
    int swiglu = 0;
    int f = 0;
    bf16* act = nullptr;
    bf16* act_lo = nullptr;
};

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes
// (64 bf16) written by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes
// apart (stride byte offset), the leading offset is unused for this layout.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);         // start address, bits [0,14)
    d |= (uint64_t)1 << 16;                              // leading byte offset (ignored), bits [16,30)
    d |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset, bits [32,46)
    d |= (uint64_t)1 << 46;                              // descriptor version of sm_100
    d |= (uint64_t)2 << 61;                              // layout: 128-byte swizzle
    return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = T.
__host__ __device__ __forceinline__ uint32_t instr_desc_bf16(int T) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(T >> 3) << 17) | ((uint32_t)(BLOCK_N >> 4) << 24);
}

// TN: token rows of one stage (T, or 2T with two-term inputs); wtiles: weight sub-tiles of one stage
__host__ __device__ __forceinline__ size_t stage_bytes(int TN, int wtiles = 1) { return (size_t)wtiles * BLOCK_N * 128 + (size_t)TN * 128; }
__host__ __device__ __forceinline__ size_t smem_bytes(int TN, int stages, int wtiles = 1) { return stages * stage_bytes(TN, wtiles) + 1024 + 256; }

static __global__ void __launch_bounds__(THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const __grid_constant__ CUtensorMap map_x_lo, GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // tiles need 1024-byte alignment for the 128-byte swizzle
    uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int S = p.stages, T = p.T, TN = p.hilo ? 2 * p.T : p.T;
    const int WT = p.wtiles, NW = WT * BLOCK_N;      // weight rows of this CTA's tile
    const size_t sbytes = stage_bytes(TN, WT);
    uint64_t* full = (uint64_t*)(tiles + S * sbytes);
    uint64_t* empty = full + S;
    uint64_t* acc_ready = empty + S;
    uint32_t* tmem_slot = (uint32_t*)(acc_ready + 1);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    volatile int* issued = abort_flag + 1;
    volatile int* consumed = issued + 1;
    int* last_flag = (int*)(consumed + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // work item: blockIdx.x -> (n_tile, m_tile, split); the token tile varies fastest so that CTAs
    // sharing a weight tile run together and the tile is fetched from DRAM once
    int item = blockIdx.x;
    const int m_tile = item % p.m_tiles;
    item /= p.m_tiles;
    const int split = item % p.splits;
    const int n_tile = item / p.splits;
    const int kb0 = (int)((long long)p.kb_total * split / p.splits);
    const int kb1 = (int)((long long)p.kb_total * (split + 1) / p.splits);
    const int n0 = n_tile * NW, m0 = m_tile * T;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < WT * TN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(acc_ready, 1);
        *abort_flag = 0;
        *issued = 0;
        *consumed = 0;
        *last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        if (p.hilo) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x_lo) : "memory");
    }
    if (warp == 0) {
        tmem_alloc(tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer ----------------
        uint64_t policy = 0;
        if (p.evict_first) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        for (int kb = kb0; kb < kb1; ++kb) {
            int i = kb - kb0, s = i % S;
            if (i >= S && !mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) {
                *abort_flag = 1;
                break;
            }
            if (*abort_flag) break;
            uint8_t* a = tiles + s * sbytes;
            uint8_t* b = a + (size_t)WT * BLOCK_N * 128;
            mbar_expect_tx(&full[s], (uint32_t)sbytes);
            for (int h = 0; h < WT; ++h) {      // a sub-tile past the matrix is zero-filled
                if (p.evict_first) tma_load_2d_hint(a + h * BLOCK_N * 128, &map_w, kb * BLOCK_K, n0 + h * BLOCK_N, &full[s], policy);
                else tma_load_2d(a + h * BLOCK_N * 128, &map_w, kb * BLOCK_K, n0 + h * BLOCK_N, &full[s]);
            }
            tma_load_2d(b, &map_x, kb * BLOCK_K, m0, &full[s]);
            if (p.hilo) tma_load_2d(b + (size_t)T * 128, &map_x_lo, kb * BLOCK_K, m0, &full[s]);
            *issued = i + 1;
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer ----------------
        const uint32_t idesc = instr_desc_bf16(TN);
        int i = 0;
        for (int kb = kb0; kb < kb1; ++kb, ++i) {
            int s = i % S;
            if (!mbar_wait(&full[s], (i / S) & 1, abort_flag)) {
                *abort_flag = 1;
                break;
            }
            tc_fence_after();
            uint32_t a_addr = smem_u32(tiles + s * sbytes);
            uint32_t b_addr = a_addr + WT * BLOCK_N * 128;
            uint64_t b_desc = smem_desc_sw128(b_addr);
            for (int h = 0; h < WT; ++h) {      // one accumulator of TN columns per weight sub-tile
                uint64_t a_desc = smem_desc_sw128(a_addr + h * BLOCK_N * 128);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
                    // stepping 16 elements (32 bytes) along K inside the swizzled row: +2 in the address field
                    umma_bf16(tmem_base + h * TN, a_desc + 2 * k, b_desc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
                }
            }
            umma_commit(&empty[s]);   // arrives when the MMAs that read this stage are done
            *consumed = i + 1;
        }
        umma_commit(acc_ready);       // arrives when every MMA issued above is done
    }
    __syncwarp();
    // ---------------- epilogue: all four warps ----------------
    bool ok = mbar_wait(acc_ready, 0);
    if (!ok) *abort_flag = 1;
    tc_fence_after();
    __syncthreads();
    const bool aborted = *abort_flag != 0;
    if (aborted) {
        if (threadIdx.x == 0) {
            atomicExch(p.status, 1);
            // both roles have stopped: wait (bounded) for copies already issued into this CTA's
            // shared memory before the CTA may exit
            for (int i = *consumed; i < *issued; ++i) mbar_wait(&full[i % S], (i / S) & 1);
        }
    } else {
        const uint32_t taddr0 = tmem_base + ((uint32_t)(warp * 32) << 16);
        const int m_hi = min(T, p.M - m0);
        // In both epilogues the loads of 16 rows (previous y for an accumulating GEMM, split-K partials)
        // are issued together before anything is stored: one round trip per 16 rows instead of one per row.
        if (p.splits == 1) {
            for (int h = 0; h < WT; ++h) {
            const int n = n0 + h * BLOCK_N + warp * 32 + lane;
            const uint32_t taddr = taddr0 + h * TN;
            for (int c = 0; c < T; c += 16) {
                float v[16];
                tmem_ld16(taddr + c, v);      // executed by the whole warp even past m_hi (aligned instruction)
                if (p.hilo) {
                    float w[16];
                    tmem_ld16(taddr + T + c, w);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += w[j];
                }
                if (n < p.N) {
                    float old[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        old[j] = (p.accumulate && c + j < m_hi) ? __ldcg(p.Y + (size_t)(m0 + c + j) * p.ldy + n) : 0.f;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c + j < m_hi) p.Y[(size_t)(m0 + c + j) * p.ldy + n] = old[j] + p.scale * v[j];
                }
            }
            }
        } else {
            const int tile = n_tile * p.m_tiles + m_tile;
            float* mine = p.ws + ((size_t)tile * p.splits + split) * (size_t)T * NW;
            for (int h = 0; h < WT; ++h) {
            const int n_local = h * BLOCK_N + warp * 32 + lane;
            const uint32_t taddr = taddr0 + h * TN;
            for (int c = 0; c < T; c += 16) {
                float v[16];
                tmem_ld16(taddr + c, v);
                if (p.hilo) {
                    float w[16];
                    tmem_ld16(taddr + T + c, w);
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] += w[j];
                }
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (c + j < m_hi) mine[(size_t)(c + j) * NW + n_local] = v[j];
            }
            }
            __threadfence();
            __syncthreads();
            if (threadIdx.x == 0) {
                unsigned t = atomicAdd(&p.tickets[tile], 1u);
                *last_flag = (t == (unsigned)p.splits - 1);
            }
            __syncthreads();
            if (*last_flag) {
                __threadfence();
                for (int h = 0; h < WT; ++h) {
                const int n_local = h * BLOCK_N + warp * 32 + lane, n = n0 + n_local;
                const float* base = p.ws + (size_t)tile * p.splits * (size_t)T * NW + n_local;
                if (n < p.N) {
                    for (int c = 0; c < m_hi; c += 16) {
                        float acc[16], old[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            acc[j] = 0.f;
                            old[j] = (p.accumulate && c + j < m_hi) ? __ldcg(p.Y + (size_t)(m0 + c + j) * p.ldy + n) : 0.f;
                        }
                        for (int s0 = 0; s0 < p.splits; s0 += 2) {       // partials summed in split order, two splits per round trip
                            float t0[16], t1[16];
                            const bool two = s0 + 1 < p.splits;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const bool in = c + j < m_hi;
                                t0[j] = in ? __ldcg(base + ((size_t)s0 * T + c + j) * NW) : 0.f;
                                t1[j] = in && two ? __ldcg(base + ((size_t)(s0 + 1) * T + c + j) * NW) : 0.f;
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                acc[j] += t0[j];
                                if (two) acc[j] += t1[j];
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (c + j < m_hi) p.Y[(size_t)(m0 + c + j) * p.ldy + n] = old[j] + p.scale * acc[j];
                    }
                }
                }
                if (threadIdx.x == 0) p.tickets[tile] = 0;   // ready for the next launch
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
}

}  // namespace tc
}  // namespace s2d2
