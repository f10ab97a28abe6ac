// The weight-streaming tcgen05 GEMM for wide passes (more than 64 token rows: large batches, prefill).
//
//   Y[m, n] (+)= scale * sum_k (X_hi[m, k] + X_lo[m, k]) * W[n, k]
//
// Operand roles, tiles and the producer / MMA-issuer pair are those of gemm_tc_kernel (gemm_tc.cuh); what
// differs is everything behind the last MMA.  With 100 to 130 token rows per tile the per-row epilogue of
// that kernel (a dependent round trip to L2 per 16 rows for the residual it adds to, and one thread block
// summing the split-K partials load by load) lasted longer than the stream of a K = 4096 tile, which kept
// the host from splitting K and left the GEMMs with few weight tiles (QKV, O, down) on a fraction of the
// SMs.  Here the accumulators go to shared memory once and leave it as bulk copies:
//   * no split:  one bulk store (or bulk add, for a GEMM that accumulates into the residual) per output
//     row and weight sub-tile, 512 bytes each, issued by 128 threads, no register round trip;
//   * split K:   every CTA stores its partial sub-tiles with one bulk copy each; the CTA that takes the
//     last ticket of a tile fetches the partials back by bulk copies, double-buffered, adds them in split
//     order (so the result does not depend on timing) and stores as above.
// Every wait is bounded; a time-out raises the status word and the CTA leaves after its copies have landed.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "gemm_tc.cuh"
#include "tc_ptx.cuh"

namespace s2d2 {
namespace tc {

// bytes of one sub-tile of fp32 results in shared memory: [T][128]
__host__ __device__ __forceinline__ size_t wide_sub_bytes(int T) { return (size_t)T * BLOCK_N * 4; }
// tile area of the kernel: the stage ring, or the epilogue's buffers where those need more
// (no split: one buffer per weight sub-tile; split K: the same, and for the summing CTA one sum and two staging buffers)
__host__ __device__ __forceinline__ size_t wide_tile_bytes(int T, int TN, int stages, int wtiles, int splits) {
    size_t ring = (size_t)stages * stage_bytes(TN, wtiles);
    size_t epi = (size_t)(splits > 1 ? (wtiles > 3 ? wtiles : 3) : wtiles) * wide_sub_bytes(T);
    return ring > epi ? ring : epi;
}
__host__ __device__ __forceinline__ size_t wide_smem_bytes(int T, int TN, int stages, int wtiles, int splits) {
    return wide_tile_bytes(T, TN, stages, wtiles, splits) + 1024 + 512;
}

__device__ __forceinline__ void bulk_store(void* gdst, const void* ssrc, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(ssrc)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_add_f32(void* gdst, const void* ssrc, uint32_t bytes) {
    asm volatile("cp.reduce.async.bulk.global.shared::cta.bulk_group.add.f32 [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(ssrc)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_load(void* sdst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_u32(sdst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// tcgen05.ld without its wait: several loads may be in flight before tmem_ld_wait()
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
    tmem_ld16_issue(taddr, r);
    tmem_ld16_issue(taddr + 16, r + 16);
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Partial sub-tiles of split-K launches: ws[((tile * splits + split) * wtiles + h)][T][128] fp32.
static __global__ void __launch_bounds__(THREADS)
gemm_wide_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                 const __grid_constant__ CUtensorMap map_x_lo, GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const int S = p.stages, T = p.T, TN = p.hilo ? 2 * p.T : p.T;
    const int WT = p.wtiles, NW = WT * BLOCK_N;
    const size_t sbytes = stage_bytes(TN, WT);
    const size_t sub = wide_sub_bytes(T);
    uint64_t* full = (uint64_t*)(tiles + wide_tile_bytes(T, TN, S, WT, p.splits));
    uint64_t* empty = full + S;
    uint64_t* acc_ready = empty + S;
    uint64_t* red_bar = acc_ready + 1;            // two barriers of the summing CTA's staging buffers, one of its sum buffer
    uint32_t* tmem_slot = (uint32_t*)(red_bar + 3);
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    volatile int* issued = abort_flag + 1;
    volatile int* consumed = issued + 1;
    int* last_flag = (int*)(consumed + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
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
        for (int s = 0; s < 3; ++s) mbar_init(&red_bar[s], 1);
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
            for (int h = 0; h < WT; ++h)       // a sub-tile past the matrix is zero-filled
                tma_load_2d(a + h * BLOCK_N * 128, &map_w, kb * BLOCK_K, p.swiglu ? h * p.f + n_tile * BLOCK_N : n0 + h * BLOCK_N, &full[s]);
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
            for (int h = 0; h < WT; ++h) {
                uint64_t a_desc = smem_desc_sw128(a_addr + h * BLOCK_N * 128);
#pragma unroll
                for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                    umma_bf16(tmem_base + h * TN, a_desc + 2 * k, b_desc + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit(&empty[s]);
            *consumed = i + 1;
        }
        umma_commit(acc_ready);
    }
    __syncwarp();
    bool ok = mbar_wait(acc_ready, 0);
    if (!ok) *abort_flag = 1;
    tc_fence_after();
    __syncthreads();
    if (*abort_flag != 0) {
        if (threadIdx.x == 0) {
            atomicExch(p.status, 1);
            for (int i = *consumed; i < *issued; ++i) mbar_wait(&full[i % S], (i / S) & 1);
        }
        tc_fence_before();
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
        return;
    }

    // ---------------- accumulators -> shared memory, one [T][128] fp32 buffer per weight sub-tile ----------------
    const int m_hi = min(T, p.M - m0);
    const int n_local = warp * 32 + lane;
    const float out_scale = p.splits == 1 ? p.scale : 1.f;
    for (int h = 0; h < WT; ++h) {
        float* buf = (float*)(tiles + h * sub) + n_local;
        const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + h * TN;
        int c = 0;
        for (; c + 32 <= T; c += 32) {        // both terms' columns requested before the one wait
            uint32_t v[32], w[32];
            tmem_ld32_issue(taddr + c, v);
            if (p.hilo) tmem_ld32_issue(taddr + T + c, w);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j)
                buf[(c + j) * BLOCK_N] = (__uint_as_float(v[j]) + (p.hilo ? __uint_as_float(w[j]) : 0.f)) * out_scale;
        }
        if (c < T) {                          // T is a multiple of 16
            uint32_t v[16], w[16];
            tmem_ld16_issue(taddr + c, v);
            if (p.hilo) tmem_ld16_issue(taddr + T + c, w);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 16; ++j)
                buf[(c + j) * BLOCK_N] = (__uint_as_float(v[j]) + (p.hilo ? __uint_as_float(w[j]) : 0.f)) * out_scale;
        }
    }
    fence_async_smem();       // the bulk copies below read what the threads have just written
    tc_fence_before();
    __syncthreads();

    // rows of one finished sub-tile go to Y: 512 bytes (less at the right edge of the matrix) per bulk operation
    auto rows_out = [&](const uint8_t* buf, int h) {
        const int n_valid = min(BLOCK_N, p.N - (n0 + h * BLOCK_N));
        if (n_valid > 0) {
            for (int m = threadIdx.x; m < m_hi; m += THREADS) {
                float* dst = p.Y + (size_t)(m0 + m) * p.ldy + n0 + h * BLOCK_N;
                if (p.accumulate) bulk_add_f32(dst, buf + (size_t)m * BLOCK_N * 4, (uint32_t)n_valid * 4);
                else bulk_store(dst, buf + (size_t)m * BLOCK_N * 4, (uint32_t)n_valid * 4);
            }
        }
        bulk_commit();
    };

    if (p.swiglu) {
        // sub-tile 0 holds the gate columns, sub-tile 1 the up columns of the same 128 outputs: eight columns per thread and step
        const float* g = (const float*)tiles;
        const float* u = (const float*)(tiles + sub);
        const int col0 = n_tile * BLOCK_N;
        for (int idx = threadIdx.x; idx < m_hi * (BLOCK_N / 8); idx += THREADS) {
            const int m = idx / (BLOCK_N / 8), c8 = (idx % (BLOCK_N / 8)) * 8;
            float a[8];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const float4 gv = *(const float4*)(g + m * BLOCK_N + c8 + 4 * q), uv = *(const float4*)(u + m * BLOCK_N + c8 + 4 * q);
                a[4 * q + 0] = gv.x / (1.f + expf(-gv.x)) * uv.x;
                a[4 * q + 1] = gv.y / (1.f + expf(-gv.y)) * uv.y;
                a[4 * q + 2] = gv.z / (1.f + expf(-gv.z)) * uv.z;
                a[4 * q + 3] = gv.w / (1.f + expf(-gv.w)) * uv.w;
            }
            uint32_t hi[4], lo[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const bf16 h0 = __float2bfloat16_rn(a[2 * q]), h1 = __float2bfloat16_rn(a[2 * q + 1]);
                const bf16 l0 = __float2bfloat16_rn(a[2 * q] - __bfloat162float(h0)), l1 = __float2bfloat16_rn(a[2 * q + 1] - __bfloat162float(h1));
                hi[q] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
                lo[q] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
            }
            const size_t o = (size_t)(m0 + m) * p.f + col0 + c8;
            *(uint4*)(p.act + o) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *(uint4*)(p.act_lo + o) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    } else if (p.splits == 1) {
        for (int h = 0; h < WT; ++h) rows_out(tiles + h * sub, h);
        bulk_wait_read();
    } else {
        const int tile = n_tile * p.m_tiles + m_tile;
        float* ws_tile = p.ws + (size_t)tile * p.splits * WT * (sub / 4);
        if (threadIdx.x == 0) {
            float* mine = ws_tile + (size_t)split * WT * (sub / 4);
            for (int h = 0; h < WT; ++h) bulk_store(mine + (size_t)h * (sub / 4), tiles + h * sub, (uint32_t)sub);
            bulk_commit();
            bulk_wait_all();          // written, not only read
            fence_async_all();
            __threadfence();
            unsigned t = atomicAdd(&p.tickets[tile], 1u);
            *last_flag = (t == (unsigned)p.splits - 1);
        }
        __syncthreads();
        if (*last_flag) {
            // this CTA took the tile's last ticket: every partial is in the workspace
            if (threadIdx.x == 0) {
                __threadfence();
                fence_async_all();
            }
            uint8_t* sum = tiles;
            uint8_t* stg[2] = {tiles + sub, tiles + 2 * sub};
            uint32_t uses[2] = {0, 0};
            const int n4 = T * (BLOCK_N / 4);                  // float4 elements of a sub-tile
            for (int h = 0; h < WT; ++h) {
                const float* part = ws_tile + (size_t)h * (sub / 4);
                const size_t part_stride = (size_t)WT * (sub / 4);
                if (threadIdx.x == 0) {
                    mbar_expect_tx(&red_bar[2], (uint32_t)sub);
                    bulk_load(sum, part, (uint32_t)sub, &red_bar[2]);
                    for (int s = 1; s < p.splits && s <= 2; ++s) {
                        mbar_expect_tx(&red_bar[(s - 1) & 1], (uint32_t)sub);
                        bulk_load(stg[(s - 1) & 1], part + s * part_stride, (uint32_t)sub, &red_bar[(s - 1) & 1]);
                    }
                }
                if (!mbar_wait(&red_bar[2], h & 1, abort_flag)) *abort_flag = 1;
                for (int s = 1; s < p.splits; ++s) {           // partials added in split order
                    const int b = (s - 1) & 1;
                    if (!mbar_wait(&red_bar[b], uses[b] & 1, abort_flag)) *abort_flag = 1;
                    ++uses[b];
                    const float sc = s == p.splits - 1 ? p.scale : 1.f;
                    float4* a4 = (float4*)sum;
                    const float4* b4 = (const float4*)stg[b];
                    for (int i = threadIdx.x; i < n4; i += THREADS) {
                        float4 x = a4[i], y = b4[i];
                        x.x = (x.x + y.x) * sc;
                        x.y = (x.y + y.y) * sc;
                        x.z = (x.z + y.z) * sc;
                        x.w = (x.w + y.w) * sc;
                        a4[i] = x;
                    }
                    __syncthreads();
                    if (threadIdx.x == 0 && s + 2 < p.splits) {
                        mbar_expect_tx(&red_bar[b], (uint32_t)sub);
                        bulk_load(stg[b], part + (size_t)(s + 2) * part_stride, (uint32_t)sub, &red_bar[b]);
                    }
                }
                fence_async_smem();
                __syncthreads();
                rows_out(sum, h);
                bulk_wait_read();
                __syncthreads();          // the next sub-tile's first partial lands in the sum buffer
            }
            if (threadIdx.x == 0) {
                p.tickets[tile] = 0;      // ready for the next launch
                if (*abort_flag) atomicExch(p.status, 1);
            }
        }
    }
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
}

}  // namespace tc
}  // namespace s2d2
