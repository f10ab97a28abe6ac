// Two-mask prefix + block attention for bf16 models.
//
// Every row of a pass attends (1) the whole cached prefix of its sequence, read from
// the paged KV pool, and (2) the rows of the same pass that its 64-bit mask allows
// (the verifier mask [[A, 0], [A<, I]] and the partially causal drafting mask both
// arrive as such masks).  Work is split over (sequence, kv head, tile of 64 query
// vectors, key split): the query vectors of one kv head are the rows of the pass times
// the GQA group, so one CTA serves a whole group with one read of K and V.
//   * cache splits stream whole pages: K and V tiles of one (page, head) are fetched by
//     TMA (2D tensor map over the pool, 128-byte swizzle) into a two-stage ring;
//   * the last split handles the in-pass rows, copied with plain loads into the same
//     swizzled layout, and applies the row masks.
// Each warp owns 16 query vectors: S = Q K^T and O += P V run on mma.sync m16n8k16 (bf16 in,
// fp32 accumulate) with ldmatrix fragments; the online softmax is per thread quad with
// warp shuffles.  Every split writes an unnormalised partial (max, sum, O) and
// attn_combine_kernel merges them in split order.
#pragma once
#include "common.cuh"
#include "tc_ptx.cuh"

namespace s2d2 {
namespace att {

constexpr int QT = 64;          // query vectors per CTA
constexpr int THREADS = 128;
constexpr int STAGES = 2;

struct AttnParams {
    const bf16* q;              // [M, Hq, HD]
    const bf16* q_lo;           // low halves of q (q = hi + lo, both bf16) for the two-term variant, else unused
    bf16* out_lo;               // low halves of the combined output (attn_combine_kernel; may be null)
    const int* sched_off;       // persistent kernel, several sequences: items of CTA c are sched_items[sched_off[c] .. sched_off[c+1])
    const int* sched_items;     // item index = ((seq * Hkv + kv head) * n_qtiles + q tile) * (n_cache_splits + 1) + split; null: idx = cta, cta + G, ..
    const bf16* k_rows;         // [M, Hkv, HD] K of this pass's rows
    const bf16* v_rows;
    bf16* out;                  // [M, Hq*HD]
    float* part_o;              // [items, QT, HD] unnormalised partial outputs
    float* part_ml;             // [items, QT, 2]  (max in log2 units, sum)
    PassView pv;
    int layer, Hq, Hkv, group;
    int page_tokens, page_shift;
    int n_pages_pool;
    int pages_per_split;
    int n_cache_splits;         // grid.x = n_cache_splits + 1 (the last split is the in-pass part)
    int n_qtiles;               // grid.y
    float scale_log2;           // log2(e) / sqrt(HD)
    int* status;
};

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// Byte offset of 16-byte chunk c of row r in a tile of `rows` rows stored as 64-column halves
// of 128-byte rows with the 128-byte swizzle (the layout TMA writes).
__host__ __device__ inline size_t attn_tiles_bytes(int HD) { return (size_t)QT * HD * 2 + (size_t)STAGES * 2 * 64 * HD * 2; }
__device__ __forceinline__ uint32_t sw_off(int r, int c, int rows) {
    return (uint32_t)((c >> 3) * rows * 128 + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// Barrier over a group of `n` threads of the CTA (a whole CTA of 128 threads with id 0, or the
// compute warps of a larger CTA with their own id).
__device__ __forceinline__ void group_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ __forceinline__ bool group_or(int id, int n, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)pred), "r"(id), "r"(n)
        : "memory");
    return r != 0;
}
__device__ __forceinline__ uint4 ldcg16(const void* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }
// x / d for 0 <= x < 2^20 and a small run-time d by one multiplication (an integer division is about 40
// dependent instructions, which a thread that has its scheduler to itself pays in full)
__device__ __forceinline__ int fast_div(int x, int d, float inv_d) {
    int q = (int)(((float)x + 0.5f) * inv_d);
    const int r = x - q * d;
    if (r < 0) --q;
    else if (r >= d) ++q;
    return q;
}

// One work item (sequence z / Hkv, kv head z % Hkv, query tile qt, key split) of the attention
// step, run by a group of 128 threads (`tid` 0..127, barrier `bar_id`).  `base` is 1024-byte
// aligned shared memory of attn_tiles_bytes(HD); `full` are STAGES mbarriers initialised once
// by the caller and `ring_pos` counts the cache tiles this group has streamed through them so
// far (it carries the barrier phase from one item to the next).  Activations are read with
// L2-only loads: inside a persistent kernel they are rewritten by other CTAs between items.
// Returns false when a bounded wait ran out (the status word is raised).
// HL: two-term arithmetic.  q arrives as hi + lo (both bf16) and the probabilities are split the
// same way, so that S = (q_hi + q_lo) K^T and O += (p_hi + p_lo) V carry 16 significant bits of q
// and p; K and V are bf16 as the cache stores them.  Costs twice the (tiny) tensor work.
template <int HD, bool HL = false>
__device__ __forceinline__ bool attn_item(const CUtensorMap* map_kv_ptr, const AttnParams& p, int split, int qt, int z,
                                          uint8_t* base, uint64_t* full, uint32_t& ring_pos, int tid, int bar_id) {
    constexpr int CH = HD / 8;          // 16-byte chunks per row
    constexpr int KS = HD / 16;         // k-steps of Q K^T
    constexpr int NT_O = HD / 8;        // n-tiles of the output
    const int PT = p.page_tokens;                 // keys per tile (16, 32 or 64)
    const int tile_bytes = 64 * HD * 2;           // room for 64 keys even when the page is smaller
    uint8_t* q_s = base;                          // [QT][HD]
    uint8_t* kv_s = base + QT * HD * 2;           // STAGES x (K tile, V tile)

    const int seq = z / p.Hkv, kvh = z % p.Hkv;
    const int nrows = p.pv.seq_nrows[seq], row0 = p.pv.seq_row0[seq];
    const int nq = nrows * p.group;
    const int q0 = qt * QT;
    if (q0 >= nq) return true;
    const int n_ctx = p.pv.seq_nctx[seq];
    const bool in_pass = split == p.n_cache_splits;
    const int n_pages = (n_ctx + PT - 1) >> p.page_shift;
    const int pg0 = split * p.pages_per_split;
    const int pg1 = in_pass ? 0 : min(n_pages, pg0 + p.pages_per_split);
    const int n_tiles = in_pass ? 1 : max(0, pg1 - pg0);
    const size_t item = ((size_t)z * p.n_qtiles + qt) * (p.n_cache_splits + 1) + split;
    const int warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, tq = lane & 3;
    const uint32_t ring0 = ring_pos;
    if (!in_pass) ring_pos += (uint32_t)n_tiles;

    const int* pages = p.pv.seq_pages + (size_t)seq * p.pv.max_pages;
    auto issue = [&](int t) {   // thread 0: TMA of cache tile t of this split into stage t % STAGES
        int s = (int)((ring0 + t) % STAGES);
        int page = pages[pg0 + t];
        uint8_t* kd = kv_s + (size_t)s * 2 * tile_bytes;
        uint8_t* vd = kd + tile_bytes;
        // row of the pool viewed as a 2D matrix [.., HD]: (((layer*n_pages + page)*2 + kv)*Hkv + head)*PT
        long long rk = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 0) * p.Hkv + kvh) * PT;
        long long rv = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 1) * p.Hkv + kvh) * PT;
        tc::mbar_expect_tx(&full[s], (uint32_t)(2 * PT * HD * 2));
#pragma unroll
        for (int h = 0; h < HD / 64; ++h) {
            tc::tma_load_2d(kd + h * PT * 128, map_kv_ptr, h * 64, (int)rk, &full[s]);
            tc::tma_load_2d(vd + h * PT * 128, map_kv_ptr, h * 64, (int)rv, &full[s]);
        }
    };
    if (!in_pass && tid == 0)
        for (int t = 0; t < min(n_tiles, STAGES); ++t) issue(t);

    // ---- Q tile: global -> swizzled shared -> A fragments ----
    constexpr int NQ = QT * CH / THREADS;
    uint4 q_lo_val[HL ? NQ : 1];
    {   // all loads first, then the stores: one round trip for the tile
        uint4 val[NQ];
#pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH, qv = q0 + r;
            val[k] = make_uint4(0, 0, 0, 0);
            if (HL) q_lo_val[k] = val[k];
            if (qv < nq) {
                int row = row0 + qv / p.group, hq = kvh * p.group + qv % p.group;
                val[k] = ldcg16(p.q + ((size_t)row * p.Hq + hq) * HD + c * 8);
                if (HL) q_lo_val[k] = ldcg16(p.q_lo + ((size_t)row * p.Hq + hq) * HD + c * 8);
            }
        }
#pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            *reinterpret_cast<uint4*>(q_s + sw_off(r, c, QT)) = val[k];
        }
    }
    if (in_pass) {
        // K and V of this pass's rows of the sequence into stage 0 (rows past nrows are zero)
        uint8_t* kd = kv_s;
        uint8_t* vd = kd + tile_bytes;
        constexpr int NK = 64 * CH / THREADS;
        uint4 kk[NK], vv[NK];
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            kk[k] = make_uint4(0, 0, 0, 0);
            vv[k] = kk[k];
            if (r < nrows) {
                size_t o = ((size_t)(row0 + r) * p.Hkv + kvh) * HD + c * 8;
                kk[k] = ldcg16(p.k_rows + o);
                vv[k] = ldcg16(p.v_rows + o);
            }
        }
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            *reinterpret_cast<uint4*>(kd + sw_off(r, c, 64)) = kk[k];
            *reinterpret_cast<uint4*>(vd + sw_off(r, c, 64)) = vv[k];
        }
    }
    group_sync(bar_id, THREADS);
    uint32_t qf[KS][4], qf_lo[HL ? KS : 1][4];
    {
        const uint32_t qb = tc::smem_u32(q_s);
        int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            int c = ks * 2 + (lane >> 4);
            ldsm_x4(qb + sw_off(r, c, QT), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
        }
        if (HL) {   // the low halves pass through the same tile
            group_sync(bar_id, THREADS);
#pragma unroll
            for (int k = 0; k < NQ; ++k) {
                const int i = tid + k * THREADS, rr = i / CH, c = i % CH;
                *reinterpret_cast<uint4*>(q_s + sw_off(rr, c, QT)) = q_lo_val[k];
            }
            group_sync(bar_id, THREADS);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                int c = ks * 2 + (lane >> 4);
                ldsm_x4(qb + sw_off(r, c, QT), qf_lo[ks][0], qf_lo[ks][1], qf_lo[ks][2], qf_lo[ks][3]);
            }
        }
    }
    // masks of this thread's two query vectors (rows g and g + 8 of the warp's 16)
    const int qa = q0 + warp * 16 + g, qb_ = qa + 8;
    unsigned long long mask_a = 0, mask_b = 0;
    if (in_pass) {
        if (qa < nq) mask_a = p.pv.row_mask[row0 + qa / p.group];
        if (qb_ < nq) mask_b = p.pv.row_mask[row0 + qb_ / p.group];
    }

    float o[NT_O][4];
#pragma unroll
    for (int i = 0; i < NT_O; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float m_a = -INFINITY, m_b = -INFINITY, l_a = 0.f, l_b = 0.f;
    bool failed = false;

    for (int t = 0; t < n_tiles; ++t) {
        const int s = in_pass ? 0 : (int)((ring0 + t) % STAGES);
        const int rows_t = in_pass ? 64 : PT;           // rows of the tile layout
        const int keys = in_pass ? ((nrows + 15) & ~15) : PT;
        // the wait is bounded; all threads agree on its outcome before going on
        bool ok = in_pass || tc::mbar_wait(&full[s], ((ring0 + t) / STAGES) & 1);
        if (group_or(bar_id, THREADS, !ok)) {
            failed = true;
            break;
        }
        const uint32_t kb = tc::smem_u32(kv_s + (size_t)s * 2 * tile_bytes);
        const uint32_t vb = kb + tile_bytes;
        // ---- S = Q K^T for `keys` keys (8 keys per n-tile) ----
        float sc[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
        for (int np = 0; np < 4; ++np) {             // pairs of n-tiles = 16 keys
            if (np * 16 < keys) {
                int r = np * 16 + (lane & 7) + (lane >> 4) * 8;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    int c = ks * 2 + ((lane >> 3) & 1);
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(kb + sw_off(r, c, rows_t), b0, b1, b2, b3);
                    mma_bf16(sc[np * 2], qf[ks], b0, b1);
                    mma_bf16(sc[np * 2 + 1], qf[ks], b2, b3);
                    if (HL) {
                        mma_bf16(sc[np * 2], qf_lo[ks], b0, b1);
                        mma_bf16(sc[np * 2 + 1], qf_lo[ks], b2, b3);
                    }
                }
            }
        }
        // ---- mask, online softmax (log2 domain) ----
        const int key0 = in_pass ? 0 : (pg0 + t) * PT;
        float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                int col = nt * 8 + tq * 2 + (e & 1);
                bool ok;
                if (in_pass) ok = col < nrows && (((e < 2 ? mask_a : mask_b) >> col) & 1ull);
                else ok = col < keys && key0 + col < n_ctx;
                float v = ok ? sc[nt][e] * p.scale_log2 : -INFINITY;
                sc[nt][e] = v;
                if (e < 2) mx_a = fmaxf(mx_a, v);
                else mx_b = fmaxf(mx_b, v);
            }
        }
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
        mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
        mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
        float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
        float ref_a = mn_a == -INFINITY ? 0.f : mn_a, ref_b = mn_b == -INFINITY ? 0.f : mn_b;
        float corr_a = exp2f(m_a - ref_a), corr_b = exp2f(m_b - ref_b);
        m_a = mn_a;
        m_b = mn_b;
        float sum_a = 0.f, sum_b = 0.f;
        uint32_t pf[4][4], pf_lo[HL ? 4 : 1][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float p0 = exp2f(sc[nt][0] - ref_a), p1 = exp2f(sc[nt][1] - ref_a);
            float p2 = exp2f(sc[nt][2] - ref_b), p3 = exp2f(sc[nt][3] - ref_b);
            sum_a += p0 + p1;
            sum_b += p2 + p3;
            // C fragments of two adjacent key n-tiles are the A fragment of one 16-key k-step
            const uint32_t h01 = pack_bf16(p0, p1), h23 = pack_bf16(p2, p3);
            pf[nt >> 1][(nt & 1) * 2 + 0] = h01;
            pf[nt >> 1][(nt & 1) * 2 + 1] = h23;
            if (HL) {
                const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&h01), b = *reinterpret_cast<const __nv_bfloat162*>(&h23);
                pf_lo[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0 - __low2float(a), p1 - __high2float(a));
                pf_lo[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2 - __low2float(b), p3 - __high2float(b));
            }
        }
        l_a = l_a * corr_a + sum_a;
        l_b = l_b * corr_b + sum_b;
#pragma unroll
        for (int i = 0; i < NT_O; ++i) {
            o[i][0] *= corr_a;
            o[i][1] *= corr_a;
            o[i][2] *= corr_b;
            o[i][3] *= corr_b;
        }
        // ---- O += P V ----
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {             // 16 keys per k-step
            if (kk * 16 < keys) {
                int r = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
                for (int np = 0; np < NT_O / 2; ++np) {
                    int c = np * 2 + (lane >> 4);
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(vb + sw_off(r, c, rows_t), b0, b1, b2, b3);
                    mma_bf16(o[np * 2], pf[kk], b0, b1);
                    mma_bf16(o[np * 2 + 1], pf[kk], b2, b3);
                    if (HL) {
                        mma_bf16(o[np * 2], pf_lo[kk], b0, b1);
                        mma_bf16(o[np * 2 + 1], pf_lo[kk], b2, b3);
                    }
                }
            }
        }
        group_sync(bar_id, THREADS);   // every warp is done with stage s
        if (!in_pass && tid == 0 && t + STAGES < n_tiles) issue(t + STAGES);
    }
    if (failed) {   // uniform across the group
        if (tid == 0) atomicExch(p.status, 2);
        return false;
    }
    // row sums across the quad
    l_a += __shfl_xor_sync(0xffffffffu, l_a, 1);
    l_a += __shfl_xor_sync(0xffffffffu, l_a, 2);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, 1);
    l_b += __shfl_xor_sync(0xffffffffu, l_b, 2);
    // ---- partial (max, sum, O) of this split ----
    float* po = p.part_o + item * QT * HD;
    float* pml = p.part_ml + item * QT * 2;
    int ra = warp * 16 + g, rb = ra + 8;
    if (tq == 0) {
        pml[ra * 2] = m_a;
        pml[ra * 2 + 1] = l_a;
        pml[rb * 2] = m_b;
        pml[rb * 2 + 1] = l_b;
    }
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt) {
        int col = nt * 8 + tq * 2;
        *reinterpret_cast<float2*>(po + (size_t)ra * HD + col) = make_float2(o[nt][0], o[nt][1]);
        *reinterpret_cast<float2*>(po + (size_t)rb * HD + col) = make_float2(o[nt][2], o[nt][3]);
    }
    // the group's shared memory is reused by its next item, possibly by TMA after plain stores
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    group_sync(bar_id, THREADS);
    return true;
}

// ---------------------------------------------------------------------------------------------
// The same work item on the 5th-generation tensor cores (head_dim 128, 64-token pages, two-term q
// and probabilities).  The shared-memory tiles are the ones above: 128-byte rows with the
// 128-byte swizzle, which is the canonical K-major operand layout of tcgen05.mma (and, for V,
// whose rows are keys, the MN-major one).  Per 64-key tile:
//   S[q, key]  = (Q_hi + Q_lo) K^T   16 MMAs (M = 128, N = 64, K = 16) into 64 TMEM columns;
//   one thread per query row (warps 0 and 1 of the group: TMEM lane = row) reads its 64 scores,
//   masks, updates the running maximum and sum, and writes its probabilities as two bf16 terms
//   into a K-major tile; if a maximum moved, the rows rescale their accumulator in TMEM;
//   O[q, :]   += (P_hi + P_lo) V     8 MMAs (N = 128, K = 16) into 128 TMEM columns.
// The MMA tile has 128 rows and a group has 64 query vectors: rows 64..127 read whatever follows
// the 64-row tile in shared memory and their results are never looked at.  Every wait is bounded.
// Shared memory (1024-byte aligned): Q_hi | Q_lo (16 KB each) | STAGES x (K, V).  The probabilities
// (P_hi | P_lo, 8 KB each) take the place of the stage's K tile, which is dead once S is complete;
// with 96 KB per CTA two CTAs share an SM.
__host__ __device__ inline size_t attn_umma_tiles_bytes() { return (size_t)2 * QT * 128 * 2 + (size_t)STAGES * 2 * 64 * 128 * 2; }

// Shared-memory descriptor of an MN-major operand tile stored as rows of 128 bytes (64 bf16 along
// MN) with the 128-byte swizzle, the rows being consecutive K indices: 8-row groups are 1024 bytes
// apart (stride byte offset), the next 64 MN elements start `mn_chunk_bytes` further (leading byte offset).
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t smem_addr, uint32_t mn_chunk_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((mn_chunk_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
__device__ __forceinline__ uint64_t smem_desc_sw128_k(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// D fp32, A and B bf16, A K-major, M = 128; B K-major (b_mn = 0) or MN-major (b_mn = 1)
__device__ __forceinline__ uint32_t umma_idesc(int n, int b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
        "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
        "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
        : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// `bars`: STAGES "tile landed" barriers, then the "scores ready" and "output ready" barriers;
// ring_pos / s_cnt / o_cnt carry their phases from one item to the next.  tmem: 64 columns of
// scores followed by 128 columns of output, lanes 0..127.
// SPLIT: the 80 KB variant for a kernel that cannot spare two stages: one K tile, one V tile and a
// separate P tile (P_hi | P_lo | Q_hi | Q_lo | K | V: what an MMA reads past a 64-row tile is the next
// tile of the same region), the two "tile landed" barriers being K's and
// V's.  The next K is requested as soon as S is complete and the next V as soon as the previous
// P V is, so both arrive behind the softmax of the tile in between.
// SPLIT layout: the K and V tiles of a cache-split item's first page do not depend on anything the
// current pass computes, so a kernel that knows its next item can request them long before it
// reaches the item (the tiles must be free: the previous item of the group has ended).  Every thread
// of the group evaluates the same condition, thread 0 issues the copies.  Returns whether the
// request was made; the item is then entered with first_requested = true.
__device__ __forceinline__ bool attn_umma_request_first(const CUtensorMap* map_kv_ptr, const AttnParams& p, int split, int qt, int z,
                                                        uint8_t* base, uint64_t* bars, uint32_t ring_pos, int tid) {
    constexpr int HD = 128, PT = 64, tile_bytes = 64 * HD * 2;
    const int seq = z / p.Hkv, kvh = z % p.Hkv;
    if (qt * QT >= p.pv.seq_nrows[seq] * p.group || split == p.n_cache_splits) return false;
    const int n_pages = (p.pv.seq_nctx[seq] + PT - 1) >> p.page_shift;
    const int pg0 = split * p.pages_per_split;
    if (pg0 >= n_pages) return false;
    if (tid == 0) {
        uint8_t* kd = base + 2 * QT * 128 + 2 * QT * HD * 2;      // behind P and Q
        uint8_t* vd = kd + tile_bytes;
        const int page = p.pv.seq_pages[(size_t)seq * p.pv.max_pages + pg0];
        const long long rk = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 0) * p.Hkv + kvh) * PT;
        const long long rv = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 1) * p.Hkv + kvh) * PT;
        tc::mbar_expect_tx(&bars[0], (uint32_t)(PT * HD * 2));
        tc::mbar_expect_tx(&bars[1], (uint32_t)(PT * HD * 2));
#pragma unroll
        for (int h = 0; h < HD / 64; ++h) {
            tc::tma_load_2d(kd + h * PT * 128, map_kv_ptr, h * 64, (int)rk, &bars[0]);
            tc::tma_load_2d(vd + h * PT * 128, map_kv_ptr, h * 64, (int)rv, &bars[1]);
        }
    }
    (void)ring_pos;
    return true;
}
// first_requested: tile 0 of this item was already requested by attn_umma_request_first.
// map_q (may be null): two 3D tensor maps of q's high and low halves viewed as [row, head, head_dim] with
// boxes of (64 / group) rows x group heads x 64 columns; the Q tiles then arrive by TMA in query order (one more
// barrier behind the two above, its phase in *q_cnt) instead of passing through registers.  In the SPLIT layout
// map_q[2] and map_q[3] are the same views of this pass's K and V rows (boxes of 64 rows x 1 head): the in-pass
// tile is then fetched like a page.
template <bool SPLIT>
__device__ __forceinline__ bool attn_item_umma(const CUtensorMap* map_kv_ptr, const AttnParams& p, int split, int qt, int z,
                                               uint8_t* base, uint64_t* bars, uint32_t tmem, uint32_t& ring_pos, uint32_t& s_cnt,
                                               uint32_t& o_cnt, int tid, int bar_id, bool first_requested = false,
                                               const CUtensorMap* map_q = nullptr, uint32_t* q_cnt = nullptr) {
    constexpr int HD = 128, CH = HD / 8, PT = 64;
    constexpr int tile_bytes = 64 * HD * 2;
    uint8_t* q_s = base + (SPLIT ? 2 * QT * 128 : 0);      // Q_hi, Q_lo: [QT][HD] each
    uint8_t* kv_s = q_s + 2 * QT * HD * 2;                 // STAGES x (K tile, V tile); SPLIT: one of each
    uint64_t* full = bars;
    uint64_t* bar_s = bars + STAGES;
    uint64_t* bar_o = bars + STAGES + 1;
    const uint32_t tmem_s = tmem, tmem_o = tmem + 64;

    const int seq = fast_div(z, p.Hkv, 1.0f / (float)p.Hkv), kvh = z - seq * p.Hkv;
    const float inv_group = 1.0f / (float)p.group;
    const int nrows = p.pv.seq_nrows[seq], row0 = p.pv.seq_row0[seq];
    const int nq = nrows * p.group;
    const int q0 = qt * QT;
    if (q0 >= nq) return true;
    const int n_ctx = p.pv.seq_nctx[seq];
    const bool in_pass = split == p.n_cache_splits;
    const int n_pages = (n_ctx + PT - 1) >> p.page_shift;
    const int pg0 = split * p.pages_per_split;
    const int pg1 = in_pass ? 0 : min(n_pages, pg0 + p.pages_per_split);
    const int n_tiles = in_pass ? 1 : max(0, pg1 - pg0);
    const size_t item = ((size_t)z * p.n_qtiles + qt) * (p.n_cache_splits + 1) + split;
    const int warp = tid >> 5;
    const bool kv_tma = SPLIT && in_pass && map_q != nullptr;      // the in-pass tile arrives by TMA on the K and V barriers
    const uint32_t ring0 = ring_pos;
    if (!in_pass || kv_tma) ring_pos += (uint32_t)n_tiles;

    const int* pages = p.pv.seq_pages + (size_t)seq * p.pv.max_pages;
    // thread 0: TMA of cache tile t of this split.  which: bit 0 = K, bit 1 = V.  Two-stage layout: both into
    // stage t % STAGES on that stage's barrier; SPLIT: K on barrier 0, V on barrier 1.
    auto issue = [&](int t, int which) {
        const int s = SPLIT ? 0 : (int)((ring0 + t) % STAGES);
        const int page = pages[pg0 + t];
        uint8_t* kd = kv_s + (size_t)s * 2 * tile_bytes;
        uint8_t* vd = kd + tile_bytes;
        const long long rk = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 0) * p.Hkv + kvh) * PT;
        const long long rv = ((((long long)p.layer * p.n_pages_pool + page) * 2 + 1) * p.Hkv + kvh) * PT;
        if (SPLIT) {
            if (which & 1) tc::mbar_expect_tx(&full[0], (uint32_t)(PT * HD * 2));
            if (which & 2) tc::mbar_expect_tx(&full[1], (uint32_t)(PT * HD * 2));
        } else {
            tc::mbar_expect_tx(&full[s], (uint32_t)(2 * PT * HD * 2));
        }
#pragma unroll
        for (int h = 0; h < HD / 64; ++h) {
            if (which & 1) tc::tma_load_2d(kd + h * PT * 128, map_kv_ptr, h * 64, (int)rk, &full[SPLIT ? 0 : s]);
            if (which & 2) tc::tma_load_2d(vd + h * PT * 128, map_kv_ptr, h * 64, (int)rv, &full[SPLIT ? 1 : s]);
        }
    };
    if (!in_pass && tid == 0)
        for (int t = first_requested ? 1 : 0; t < min(n_tiles, SPLIT ? 1 : STAGES); ++t) issue(t, 3);

    // ---- Q tiles (both terms): by TMA, or global -> registers -> swizzled shared ----
    const bool q_tma = map_q != nullptr && n_tiles > 0;
    if (q_tma) {
        if (tid == 0) {
            uint64_t* bar_q = bars + STAGES + 2;
            tc::mbar_expect_tx(bar_q, (uint32_t)(2 * QT * HD * 2));
            const int r_first = row0 + qt * (QT / p.group);
#pragma unroll
            for (int term = 0; term < 2; ++term)
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    tc::tma_load_3d(q_s + term * (QT * HD * 2) + h * (QT * 128), map_q + term, h * 64, kvh * p.group, r_first, bar_q);
        }
    } else {
        constexpr int NQ = QT * CH / THREADS;
        uint4 hi[NQ], lo[NQ];
#pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH, qv = q0 + r;
            hi[k] = make_uint4(0, 0, 0, 0);
            lo[k] = hi[k];
            if (qv < nq) {
                const int qr = fast_div(qv, p.group, inv_group);
                const int row = row0 + qr, hq = kvh * p.group + (qv - qr * p.group);
                hi[k] = ldcg16(p.q + ((size_t)row * p.Hq + hq) * HD + c * 8);
                lo[k] = ldcg16(p.q_lo + ((size_t)row * p.Hq + hq) * HD + c * 8);
            }
        }
#pragma unroll
        for (int k = 0; k < NQ; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            *reinterpret_cast<uint4*>(q_s + sw_off(r, c, QT)) = hi[k];
            *reinterpret_cast<uint4*>(q_s + QT * HD * 2 + sw_off(r, c, QT)) = lo[k];
        }
    }
    if (kv_tma) {
        // rows past the sequence's own are other rows of the pass: their keys are masked below
        if (tid == 0) {
            tc::mbar_expect_tx(&full[0], (uint32_t)(PT * HD * 2));
            tc::mbar_expect_tx(&full[1], (uint32_t)(PT * HD * 2));
#pragma unroll
            for (int h = 0; h < HD / 64; ++h) {
                tc::tma_load_3d(kv_s + h * PT * 128, map_q + 2, h * 64, kvh, row0, &full[0]);
                tc::tma_load_3d(kv_s + tile_bytes + h * PT * 128, map_q + 3, h * 64, kvh, row0, &full[1]);
            }
        }
    } else if (in_pass) {
        // K and V of this pass's rows of the sequence into stage 0 (rows past nrows are zero)
        uint8_t* kd = kv_s;
        uint8_t* vd = kd + tile_bytes;
        constexpr int NK = 64 * CH / THREADS;
        uint4 kk[NK], vv[NK];
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            kk[k] = make_uint4(0, 0, 0, 0);
            vv[k] = kk[k];
            if (r < nrows) {
                size_t o = ((size_t)(row0 + r) * p.Hkv + kvh) * HD + c * 8;
                kk[k] = ldcg16(p.k_rows + o);
                vv[k] = ldcg16(p.v_rows + o);
            }
        }
#pragma unroll
        for (int k = 0; k < NK; ++k) {
            const int i = tid + k * THREADS, r = i / CH, c = i % CH;
            *reinterpret_cast<uint4*>(kd + sw_off(r, c, 64)) = kk[k];
            *reinterpret_cast<uint4*>(vd + sw_off(r, c, 64)) = vv[k];
        }
    }
    // the tiles written with plain stores are read by the tensor core through the async proxy
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    group_sync(bar_id, THREADS);

    const bool row_thread = tid < QT;                       // warps 0 and 1: thread = query row = TMEM lane
    const int qv = q0 + tid;
    unsigned long long row_mask = 0;
    if (in_pass && row_thread && qv < nq) row_mask = p.pv.row_mask[row0 + fast_div(qv, p.group, inv_group)];
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    float m_run = -INFINITY, l_run = 0.f;
    bool failed = false;
    const uint32_t idesc_s = umma_idesc(64, 0), idesc_o = umma_idesc(HD, 1);

    for (int t = 0; t < n_tiles; ++t) {
        const int s = (in_pass || SPLIT) ? 0 : (int)((ring0 + t) % STAGES);
        // the tile (SPLIT: its K) has landed
        bool ok = (in_pass && !kv_tma) || tc::mbar_wait(&full[s], SPLIT ? ((ring0 + t) & 1) : (((ring0 + t) / STAGES) & 1));
        if (q_tma && t == 0) {      // the Q tiles have landed
            ok = tc::mbar_wait(bars + STAGES + 2, *q_cnt & 1) && ok;
            ++*q_cnt;
        }
        if (group_or(bar_id, THREADS, !ok)) {
            failed = true;
            break;
        }
        const uint32_t kb = tc::smem_u32(kv_s + (size_t)s * 2 * tile_bytes);
        const uint32_t vb = kb + tile_bytes;
        uint8_t* p_tile = SPLIT ? base : kv_s + (size_t)s * 2 * tile_bytes;   // P_hi | P_lo: own tile, or over the dead K tile
        if (tid == 0) {
            // ---- S = (Q_hi + Q_lo) K^T: two terms x two 64-column halves of head_dim x four k-steps ----
            tc::tc_fence_after();
            const uint32_t qb = tc::smem_u32(q_s);
#pragma unroll
            for (int term = 0; term < 2; ++term)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint64_t a = smem_desc_sw128_k(qb + term * (QT * HD * 2) + h * (QT * 128));
                    const uint64_t b = smem_desc_sw128_k(kb + h * (64 * 128));
#pragma unroll
                    for (int k = 0; k < 4; ++k) tc::umma_bf16(tmem_s, a + 2 * k, b + 2 * k, idesc_s, (term | h | k) ? 1u : 0u);
                }
            tc::umma_commit(bar_s);
        }
        ok = tc::mbar_wait(bar_s, s_cnt & 1);
        ++s_cnt;
        if (group_or(bar_id, THREADS, !ok)) {
            failed = true;
            break;
        }
        tc::tc_fence_after();
        // The commit above also covers the previous tile's P V MMAs: P, the other stage and the
        // output accumulator are free to be rewritten.
        if (!in_pass && tid == 0) {
            if (SPLIT) {
                if (t + 1 < n_tiles) issue(t + 1, 1);      // K is free: S is complete
                if (t >= 1) issue(t, 2);                   // V is free: the previous P V is complete; this tile's V is needed after the softmax
            } else if (t >= 1 && t + 1 < n_tiles) {
                issue(t + 1, 3);
            }
        }
        float alpha = 1.f;
        if (row_thread) {
            // ---- this row's scores: mask, running maximum and sum (log2 domain), probabilities ----
            const int key0 = in_pass ? 0 : (pg0 + t) * PT;
            float sc[64];
            tc::tmem_ld32(tmem_s + lane_base, sc);
            tc::tmem_ld32(tmem_s + lane_base + 32, sc + 32);
            // raw scores first: the scale is positive, so the maximum can be taken before it is applied
            const bool whole = !in_pass && key0 + 64 <= n_ctx;          // every key of the tile counts (all but a sequence's last page)
            if (!whole) {
#pragma unroll
                for (int j = 0; j < 64; ++j) {
                    const bool keep = in_pass ? (j < nrows && ((row_mask >> j) & 1ull)) : (key0 + j < n_ctx);
                    if (!keep) sc[j] = -INFINITY;
                }
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], sc[j]);
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;
            // The reference point of the exponentials follows the running maximum lazily: it moves only when
            // the maximum has grown by more than 2^8 (probabilities then stay below 256, exact in two bf16
            // terms and harmless in the fp32 sums), so the accumulator in tensor memory is rarely rescaled.
            float m_new = m_run;
            if (t == 0 || mx > m_run + 8.f) m_new = fmaxf(m_run, mx);
            const float ref = m_new == -INFINITY ? 0.f : m_new;
            alpha = m_new == m_run ? 1.f : exp2f(m_run - ref);
            m_run = m_new;
            float sum = 0.f, sum1 = 0.f;
            uint8_t* ph = p_tile + tid * 128;
            const float neg_ref = -ref;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint32_t hi[4], lo[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float p0, p1;      // 2^(s * scale - ref); a masked score (-inf) gives 0
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p0) : "f"(fmaf(sc[c * 8 + 2 * e], p.scale_log2, neg_ref)));
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(p1) : "f"(fmaf(sc[c * 8 + 2 * e + 1], p.scale_log2, neg_ref)));
                    sum += p0;
                    sum1 += p1;
                    hi[e] = pack_bf16(p0, p1);
                    // the bits of a bf16 are the high half of the float with the same value
                    lo[e] = pack_bf16(p0 - __uint_as_float(hi[e] << 16), p1 - __uint_as_float(hi[e] & 0xffff0000u));
                }
                const uint32_t off = (uint32_t)((c ^ (tid & 7)) << 4);
                *reinterpret_cast<uint4*>(ph + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                *reinterpret_cast<uint4*>(ph + QT * 128 + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
            }
            l_run = l_run * alpha + (sum + sum1);
        }
        // ---- rescale the accumulator where a maximum moved (never on the first tile: it is overwritten) ----
        if (t > 0 && group_or(bar_id, THREADS, row_thread && alpha != 1.f)) {
            if (row_thread) {
#pragma unroll
                for (int c = 0; c < HD; c += 16) {
                    float o[16];
                    tc::tmem_ld16(tmem_o + lane_base + c, o);
#pragma unroll
                    for (int j = 0; j < 16; ++j) o[j] *= alpha;
                    tmem_st16(tmem_o + lane_base + c, o);
                }
                tmem_wait_st();
            }
        }
        tc::tc_fence_before();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (SPLIT && (!in_pass || kv_tma)) {       // this tile's V has landed (the barrier below makes the group agree)
            ok = tc::mbar_wait(&full[1], (ring0 + t) & 1);
            if (group_or(bar_id, THREADS, !ok)) {
                failed = true;
                break;
            }
        } else {
            group_sync(bar_id, THREADS);
        }
        if (tid == 0) {
            // ---- O += (P_hi + P_lo) V: two terms x four k-steps of 16 keys ----
            tc::tc_fence_after();
            const uint32_t pb = tc::smem_u32(p_tile);
#pragma unroll
            for (int term = 0; term < 2; ++term) {
                const uint64_t a = smem_desc_sw128_k(pb + term * (QT * 128));
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint64_t b = smem_desc_sw128_mn(vb + k * 2048, 64 * 128);
                    tc::umma_bf16(tmem_o, a + 2 * k, b, idesc_o, (t | term | k) ? 1u : 0u);
                }
            }
            tc::umma_commit(bar_o);
        }
        ++o_cnt;
    }
    if (!failed && n_tiles > 0) {
        bool ok = tc::mbar_wait(bar_o, (o_cnt - 1) & 1);
        if (group_or(bar_id, THREADS, !ok)) failed = true;
    }
    if (failed) {   // uniform across the group
        if (tid == 0) atomicExch(p.status, 2);
        return false;
    }
    tc::tc_fence_after();
    // ---- partial (max, sum, O) of this split ----
    if (row_thread) {
        float* po = p.part_o + (item * QT + tid) * HD;
        float* pml = p.part_ml + (item * QT + tid) * 2;
        pml[0] = m_run;
        pml[1] = l_run;
#pragma unroll
        for (int c = 0; c < HD; c += 32) {
            float o[32];
            if (n_tiles > 0) {
                tc::tmem_ld32(tmem_o + lane_base + c, o);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) o[j] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < 32; j += 4) *reinterpret_cast<float4*>(po + c + j) = make_float4(o[j], o[j + 1], o[j + 2], o[j + 3]);
        }
    }
    // the accumulators are read: the next item's MMAs may overwrite them; shared memory is reused too
    tc::tc_fence_before();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    group_sync(bar_id, THREADS);
    return true;
}

// One CTA per work item, tcgen05 path.  256 columns of tensor memory (64 scores + 128 output used).
static __global__ void __launch_bounds__(THREADS) attn_umma_kernel(const __grid_constant__ CUtensorMap map_kv, AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = (uint64_t*)(base + attn_umma_tiles_bytes());
    uint32_t* tmem_slot = (uint32_t*)(bars + STAGES + 2);
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES + 2; ++s) tc::mbar_init(&bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        tc::tmem_alloc(tmem_slot, 256);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    uint32_t ring_pos = 0, s_cnt = 0, o_cnt = 0;
    bool ok = attn_item_umma<false>(&map_kv, p, blockIdx.x, blockIdx.y, blockIdx.z, base, bars, tmem, ring_pos, s_cnt, o_cnt, threadIdx.x, 0);
    if (!ok && threadIdx.x == 0) {
        // copies already issued target this CTA's shared memory: give them one more bounded wait
        for (int s = 0; s < STAGES; ++s) tc::mbar_wait(&bars[s], 0);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (threadIdx.x < 32) tc::tmem_dealloc(tmem, 256);
}
__host__ __device__ inline size_t attn_umma_smem_bytes() { return attn_umma_tiles_bytes() + 64 + 1024; }

template <int HD, bool HL>
__global__ void __launch_bounds__(THREADS) attn_tc_kernel(const __grid_constant__ CUtensorMap map_kv, AttnParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint64_t* full = (uint64_t*)(base + attn_tiles_bytes(HD));
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) tc::mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t ring_pos = 0;
    bool ok = attn_item<HD, HL>(&map_kv, p, blockIdx.x, blockIdx.y, blockIdx.z, base, full, ring_pos, threadIdx.x, 0);
    if (!ok && threadIdx.x == 0) {
        // copies already issued target this CTA's shared memory: give them one more bounded wait
        // before the CTA leaves
        for (int s = 0; s < STAGES; ++s) tc::mbar_wait(&full[s], 0);
    }
}

// Merges the partials of all splits of one query vector (fixed split order) and writes bf16 (two terms when out_lo is given).
template <int HD>
__global__ void attn_combine_kernel(AttnParams p) {
    int r = blockIdx.x, hq = blockIdx.y;
    int seq = p.pv.row_seq[r];
    int kvh = hq / p.group;
    int qv = (r - p.pv.seq_row0[seq]) * p.group + hq % p.group;
    int qt = qv / QT, qi = qv % QT;
    int n_splits = p.n_cache_splits + 1;
    int n_ctx = p.pv.seq_nctx[seq];
    int n_pages = (n_ctx + p.page_tokens - 1) >> p.page_shift;
    size_t item0 = ((size_t)(seq * p.Hkv + kvh) * p.n_qtiles + qt) * n_splits;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) {
        bool used = s == p.n_cache_splits || s * p.pages_per_split < n_pages;
        if (used) m = fmaxf(m, p.part_ml[(item0 + s) * QT * 2 + qi * 2]);
    }
    for (int c = threadIdx.x; c < HD; c += blockDim.x) {
        float acc = 0.f, l = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            bool used = s == p.n_cache_splits || s * p.pages_per_split < n_pages;
            if (!used) continue;
            float ms = p.part_ml[(item0 + s) * QT * 2 + qi * 2];
            if (ms == -INFINITY) continue;
            float w = exp2f(ms - m);
            l += w * p.part_ml[(item0 + s) * QT * 2 + qi * 2 + 1];
            acc += w * p.part_o[((item0 + s) * QT + qi) * HD + c];
        }
        const float o = acc / l;
        const bf16 hi = __float2bfloat16_rn(o);
        p.out[((size_t)r * p.Hq + hq) * HD + c] = hi;
        if (p.out_lo) p.out_lo[((size_t)r * p.Hq + hq) * HD + c] = __float2bfloat16_rn(o - __bfloat162float(hi));
    }
}

__host__ __device__ inline size_t attn_smem_bytes(int HD) { return attn_tiles_bytes(HD) + 64 + 1024; }

}  // namespace att
}  // namespace s2d2
