// Attention dispatch: bf16 models with 16/32/64-token pages run the tensor-core kernel with
// TMA-staged pages (attention_tc.cuh); everything else runs the plain SIMT kernel.
#include "attention.h"

#include <cuda.h>

#include <algorithm>

#include "attention_tc.cuh"
#include "context.h"
#include "gemm.h"
#include "kernels_simt.cuh"

using namespace s2d2;

namespace s2d2 {
namespace att {
// The merge of attn_combine_kernel for wide passes: one block per row, a warp per query head at a time, four output columns per lane
// (head_dim 128), so a pass of some hundred rows is a few hundred blocks instead of rows x heads small ones.
static __global__ void __launch_bounds__(256) attn_combine_rows_kernel(AttnParams p) {
    constexpr int HD = 128;
    const int r = blockIdx.x, lane = threadIdx.x & 31;
    const int seq = p.pv.row_seq[r];
    const int n_splits = p.n_cache_splits + 1;
    const int n_pages = (p.pv.seq_nctx[seq] + p.page_tokens - 1) >> p.page_shift;
    const int qrow = (r - p.pv.seq_row0[seq]) * p.group;
    for (int hq = threadIdx.x >> 5; hq < p.Hq; hq += 8) {
        const int kvh = hq / p.group;
        const int qv = qrow + hq % p.group;
        const int qt = qv / QT, qi = qv % QT;
        const size_t item0 = ((size_t)(seq * p.Hkv + kvh) * p.n_qtiles + qt) * n_splits;
        float m = -INFINITY;
        for (int s = 0; s < n_splits; ++s) {
            const bool used = s == p.n_cache_splits || s * p.pages_per_split < n_pages;
            if (used) m = fmaxf(m, __ldcg(p.part_ml + (item0 + s) * QT * 2 + qi * 2));
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l = 0.f;
        for (int s = 0; s < n_splits; ++s) {          // fixed split order
            const bool used = s == p.n_cache_splits || s * p.pages_per_split < n_pages;
            if (!used) continue;
            const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (item0 + s) * QT * 2 + qi * 2));
            if (ml.x == -INFINITY) continue;
            const float w = exp2f(ml.x - m);
            const float4 o = __ldcg(reinterpret_cast<const float4*>(p.part_o + ((item0 + s) * QT + qi) * HD) + lane);
            l += w * ml.y;
            acc.x += w * o.x;
            acc.y += w * o.y;
            acc.z += w * o.z;
            acc.w += w * o.w;
        }
        const float o0 = acc.x / l, o1 = acc.y / l, o2 = acc.z / l, o3 = acc.w / l;
        const size_t off = ((size_t)r * p.Hq + hq) * HD + lane * 4;
        const __nv_bfloat162 h0 = __floats2bfloat162_rn(o0, o1), h1 = __floats2bfloat162_rn(o2, o3);
        uint2 u;
        u.x = *reinterpret_cast<const uint32_t*>(&h0);
        u.y = *reinterpret_cast<const uint32_t*>(&h1);
        *reinterpret_cast<uint2*>(p.out + off) = u;
        if (p.out_lo) {
            const __nv_bfloat162 l0 = __floats2bfloat162_rn(o0 - __low2float(h0), o1 - __high2float(h0));
            const __nv_bfloat162 l1 = __floats2bfloat162_rn(o2 - __low2float(h1), o3 - __high2float(h1));
            u.x = *reinterpret_cast<const uint32_t*>(&l0);
            u.y = *reinterpret_cast<const uint32_t*>(&l1);
            *reinterpret_cast<uint2*>(p.out_lo + off) = u;
        }
    }
}
}  // namespace att
}  // namespace s2d2

namespace {
struct AttnState {
    bool tc_ok = false;
    CUtensorMap map_kv;
    float* part_o = nullptr;
    float* part_ml = nullptr;
    size_t cap_items = 0;
    bool umma_ok = false;        // tcgen05 work items (head_dim 128, 64-token pages)
    int n_sms = 148;
};
AttnState* state(s2d2_ctx* c) { return (AttnState*)c->attn_state; }

template <typename TKV>
KvPool<TKV> make_pool(s2d2_ctx* c) {
    KvPool<TKV> p;
    p.base = (TKV*)c->kv_base;
    p.page_tokens = c->page_tokens;
    p.page_shift = c->page_shift;
    p.n_kv_heads = c->m.n_kv_heads;
    p.head_dim = c->m.head_dim;
    p.page_stride = (size_t)2 * c->m.n_kv_heads * c->page_tokens * c->m.head_dim;
    p.layer_stride = (size_t)c->n_pages * p.page_stride;
    return p;
}

template <typename TA, typename TKV>
void attention_simt(s2d2_ctx* c, const PassView& pv, int layer) {
    const s2d2_model_config& m = c->m;
    int warps = pv.n_rows * m.n_q_heads;
    int blocks = (warps + 3) / 4;
    float scale = 1.f / sqrtf((float)m.head_dim);
    KvPool<TKV> pool = make_pool<TKV>(c);
#define ATT(HD)                                                                                               \
    attention_simt_kernel<TA, TKV, HD><<<blocks, 128, 0, c->stream>>>((const TA*)c->q, (const TKV*)c->k_rows, \
                                                                      (const TKV*)c->v_rows, pv, pool, layer, \
                                                                      m.n_q_heads, m.n_kv_heads, (TA*)c->attn, scale)
    if (m.head_dim == 32) ATT(32);
    else if (m.head_dim == 64) ATT(64);
    else ATT(128);
#undef ATT
    c->cnt.n_kernel_launches++;
}
}  // namespace

int attention_init(s2d2_ctx* c) {
    AttnState* a = new AttnState();
    c->attn_state = a;
    const s2d2_model_config& m = c->m;
    if (m.dtype != S2D2_DTYPE_BF16 || !gemm_tc_available(c)) return S2D2_OK;
    if (!(m.head_dim == 64 || m.head_dim == 128) || c->page_tokens < 16) return S2D2_OK;
    unsigned long long rows = (unsigned long long)m.n_layers * c->n_pages * 2 * m.n_kv_heads * c->page_tokens;
    if (rows >= (1ull << 31)) return S2D2_OK;      // row coordinates are 32-bit
    if (gemm_encode_map(c, &a->map_kv, c->kv_base, rows, m.head_dim, c->page_tokens) != 0) {
        c->err = "cuTensorMapEncodeTiled failed for the KV pool";
        return S2D2_ERR_CUDA;
    }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) return S2D2_ERR_CUDA;
    a->n_sms = prop.multiProcessorCount;
    int group = m.n_q_heads / m.n_kv_heads;
    // (a prefill pass lists every 64-row chunk of a prompt as a sequence of its own)
    size_t base_items = (size_t)(c->dc.max_batch + c->max_rows / S2D2_MAX_ROWS_PER_SEQ) * m.n_kv_heads * ((S2D2_MAX_ROWS_PER_SEQ * group + att::QT - 1) / att::QT);
    a->cap_items = std::max<size_t>(2048, base_items * 2);
    if (cudaMalloc((void**)&a->part_o, a->cap_items * att::QT * m.head_dim * 4) != cudaSuccess) return S2D2_ERR_CUDA;
    if (cudaMalloc((void**)&a->part_ml, a->cap_items * att::QT * 2 * 4) != cudaSuccess) return S2D2_ERR_CUDA;
    const int smem = (int)att::attn_smem_bytes(m.head_dim);
    const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
    cudaError_t e = m.head_dim == 128 ? cudaFuncSetAttribute(att::attn_tc_kernel<128, true>, attr, smem)
                                      : cudaFuncSetAttribute(att::attn_tc_kernel<64, true>, attr, smem);
    if (e == cudaSuccess)
        e = m.head_dim == 128 ? cudaFuncSetAttribute(att::attn_tc_kernel<128, false>, attr, smem)
                              : cudaFuncSetAttribute(att::attn_tc_kernel<64, false>, attr, smem);
    if (e == cudaSuccess && m.head_dim == 128 && c->page_tokens == 64) {
        e = cudaFuncSetAttribute(att::attn_umma_kernel, attr, (int)att::attn_umma_smem_bytes());
        a->umma_ok = e == cudaSuccess;
    }
    if (e != cudaSuccess) return S2D2_ERR_CUDA;
    a->tc_ok = true;
    return S2D2_OK;
}

void attention_destroy(s2d2_ctx* c) {
    AttnState* a = state(c);
    if (!a) return;
    if (a->part_o) cudaFree(a->part_o);
    if (a->part_ml) cudaFree(a->part_ml);
    delete a;
    c->attn_state = nullptr;
}

// Geometry of the tensor-core attention for one pass (query tiles, key splits, partial buffers).
// Returns false when the pass must take the plain kernel instead.
bool attention_plan(s2d2_ctx* c, const PassView& pv, int max_ctx, int max_rows, int target_items, att::AttnParams* out,
                    const void** map_kv) {
    const s2d2_model_config& m = c->m;
    AttnState* a = state(c);
    if (!a || !a->tc_ok) return false;
    att::AttnParams p;
    p.q = (const bf16*)c->q;
    p.q_lo = (const bf16*)c->q_lo;
    p.k_rows = (const bf16*)c->k_rows;
    p.v_rows = (const bf16*)c->v_rows;
    p.out = (bf16*)c->attn;
    p.out_lo = (bf16*)c->attn_lo;
    p.sched_off = nullptr;
    p.sched_items = nullptr;
    p.part_o = a->part_o;
    p.part_ml = a->part_ml;
    p.pv = pv;
    p.layer = 0;
    p.Hq = m.n_q_heads;
    p.Hkv = m.n_kv_heads;
    p.group = m.n_q_heads / m.n_kv_heads;
    p.page_tokens = c->page_tokens;
    p.page_shift = c->page_shift;
    p.n_pages_pool = c->n_pages;
    p.n_qtiles = std::max(1, (max_rows * p.group + att::QT - 1) / att::QT);
    int max_pages = (max_ctx + c->page_tokens - 1) / c->page_tokens;
    size_t base = (size_t)pv.n_seqs * m.n_kv_heads * p.n_qtiles;
    // enough key splits to reach the wanted number of work items, bounded by the partial buffers
    if (target_items <= 0) target_items = 2 * a->n_sms;
    int want = (int)std::min<size_t>((target_items + base - 1) / base, a->cap_items / base - 1);
    want = std::max(1, std::min(want, std::max(1, max_pages)));
    p.pages_per_split = std::max(1, (max_pages + want - 1) / want);
    p.n_cache_splits = (max_pages + p.pages_per_split - 1) / p.pages_per_split;
    p.scale_log2 = 1.4426950408889634f / sqrtf((float)m.head_dim);
    p.status = c->d_status;
    if (base * (p.n_cache_splits + 1) > a->cap_items) return false;
    *out = p;
    if (map_kv) *map_kv = &a->map_kv;
    return true;
}

int attention(s2d2_ctx* c, const PassView& pv, int layer, int max_ctx, int max_rows) {
    const s2d2_model_config& m = c->m;
    AttnState* a = state(c);
    if (m.dtype == S2D2_DTYPE_F32) {
        attention_simt<float, float>(c, pv, layer);
        return S2D2_OK;
    }
    att::AttnParams p;
    if (!attention_plan(c, pv, max_ctx, max_rows, 0, &p, nullptr)) {
        attention_simt<bf16, bf16>(c, pv, layer);
        return S2D2_OK;
    }
    p.layer = layer;
    dim3 grid(p.n_cache_splits + 1, p.n_qtiles, pv.n_seqs * m.n_kv_heads);
    const size_t smem = att::attn_smem_bytes(m.head_dim);
    // two-term queries and probabilities whenever the low halves of q exist (always on this path)
    if (a->umma_ok && p.q_lo) {
        att::attn_umma_kernel<<<grid, att::THREADS, att::attn_umma_smem_bytes(), c->stream>>>(a->map_kv, p);
        if (pv.n_rows > 64) att::attn_combine_rows_kernel<<<pv.n_rows, 256, 0, c->stream>>>(p);
        else att::attn_combine_kernel<128><<<dim3(pv.n_rows, m.n_q_heads), 128, 0, c->stream>>>(p);
    } else if (m.head_dim == 128) {
        if (p.q_lo) att::attn_tc_kernel<128, true><<<grid, att::THREADS, smem, c->stream>>>(a->map_kv, p);
        else att::attn_tc_kernel<128, false><<<grid, att::THREADS, smem, c->stream>>>(a->map_kv, p);
        att::attn_combine_kernel<128><<<dim3(pv.n_rows, m.n_q_heads), 128, 0, c->stream>>>(p);
    } else {
        if (p.q_lo) att::attn_tc_kernel<64, true><<<grid, att::THREADS, smem, c->stream>>>(a->map_kv, p);
        else att::attn_tc_kernel<64, false><<<grid, att::THREADS, smem, c->stream>>>(a->map_kv, p);
        att::attn_combine_kernel<64><<<dim3(pv.n_rows, m.n_q_heads), 64, 0, c->stream>>>(p);
    }
    c->cnt.n_kernel_launches += 2;
    return S2D2_OK;
}
