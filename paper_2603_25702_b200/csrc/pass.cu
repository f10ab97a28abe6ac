// Launch logic of the persistent pass kernel: tensor maps of every weight matrix and activation
// buffer, split-K workspace sizing, eligibility, cooperative launch.
#include "pass.h"

#include <cuda.h>

#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <queue>
#include <utility>
#include <vector>

#include "attention.h"
#include "context.h"
#include "gemm.h"
#include "pass_kernel.cuh"

using namespace s2d2;

namespace {
struct PassState {
    bool ok = false;
    bool moe = false;
    int grid = 0;
    int max_smem = 0;
    int maps_per_layer = 4;
    int map_x0 = 0;              // xn maps for T = 16, 32, 48, 64; then attn; then act; then their low halves; then xn_b (+24) and its low halves (+36)
    int map_act_e = 0;           // per T: experts' SwiGLU output, high halves then low halves
    int map_kv = 0;
    bool q_by_tma = false;       // maps map_kv + 1 / + 2: q high and low halves as 3D boxes
    CUtensorMap* d_maps = nullptr;
    pp::LayerGains* d_gains = nullptr;
    float* ws = nullptr;
    bf16 *xn_lo = nullptr, *attn_lo = nullptr, *act_lo = nullptr, *q_lo = nullptr, *act_e = nullptr, *act_e_lo = nullptr;
    bf16 *xn_b = nullptr, *xn_b_lo = nullptr;
    pp::SubDesc subs[pp::N_KINDS][pp::MAX_SUBS] = {};
    int n_subs[pp::N_KINDS] = {};
    long long ws_off[pp::N_KINDS] = {};
    int max_segs[pp::N_KINDS] = {};
    float *ssq_a = nullptr, *ssq_b = nullptr;
    unsigned* barrier = nullptr;     // [64 | tile counters of the static GEMM kinds | x counters], zeroed before every launch
    size_t sync_bytes = 0;
    long long cnt_off[pp::N_KINDS] = {};     // -1: the kind publishes through a grid barrier
    size_t xcnt_off[4] = {0, 0, 0, 0};
    size_t attn_cnt_off = 0;
    unsigned long long* trace = nullptr;
    int trace_cap = 0;
    int trace_mma0 = 0, n_sub_gemms = 0;
    int4* segs = nullptr;            // dense models: per CTA the list of its (weight tile, k-block range) segments, a layer's then the LM head's
    int* seg_sub_begin = nullptr;    // per CTA: first segment of every sub-GEMM of the two lists, then the total
    int seg_stride = 0, n_layer_subs = 0, n_lm_subs = 0;
    int last_marks = 0;
    int barriers_per_layer = 6;
    int* parts[pp::N_KINDS] = {};    // split-K part tables of the static GEMM kinds
    int* n_touched = nullptr;        // [n_layers] device, touched experts of the last pass
    int* n_touched_h = nullptr;      // pinned mirror
    // attention schedule of passes with several sequences: [grid + 1 offsets | items], two slots used in turn
    int* sched_h[2] = {nullptr, nullptr};   // pinned
    int* sched_d[2] = {nullptr, nullptr};
    cudaEvent_t sched_copied[2] = {nullptr, nullptr};
    size_t sched_cap = 0;            // items per slot
    int sched_next = 0;
    double weight_bytes = 0;         // bytes of every matrix a pass always streams (without the LM head)
    double expert_bytes = 0;         // bytes of one routed expert's three matrices
    double head_bytes = 0;
};
PassState* state(s2d2_ctx* c) { return (PassState*)c->pass_state; }

// Attention items of a pass with several sequences, dealt out to the CTAs by cost (longest first,
// each to the least loaded CTA): context lengths differ between sequences, and dealing items out
// by index leaves some CTAs with twice the median work.  Item cost in units of about a
// microsecond: a fixed part (query tile, first page latency, partial store) + one per 64-key page.
// Returns the device pointer of [grid + 1 offsets | items], or null (the caller falls back to
// the index order) when a copy could not be set up.
const int* attention_schedule(s2d2_ctx* c, PassState* s, const att::AttnParams& ap) {
    const PassMeta& pm = c->meta;
    const int* nctx = pm.hp<int>(pm.off_nctx);
    const int* nrows = pm.hp<int>(pm.off_nrows);
    const int n_splits = ap.n_cache_splits + 1, G = s->grid;
    std::vector<std::pair<float, int>> items;      // (cost, item index)
    for (int seq = 0; seq < ap.pv.n_seqs; ++seq) {
        const int n_pages = (nctx[seq] + ap.page_tokens - 1) >> ap.page_shift;
        const int nq = nrows[seq] * ap.group;
        for (int kvh = 0; kvh < ap.Hkv; ++kvh)
            for (int qt = 0; qt < ap.n_qtiles && qt * att::QT < nq; ++qt)
                for (int split = 0; split < n_splits; ++split) {
                    const int idx = ((seq * ap.Hkv + kvh) * ap.n_qtiles + qt) * n_splits + split;
                    if (split == ap.n_cache_splits) {
                        items.emplace_back(5.f, idx);
                    } else {
                        const int pg0 = split * ap.pages_per_split;
                        if (pg0 >= n_pages) continue;
                        items.emplace_back(3.f + 3.f * (float)(std::min(n_pages, pg0 + ap.pages_per_split) - pg0), idx);
                    }
                }
    }
    const size_t need = (size_t)G + 1 + items.size();
    const int k = s->sched_next;
    if (need > s->sched_cap || !s->sched_h[k]) {
        if (s->sched_copied[k]) cudaEventSynchronize(s->sched_copied[k]);
        if (cudaStreamSynchronize(c->stream) != cudaSuccess) return nullptr;
        for (int j = 0; j < 2; ++j) {
            if (s->sched_h[j]) cudaFreeHost(s->sched_h[j]);
            if (s->sched_d[j]) cudaFree(s->sched_d[j]);
            s->sched_h[j] = s->sched_d[j] = nullptr;
        }
        s->sched_cap = std::max<size_t>(2 * need, 4096);
        for (int j = 0; j < 2; ++j) {
            if (cudaMallocHost((void**)&s->sched_h[j], s->sched_cap * 4) != cudaSuccess ||
                cudaMalloc((void**)&s->sched_d[j], s->sched_cap * 4) != cudaSuccess)
                return nullptr;
            if (!s->sched_copied[j] && cudaEventCreateWithFlags(&s->sched_copied[j], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
    } else if (cudaEventSynchronize(s->sched_copied[k]) != cudaSuccess) {      // the slot's previous copy has left the host buffer
        return nullptr;
    }
    std::stable_sort(items.begin(), items.end(), [](const std::pair<float, int>& a, const std::pair<float, int>& b) { return a.first > b.first; });
    typedef std::pair<float, int> Load;           // (load, cta): the least loaded CTA, lowest id first
    std::priority_queue<Load, std::vector<Load>, std::greater<Load>> heap;
    for (int g = 0; g < G; ++g) heap.push(Load(0.f, g));
    std::vector<std::vector<int>> mine(G);
    for (const auto& it : items) {
        Load l = heap.top();
        heap.pop();
        mine[l.second].push_back(it.second);
        heap.push(Load(l.first + it.first, l.second));
    }
    int* h = s->sched_h[k];
    int o = 0;
    for (int g = 0; g < G; ++g) {
        h[g] = o;
        for (int idx : mine[g]) h[G + 1 + o++] = idx;
    }
    h[G] = o;
    if (cudaMemcpyAsync(s->sched_d[k], h, need * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) return nullptr;
    cudaEventRecord(s->sched_copied[k], c->stream);
    c->cnt.h2d_bytes += need * 4;
    s->sched_next = k ^ 1;
    return s->sched_d[k];
}

template <int HD>
cudaError_t prepare_kernel(PassState* s, int smem) {
    cudaError_t e = cudaFuncSetAttribute(pp::pass_kernel<HD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, pp::pass_kernel<HD>, pp::THREADS, smem);
    if (e != cudaSuccess) return e;
    return per_sm >= 1 ? cudaSuccess : cudaErrorCooperativeLaunchTooLarge;
}
int stages_for(const PassState* s, int T, int hd) {
    long avail = (long)s->max_smem - 1024 - (long)att::attn_tiles_bytes(hd) - (long)pp::misc_bytes();
    return (int)std::min<long>(12, avail / (long)pp::stage_bytes(T));
}
int fail_alloc(s2d2_ctx* c) {
    c->err = "cudaMalloc failed for the persistent pass";
    return S2D2_ERR_CUDA;
}
}  // namespace

int pass_init(s2d2_ctx* c) {
    PassState* s = new PassState();
    c->pass_state = s;
    const s2d2_model_config& m = c->m;
    if (m.dtype != S2D2_DTYPE_BF16 || (c->dc.use_tensor_cores != 1 && c->dc.use_tensor_cores != 3) || !gemm_tc_available(c)) return S2D2_OK;
    const bool moe = m.n_experts > 0;
    const int d = m.d_model, hd = m.head_dim, nq = m.n_q_heads * hd, nqkv = (m.n_q_heads + 2 * m.n_kv_heads) * hd;
    const int fe = m.expert_ffn, fs = moe ? m.expert_ffn * m.n_shared : 0, E = m.n_experts;
    const int f = moe ? fs : m.ffn;                 // width of the dense / shared-expert SwiGLU
    if (!(hd == 64 || hd == 128) || d % 128 || f % 128 || f < 128 || nqkv % 128 || nq % 64 || c->page_tokens < 16) return S2D2_OK;
    if (moe && (E % 128 || E > pp::MAX_EXPERTS || fe % 128 || m.top_k > 32 || m.top_k < 1 || m.n_shared < 1)) return S2D2_OK;
    if (c->max_rows < pp::MAX_T) return S2D2_OK;
    int coop = 0, n_sms = 0, optin = 0;
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device);
    cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, c->device);
    cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, c->device);
    if (!coop || n_sms < 1) return S2D2_OK;
    s->grid = n_sms;
    s->max_smem = optin;
    s->moe = moe;
    const int G = s->grid;
    if (stages_for(s, pp::MAX_T, hd) < 3) return S2D2_OK;
    cudaError_t e = hd == 128 ? prepare_kernel<128>(s, optin) : prepare_kernel<64>(s, optin);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return S2D2_OK;       // the one-kernel-per-operation path stays in charge
    }
    // ---- tensor maps: weights [layer][maps_per_layer], LM head, activations per T, KV pool ----
    const int L = m.n_layers;
    s->maps_per_layer = moe ? 8 : 4;
    s->barriers_per_layer = moe ? 9 : 6;
    s->map_x0 = L * s->maps_per_layer + 1;
    s->map_act_e = s->map_x0 + 40;
    s->map_kv = s->map_act_e + 8;
    std::vector<CUtensorMap> maps(s->map_kv + 5);      // KV pool, then q (high and low halves) and this pass's K and V rows as [row, head, head_dim] for the attention items
    auto enc = [&](int idx, const void* ptr, unsigned long long rows, int cols, int box_rows) {
        return gemm_encode_map(c, &maps[idx], ptr, rows, cols, box_rows) == 0;
    };
    bool good = true;
    for (int l = 0; l < L && good; ++l) {
        const LayerWeights& W = c->layers[l];
        const int b = l * s->maps_per_layer;
        good = enc(b + 0, W.wqkv, nqkv, d, 128) && enc(b + 1, W.wo, d, nq, 128);
        s->weight_bytes += 2.0 * ((double)nqkv * d + (double)d * nq);
        if (!moe) {
            good = good && enc(b + 2, W.wgu, 2 * f, d, 128) && enc(b + 3, W.wdown, d, f, 128);
            s->weight_bytes += 2.0 * (3.0 * f * d);
        } else {
            good = good && enc(b + 2, W.router, E, d, 128) && enc(b + 3, W.s_gu, 2 * fs, d, 128) &&
                   enc(b + 4, W.e_gate, (unsigned long long)E * fe, d, 128) && enc(b + 5, W.e_up, (unsigned long long)E * fe, d, 128) &&
                   enc(b + 6, W.s_down, d, fs, 128) && enc(b + 7, W.e_down, (unsigned long long)E * d, fe, 128);
            s->weight_bytes += 2.0 * ((double)E * d + 3.0 * fs * d);
        }
    }
    s->expert_bytes = 2.0 * 3.0 * fe * d;
    good = good && enc(L * s->maps_per_layer, c->lm_head, m.vocab, d, 128);
    s->head_bytes = 2.0 * (double)m.vocab * d;
    {
        size_t rows = c->max_rows;
        if (cudaMalloc((void**)&s->xn_lo, rows * d * 2) != cudaSuccess || cudaMalloc((void**)&s->attn_lo, rows * nq * 2) != cudaSuccess ||
            cudaMalloc((void**)&s->act_lo, rows * f * 2) != cudaSuccess || cudaMalloc((void**)&s->q_lo, rows * nq * 2) != cudaSuccess ||
            cudaMalloc((void**)&s->xn_b, rows * d * 2) != cudaSuccess || cudaMalloc((void**)&s->xn_b_lo, rows * d * 2) != cudaSuccess)
            return fail_alloc(c);
        cudaMemset(s->xn_b, 0, rows * d * 2);
        cudaMemset(s->xn_b_lo, 0, rows * d * 2);
        cudaMemset(s->xn_lo, 0, rows * d * 2);
        cudaMemset(s->attn_lo, 0, rows * nq * 2);
        cudaMemset(s->act_lo, 0, rows * f * 2);
        cudaMemset(s->q_lo, 0, rows * nq * 2);
        if (moe) {
            // SwiGLU outputs of the touched experts: [expert slot][T rows][fe]
            size_t bytes = (size_t)E * pp::MAX_T * fe * 2;
            if (cudaMalloc((void**)&s->act_e, bytes) != cudaSuccess || cudaMalloc((void**)&s->act_e_lo, bytes) != cudaSuccess ||
                cudaMalloc((void**)&s->n_touched, L * 4) != cudaSuccess || cudaMallocHost((void**)&s->n_touched_h, L * 4) != cudaSuccess)
                return fail_alloc(c);
            cudaMemset(s->act_e, 0, bytes);
            cudaMemset(s->act_e_lo, 0, bytes);
            cudaMemset(s->n_touched, 0, L * 4);
            memset(s->n_touched_h, 0, L * 4);
        }
    }
    for (int t = 0; t < 4 && good; ++t) {
        const int T = 16 * (t + 1);
        good = enc(s->map_x0 + t, c->xn, c->max_rows, d, T) && enc(s->map_x0 + 4 + t, c->attn, c->max_rows, nq, T) &&
               enc(s->map_x0 + 8 + t, c->act, c->max_rows, f, T) && enc(s->map_x0 + 12 + t, s->xn_lo, c->max_rows, d, T) &&
               enc(s->map_x0 + 16 + t, s->attn_lo, c->max_rows, nq, T) && enc(s->map_x0 + 20 + t, s->act_lo, c->max_rows, f, T) &&
               enc(s->map_x0 + 24 + t, s->xn_b, c->max_rows, d, T) && enc(s->map_x0 + 36 + t, s->xn_b_lo, c->max_rows, d, T);
        if (moe && good)
            good = enc(s->map_act_e + t, s->act_e, (unsigned long long)E * pp::MAX_T, fe, T) &&
                   enc(s->map_act_e + 4 + t, s->act_e_lo, (unsigned long long)E * pp::MAX_T, fe, T);
    }
    if (!good) {
        c->err = "cuTensorMapEncodeTiled failed for the persistent pass";
        return S2D2_ERR_CUDA;
    }
    {   // the KV pool map is the attention kernel's
        PassView dummy{};
        dummy.n_seqs = 1;
        att::AttnParams ap;
        const void* mk = nullptr;
        if (!attention_plan(c, dummy, 1, 1, 0, &ap, &mk) || !mk) return S2D2_OK;
        maps[s->map_kv] = *(const CUtensorMap*)mk;
    }
    {
        // A tile of 64 query vectors of one kv head is a box of (64 / group) rows x group heads: TMA writes it in query order
        const int group = m.n_q_heads / m.n_kv_heads;
        s->q_by_tma = m.head_dim == 128 && att::QT % group == 0 && group <= att::QT;
        if (s->q_by_tma)
            s->q_by_tma = gemm_encode_map3(c, &maps[s->map_kv + 1], c->q, m.head_dim, m.n_q_heads, c->max_rows, group, att::QT / group) == 0 &&
                          gemm_encode_map3(c, &maps[s->map_kv + 2], s->q_lo, m.head_dim, m.n_q_heads, c->max_rows, group, att::QT / group) == 0 &&
                          gemm_encode_map3(c, &maps[s->map_kv + 3], c->k_rows, m.head_dim, m.n_kv_heads, c->max_rows, 1, 64) == 0 &&
                          gemm_encode_map3(c, &maps[s->map_kv + 4], c->v_rows, m.head_dim, m.n_kv_heads, c->max_rows, 1, 64) == 0;
    }
    // ---- per GEMM kind: shape, split-K workspace region, publish counters, part tables ----
    // N < 0 marks a kind this model does not run; for the two routed-expert GEMMs N is the largest (all experts touched).
    long long NK[pp::N_KINDS][2];
    for (auto& nk : NK) nk[0] = -1, nk[1] = 64;
    NK[pp::K_QKV][0] = nqkv, NK[pp::K_QKV][1] = d;
    NK[pp::K_O][0] = d, NK[pp::K_O][1] = nq;
    NK[pp::K_LM][0] = m.vocab, NK[pp::K_LM][1] = d;
    if (!moe) {
        NK[pp::K_GU][0] = 2LL * f, NK[pp::K_GU][1] = d;
        NK[pp::K_DOWN][0] = d, NK[pp::K_DOWN][1] = f;
    } else {
        NK[pp::K_ROUTER][0] = E, NK[pp::K_ROUTER][1] = d;
        NK[pp::K_SGU][0] = 2LL * fs, NK[pp::K_SGU][1] = d;
        NK[pp::K_EGU][0] = 2LL * fe * E, NK[pp::K_EGU][1] = d;
        NK[pp::K_SDOWN][0] = d, NK[pp::K_SDOWN][1] = fs;
        NK[pp::K_EDOWN][0] = (long long)d * E, NK[pp::K_EDOWN][1] = fe;
    }
    // ---- sub-GEMMs of every kind (see pp::SubDesc) ----
    // Dense layers: O finishes its first half of output tiles early; gate/up starts with the k-blocks that half
    // feeds and finishes the first half of the SwiGLU columns early; down starts with those and finishes its first
    // half of tiles early; the next layer's QKV starts with the k-blocks they feed.  A GEMM is only cut where every
    // sub-GEMM still gives each CTA a few units; otherwise (small models, mixture-of-experts kinds) it stays whole.
    // use_tensor_cores = 3 cuts wherever the tile counts allow (test setting); when a small model then ends up with more
    // split-K parts per tile than the part lists hold, the next, more conservative threshold is taken
    const int min_units_options[3] = {c->dc.use_tensor_cores == 3 ? 0 : 4, c->dc.use_tensor_cores == 3 ? 1 : 4, 1 << 30};
    long long ws_floats = 0;
    size_t sync_words = 64;
    for (int attempt = 0; attempt < 3; ++attempt) {
    bool parts_fit = true;
    {
        const int MIN_UNITS = min_units_options[attempt];
        auto whole = [&](int k) {
            const int n_tiles = (int)((NK[k][0] + 127) / 128), kbt = (int)(NK[k][1] / 64);
            s->n_subs[k] = 1;
            s->subs[k][0] = pp::SubDesc{0, n_tiles, n_tiles, 0, 0, kbt, 0, 0, k == pp::K_GU || k == pp::K_SGU ? n_tiles / 2 : n_tiles};
        };
        for (int k = 0; k < pp::N_KINDS; ++k)
            if (NK[k][0] >= 0) whole(k);
        if (!moe) {
            const int dt = d / 128, ft = f / 128, h = dt / 2, hd = dt / 2;
            auto enough = [&](long long units) { return units / G >= MIN_UNITS; };
            const int kq = d / 64, ko = nq / 64, kd = f / 64, tq = nqkv / 128;
            // O stays whole unless the test setting forces cuts: it is small (14 units per CTA on the 8B-class shape), halves
            // of it leave 18 split-K parts per tile, and the 8B-class pass measured no faster with it cut (3.70 against 3.61 ms)
            const bool o_split = c->dc.use_tensor_cores == 3 && h >= 1 && enough((long long)h * ko) && enough((long long)(dt - h) * ko);
            if (o_split) {                                   // (H0, all K), (H1, all K)
                s->n_subs[pp::K_O] = 2;
                s->subs[pp::K_O][0] = pp::SubDesc{0, h, h, 0, 0, ko, 0, 0, h};
                s->subs[pp::K_O][1] = pp::SubDesc{h, dt - h, dt - h, 0, 0, ko, 0, h, dt};
            }
            // gate/up: its SwiGLU columns in nh groups that complete one after the other, so that the element-wise
            // chain behind a group (partials published, summed, activated, counted, fetched by the next GEMM) runs
            // under the groups that follow; down: the k-blocks those groups feed, in the same order, its own output
            // tiles in two groups during the last of them.  Two groups: every group boundary is a point where all
            // CTAs wait for the slowest one's partials, and with three groups (measured on the 8B-class shape: 107 us per
            // layer against 100) the added waits cost more than the shorter chains gain.
            const int k0 = o_split ? 2 * h : 0;              // gate/up k-blocks fed by O's first half run first, over all tiles
            int nh = 1;
            for (int cand = 2; cand >= 2 && nh == 1; --cand) {
                if (ft < cand) continue;
                bool fits = k0 == 0 || enough(2LL * ft * k0);
                for (int i = 0; i < cand && fits; ++i) {
                    const int a = ft * i / cand, b2 = ft * (i + 1) / cand;
                    fits = enough(2LL * (b2 - a) * (kq - k0));
                }
                if (fits) nh = cand;
            }
            if (nh > 1) {
                int n = 0;
                if (k0 > 0) s->subs[pp::K_GU][n++] = pp::SubDesc{0, 2 * ft, 2 * ft, 0, 0, k0, 0, 0, 0};
                auto gu_a = [&](int i) { return ft * i / nh; };
                auto gu_b = [&](int i) { return ft * (i + 1) / nh; };
                for (int i = 0; i < nh; ++i) {
                    const int a = gu_a(i), b2 = gu_b(i);
                    s->subs[pp::K_GU][n++] = pp::SubDesc{a, 2 * (b2 - a), b2 - a, ft, k0, kq - k0, 0, a, b2};
                }
                s->n_subs[pp::K_GU] = n;
                // down: k-blocks of group i = SwiGLU columns [128 a_i, 128 b_i)
                bool three_way = hd >= 1 && hd < dt;         // last group's k-blocks over two groups of output tiles
                for (int i = 0; i < nh && three_way; ++i) {
                    const int a = gu_a(i), b2 = gu_b(i);
                    three_way = i + 1 < nh ? enough((long long)dt * 2 * (b2 - a)) : (enough((long long)hd * 2 * (b2 - a)) && enough((long long)(dt - hd) * 2 * (b2 - a)));
                }
                bool k_only = !three_way;
                for (int i = 0; i < nh && k_only; ++i) k_only = enough((long long)dt * 2 * (gu_b(i) - gu_a(i)));
                if (three_way || k_only) {
                    n = 0;
                    for (int i = 0; i < nh; ++i) {
                        const int a = gu_a(i), b2 = gu_b(i);
                        if (i + 1 < nh || k_only) {
                            s->subs[pp::K_DOWN][n++] = pp::SubDesc{0, dt, dt, 0, 2 * a, 2 * (b2 - a), 0, 0, i + 1 < nh ? 0 : dt};
                        } else {
                            s->subs[pp::K_DOWN][n++] = pp::SubDesc{0, hd, hd, 0, 2 * a, 2 * (b2 - a), 0, 0, hd};
                            s->subs[pp::K_DOWN][n++] = pp::SubDesc{hd, dt - hd, dt - hd, 0, 2 * a, 2 * (b2 - a), 0, hd, dt};
                        }
                    }
                    s->n_subs[pp::K_DOWN] = n;
                }
                if (three_way && enough((long long)tq * 2 * hd) && enough((long long)tq * (kq - 2 * hd))) {      // (all, K0), (all, K1): K0 = what down's first group feeds
                    s->n_subs[pp::K_QKV] = 2;
                    s->subs[pp::K_QKV][0] = pp::SubDesc{0, tq, tq, 0, 0, 2 * hd, 0, 0, 0};
                    s->subs[pp::K_QKV][1] = pp::SubDesc{0, tq, tq, 0, 2 * hd, kq - 2 * hd, 0, 0, tq};
                }
            }
        }
    }
    // ---- per GEMM kind: split-K workspace region, publish counters, part tables ----
    ws_floats = 0;
    sync_words = 64;
    for (int k = 0; k < pp::N_KINDS && parts_fit; ++k) {
        s->cnt_off[k] = -1;
        if (NK[k][0] < 0) continue;
        const bool dynamic = k == pp::K_EGU || k == pp::K_EDOWN;
        const long long n_tiles_all = (NK[k][0] + 127) / 128;
        int segs = 0;
        for (int sb = 0; sb < s->n_subs[k]; ++sb) {
            pp::SubDesc& sd = s->subs[k][sb];
            const long long U = (long long)sd.nt * sd.nkb;
            if (U * (long long)G >= (1LL << 40)) return S2D2_OK;
            // the kernel shares a sub-GEMM's units among Geff CTAs (pp::effective_ctas); for the routed-expert GEMMs the
            // largest per-CTA share is that of the largest U, since Geff only grows with U
            const int Geff = pp::effective_ctas(U, sd.nkb, G);
            const long long per = (U + Geff - 1) / Geff;
            sd.seg_base = segs;
            segs += (int)((per + sd.nkb - 1) / sd.nkb + 1);
        }
        s->max_segs[k] = segs;
        s->ws_off[k] = ws_floats;
        ws_floats += (long long)G * s->max_segs[k] * pp::MAX_T * 128;
        if (dynamic) continue;
        s->cnt_off[k] = (long long)sync_words;
        sync_words += (size_t)n_tiles_all;
        // per weight tile: the workspace slots of its split-K partials, sub-GEMM by sub-GEMM and in CTA order inside
        // each (the kernel cuts a sub-GEMM's tile-major (tile, k-block) units into Geff equal contiguous ranges)
        std::vector<int> tab((size_t)n_tiles_all * (1 + pp::MAX_PARTS), 0);
        for (int sb = 0; sb < s->n_subs[k]; ++sb) {
            const pp::SubDesc& sd = s->subs[k][sb];
            const long long U = (long long)sd.nt * sd.nkb;
            const int Geff = pp::effective_ctas(U, sd.nkb, G);
            for (int cta = 0; cta < Geff; ++cta) {
                const long long u0 = U * cta / Geff, u1 = U * (cta + 1) / Geff;
                if (u1 <= u0) continue;
                const long long first = u0 / sd.nkb, last = (u1 - 1) / sd.nkb;
                for (long long tl = first; tl <= last; ++tl) {
                    const long long t = tl < sd.t_split ? sd.t0 + tl : sd.t0 + sd.t_jump + (tl - sd.t_split);
                    int& cnt = tab[(size_t)t * (1 + pp::MAX_PARTS)];
                    if (cnt >= pp::MAX_PARTS) {       // too finely split for the tables
                        parts_fit = false;
                        break;
                    }
                    tab[(size_t)t * (1 + pp::MAX_PARTS) + 1 + cnt] = cta * s->max_segs[k] + sd.seg_base + (int)(tl - first);
                    ++cnt;
                }
            }
        }
        if (!parts_fit) break;
        if (s->parts[k]) cudaFree(s->parts[k]);
        s->parts[k] = nullptr;
        if (cudaMalloc((void**)&s->parts[k], tab.size() * 4) != cudaSuccess ||
            cudaMemcpy(s->parts[k], tab.data(), tab.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)
            return fail_alloc(c);
    }
    if (parts_fit) break;
    if (attempt == 2) return S2D2_OK;       // even whole GEMMs are split too finely for the tables: the per-operation path stays in charge
    }
    if (!moe) {
        // Static schedule of a dense model: what each CTA streams does not depend on the data, so the list of its
        // segments (one weight tile times a range of k-blocks, in execution order) is made here once; the producer
        // and MMA threads then walk a table instead of recomputing unit ranges with 64-bit divisions per GEMM.
        const int order[4] = {pp::K_QKV, pp::K_O, pp::K_GU, pp::K_DOWN};
        std::vector<std::vector<int4>> per_cta(G);
        std::vector<std::vector<int>> begins(G);
        auto add_kind = [&](int k) {
            for (int sb = 0; sb < s->n_subs[k]; ++sb) {
                const pp::SubDesc& sd = s->subs[k][sb];
                const long long U = (long long)sd.nt * sd.nkb;
                const int Geff = pp::effective_ctas(U, sd.nkb, G);
                for (int cta = 0; cta < G; ++cta) {
                    begins[cta].push_back((int)per_cta[cta].size());
                    if (cta >= Geff) continue;
                    long long u = U * cta / Geff;
                    const long long u1 = U * (cta + 1) / Geff;
                    const long long first = u / sd.nkb;
                    while (u < u1) {
                        const long long tl = u / sd.nkb;
                        const int kb0 = (int)(u - tl * sd.nkb);
                        const int kb1 = (int)std::min<long long>(sd.nkb, kb0 + (u1 - u));
                        const long long t = tl < sd.t_split ? sd.t0 + tl : sd.t0 + sd.t_jump + (tl - sd.t_split);
                        const int slot = sd.seg_base + (int)(tl - first);
                        int4 e;
                        e.x = k | (sb << 8) | (slot << 16);
                        e.y = (int)(t * 128);
                        e.z = (sd.kb0 + kb0) | ((kb1 - kb0) << 16);
                        e.w = (int)t;
                        per_cta[cta].push_back(e);
                        u += kb1 - kb0;
                    }
                }
            }
        };
        for (int k : order) add_kind(k);
        s->n_layer_subs = s->n_subs[pp::K_QKV] + s->n_subs[pp::K_O] + s->n_subs[pp::K_GU] + s->n_subs[pp::K_DOWN];
        add_kind(pp::K_LM);
        s->n_lm_subs = s->n_subs[pp::K_LM];
        size_t stride = 1;
        for (int cta = 0; cta < G; ++cta) {
            begins[cta].push_back((int)per_cta[cta].size());
            stride = std::max(stride, per_cta[cta].size());
        }
        s->seg_stride = (int)stride;
        const int nb = s->n_layer_subs + s->n_lm_subs + 1;
        std::vector<int4> flat((size_t)G * stride, int4{0, 0, 0, 0});
        std::vector<int> fb((size_t)G * nb);
        for (int cta = 0; cta < G; ++cta) {
            std::copy(per_cta[cta].begin(), per_cta[cta].end(), flat.begin() + (size_t)cta * stride);
            std::copy(begins[cta].begin(), begins[cta].end(), fb.begin() + (size_t)cta * nb);
        }
        if (cudaMalloc((void**)&s->segs, flat.size() * sizeof(int4)) != cudaSuccess ||
            cudaMalloc((void**)&s->seg_sub_begin, fb.size() * 4) != cudaSuccess ||
            cudaMemcpy(s->segs, flat.data(), flat.size() * sizeof(int4), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(s->seg_sub_begin, fb.data(), fb.size() * 4, cudaMemcpyHostToDevice) != cudaSuccess)
            return fail_alloc(c);
    }
    {
        const long long Xs[4] = {d, nq, f, d};       // columns of xn, attn, act, xn_b
        for (int k = 0; k < 4; ++k) {
            s->xcnt_off[k] = sync_words;
            sync_words += (size_t)((Xs[k] + 127) / 128);
        }
        s->attn_cnt_off = sync_words;       // per (sequence, kv head, query tile) of a pass: at most 64 sequences x query heads
        sync_words += (size_t)pp::MAX_T * m.n_q_heads;
        s->sync_bytes = sync_words * 4;
        if (cudaMalloc((void**)&s->barrier, s->sync_bytes) != cudaSuccess) return fail_alloc(c);
    }
    std::vector<pp::LayerGains> gains(L);
    for (int l = 0; l < L; ++l) gains[l] = {c->layers[l].attn_norm, c->layers[l].ffn_norm, c->layers[l].q_norm, c->layers[l].k_norm};
    size_t ssq_bytes = (size_t)(d / 128) * pp::MAX_T * 4;
    {
        int spl = 0;      // sub-GEMMs per layer, and the LM head's
        const int dense_kinds[4] = {pp::K_QKV, pp::K_O, pp::K_GU, pp::K_DOWN};
        const int moe_kinds[7] = {pp::K_QKV, pp::K_O, pp::K_ROUTER, pp::K_SGU, pp::K_EGU, pp::K_SDOWN, pp::K_EDOWN};
        for (int j = 0; j < (moe ? 7 : 4); ++j) spl += s->n_subs[moe ? moe_kinds[j] : dense_kinds[j]];
        s->n_sub_gemms = spl * L + s->n_subs[pp::K_LM];
    }
    s->trace_mma0 = 3 + (moe ? 27 : 12) * L + 2;
    s->trace_cap = s->trace_mma0 + 6 * s->n_sub_gemms + 1;      // embedding barrier, per-layer marks, LM-head phase, two per sub-GEMM, the SM id
    if (cudaMalloc((void**)&s->trace, (size_t)G * s->trace_cap * 8) != cudaSuccess) return fail_alloc(c);
    if (cudaMalloc((void**)&s->d_maps, maps.size() * sizeof(CUtensorMap)) != cudaSuccess ||
        cudaMalloc((void**)&s->d_gains, gains.size() * sizeof(pp::LayerGains)) != cudaSuccess ||
        cudaMalloc((void**)&s->ws, (size_t)ws_floats * 4) != cudaSuccess || cudaMalloc((void**)&s->ssq_a, ssq_bytes) != cudaSuccess ||
        cudaMalloc((void**)&s->ssq_b, ssq_bytes) != cudaSuccess)
        return fail_alloc(c);
    if (cudaMemcpy(s->d_maps, maps.data(), maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(s->d_gains, gains.data(), gains.size() * sizeof(pp::LayerGains), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemset(s->ws, 0, (size_t)ws_floats * 4) != cudaSuccess) {
        c->err = "device copy failed for the persistent pass";
        return S2D2_ERR_CUDA;
    }
    // rows past the pass's own rows ride along as unused MMA columns: keep them finite
    size_t es = 2;
    cudaMemset(c->xn, 0, (size_t)c->max_rows * d * es);
    cudaMemset(c->attn, 0, (size_t)c->max_rows * nq * es);
    cudaMemset(c->q, 0, (size_t)c->max_rows * nq * es);       // a Q tile fetched by TMA covers 64 / group rows, also past the sequence's own
    cudaMemset(c->k_rows, 0, (size_t)c->max_rows * m.n_kv_heads * m.head_dim * es);      // likewise the 64 in-pass key rows
    cudaMemset(c->v_rows, 0, (size_t)c->max_rows * m.n_kv_heads * m.head_dim * es);
    cudaMemset(c->act, 0, (size_t)c->max_rows * f * es);
    s->ok = true;
    return S2D2_OK;
}

int pass_max_rows(s2d2_ctx* c) {
    PassState* s = state(c);
    return s && s->ok ? pp::MAX_T : 0;
}

void pass_destroy(s2d2_ctx* c) {
    PassState* s = state(c);
    if (!s) return;
    void* ptrs[] = {s->d_maps, s->d_gains, s->ws, s->ssq_a, s->ssq_b, s->barrier, s->trace, s->xn_lo, s->attn_lo, s->act_lo, s->q_lo,
                    s->act_e, s->act_e_lo, s->n_touched, s->xn_b, s->xn_b_lo, s->segs, s->seg_sub_begin};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (int* p : s->parts)
        if (p) cudaFree(p);
    if (s->n_touched_h) cudaFreeHost(s->n_touched_h);
    for (int k = 0; k < 2; ++k) {
        if (s->sched_h[k]) cudaFreeHost(s->sched_h[k]);
        if (s->sched_d[k]) cudaFree(s->sched_d[k]);
        if (s->sched_copied[k]) cudaEventDestroy(s->sched_copied[k]);
    }
    delete s;
    c->pass_state = nullptr;
}

int pass_run(s2d2_ctx* c, const PassView& pv, int max_ctx, int max_rows, long long sum_ctx, float* logits_out, bool* taken) {
    *taken = false;
    PassState* s = state(c);
    const s2d2_model_config& m = c->m;
    if (!s || !s->ok || pv.n_rows < 1 || pv.n_rows > pp::MAX_T) return S2D2_OK;
    pp::PassParams p{};      // every field starts from zero; the ones a pass needs are set below
    // several sequences: finer key splits (about two items per CTA), dealt out by cost
    if (!attention_plan(c, pv, max_ctx, max_rows, pv.n_seqs > 1 ? 2 * s->grid : s->grid, &p.ap, nullptr)) return S2D2_OK;
    if (pv.n_seqs > 1) {
        const int* sched = attention_schedule(c, s, p.ap);
        if (sched) {
            p.ap.sched_off = sched;
            p.ap.sched_items = sched + s->grid + 1;
        }
    }
    p.n_layers = m.n_layers;
    p.d = m.d_model;
    p.Hq = m.n_q_heads;
    p.Hkv = m.n_kv_heads;
    p.hd = m.head_dim;
    p.moe = s->moe;
    p.n_experts = m.n_experts;
    p.top_k = m.top_k;
    p.fe = m.expert_ffn;
    p.fs = s->moe ? m.expert_ffn * m.n_shared : 0;
    p.f = s->moe ? p.fs : m.ffn;
    p.maps_per_layer = s->maps_per_layer;
    p.V = m.vocab;
    p.qk_norm = m.qk_norm;
    p.eps = m.rms_eps;
    p.logit_scale = m.logit_scale;
    p.pv = pv;
    p.M = pv.n_rows;
    p.T = (pv.n_rows + 15) / 16 * 16;
    p.n_logit = logits_out ? pv.n_logit_rows : 0;
    p.embed = (const bf16*)c->embed;
    p.gains = s->d_gains;
    p.final_norm = c->final_norm;
    p.h = c->h;
    p.xn = (bf16*)c->xn;
    p.q = (bf16*)c->q;
    p.k_rows = (bf16*)c->k_rows;
    p.v_rows = (bf16*)c->v_rows;
    p.attn = (bf16*)c->attn;
    p.act = (bf16*)c->act;
    p.xn_lo = s->xn_lo;
    p.xn_b = s->xn_b;
    p.xn_b_lo = s->xn_b_lo;
    p.attn_lo = s->attn_lo;
    p.act_lo = s->act_lo;
    p.map_lo_off = 12;
    p.q_lo = s->q_lo;
    p.ap.q_lo = s->q_lo;
    p.ws = s->ws;
    for (int k = 0; k < pp::N_KINDS; ++k) {
        p.ws_off[k] = s->ws_off[k];
        p.max_segs[k] = s->max_segs[k];
        p.parts[k] = s->parts[k];
        p.tile_cnt[k] = s->cnt_off[k] >= 0 ? s->barrier + s->cnt_off[k] : nullptr;
        p.n_subs[k] = s->n_subs[k];
        for (int sb = 0; sb < pp::MAX_SUBS; ++sb) p.subs[k][sb] = s->subs[k][sb];
    }
    p.acc_stride = p.T <= 16 ? 32 : (p.T <= 32 ? 64 : 128);
    p.n_acc = pp::ACC_COLS / p.acc_stride;
    p.act_e = s->act_e;
    p.act_e_lo = s->act_e_lo;
    p.moe_ids = c->moe_ids;
    p.moe_gates = c->moe_gates;
    p.moe_ids_trace = c->moe_ids_trace;
    p.trace_stride = c->max_rows * std::max(1, m.top_k);
    p.n_touched_out = s->n_touched;
    p.ssq_a = s->ssq_a;
    p.ssq_b = s->ssq_b;
    p.logits = logits_out;
    p.rope_cos = c->rope_cos;
    p.rope_sin = c->rope_sin;
    p.pool.base = (bf16*)c->kv_base;
    p.pool.page_tokens = c->page_tokens;
    p.pool.page_shift = c->page_shift;
    p.pool.n_kv_heads = m.n_kv_heads;
    p.pool.head_dim = m.head_dim;
    p.pool.page_stride = (size_t)2 * m.n_kv_heads * c->page_tokens * m.head_dim;
    p.pool.layer_stride = (size_t)c->n_pages * p.pool.page_stride;
    p.maps = s->d_maps;
    const int ti = p.T / 16 - 1;
    p.map_xn = s->map_x0 + ti;
    p.map_xn_b = s->map_x0 + 24 + ti;
    p.map_attn = s->map_x0 + 4 + ti;
    p.map_act = s->map_x0 + 8 + ti;
    p.map_act_e = s->map_act_e + ti;
    p.map_kv = s->map_kv;
    p.map_q = s->q_by_tma ? s->map_kv + 1 : -1;
    p.barrier = s->barrier;
    p.status = c->d_status;
    p.S = stages_for(s, p.T, m.head_dim);
    p.trace = c->tracing ? s->trace : nullptr;
    p.trace_cap = s->trace_cap;
    p.trace_mma0 = s->trace_mma0;
    p.trace_n_sub = s->n_sub_gemms;
    p.segs = s->segs;
    p.seg_sub_begin = s->seg_sub_begin;
    p.seg_stride = s->seg_stride;
    p.n_layer_subs = s->n_layer_subs;
    p.n_lm_subs = s->n_lm_subs;
    if (c->tracing) {
        s->last_marks = s->trace_cap - 1;
        cudaMemsetAsync(s->trace, 0, (size_t)s->grid * s->trace_cap * 8, c->stream);
    }
    size_t smem = pp::smem_bytes(p.T, p.S, m.head_dim);
    if (cudaMemsetAsync(s->barrier, 0, s->sync_bytes, c->stream) != cudaSuccess) return S2D2_ERR_CUDA;
    for (int k = 0; k < 4; ++k) p.x_cnt[k] = s->barrier + s->xcnt_off[k];
    p.attn_cnt = s->barrier + s->attn_cnt_off;
    void* args[] = {&p};
    gemm_prof_begin(c);
    cudaError_t e = m.head_dim == 128
                        ? cudaLaunchCooperativeKernel((void*)pp::pass_kernel<128>, dim3(s->grid), dim3(pp::THREADS), args, smem, c->stream)
                        : cudaLaunchCooperativeKernel((void*)pp::pass_kernel<64>, dim3(s->grid), dim3(pp::THREADS), args, smem, c->stream);
    // algorithmic bytes of the pass: every matrix once (for routed experts: those the previous pass of this
    // context touched, the closest count the host has without a read-back), the cached K/V of every sequence
    // once, this pass's K/V rows written, logits written
    double kv_tok = 2.0 * m.n_layers * m.n_kv_heads * m.head_dim * 2.0;
    double bytes = s->weight_bytes + (p.n_logit > 0 ? s->head_bytes + 4.0 * p.n_logit * m.vocab : 0.0) + kv_tok * (double)sum_ctx +
                   kv_tok * pv.n_rows;
    if (s->moe) {
        long long touched = 0;
        for (int l = 0; l < m.n_layers; ++l) touched += s->n_touched_h[l];
        bytes += s->expert_bytes * (double)touched;
        c->cnt.moe_expert_tiles_touched += touched;
        cudaMemcpyAsync(s->n_touched_h, s->n_touched, m.n_layers * 4, cudaMemcpyDeviceToHost, c->stream);
    }
    gemm_prof_end(c, bytes);
    if (e != cudaSuccess) {
        c->err = std::string("persistent pass launch: ") + cudaGetErrorString(e);
        return S2D2_ERR_CUDA;
    }
    c->cnt.n_kernel_launches++;
    c->last_pass_rows = pv.n_rows;
    *taken = true;
    return S2D2_OK;
}

int pass_copy_trace(s2d2_ctx* c, unsigned long long* out, long long cap, int* n_ctas, int* n_marks) {
    PassState* s = state(c);
    if (!s || !s->ok || s->last_marks == 0) {
        c->err = "no persistent pass has run";
        return S2D2_ERR_STATE;
    }
    if (cap < (long long)s->grid * (s->last_marks + 1)) {
        c->err = "trace buffer too small";
        return S2D2_ERR_INVALID;
    }
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return S2D2_ERR_CUDA;
    const size_t row = (size_t)s->last_marks + 1;
    for (int g = 0; g < s->grid; ++g)
        if (cudaMemcpy(out + g * row, s->trace + (size_t)g * s->trace_cap, (size_t)s->last_marks * 8, cudaMemcpyDeviceToHost) !=
                cudaSuccess ||
            cudaMemcpy(out + g * row + s->last_marks, s->trace + (size_t)g * s->trace_cap + s->trace_cap - 1, 8,
                       cudaMemcpyDeviceToHost) != cudaSuccess)
            return S2D2_ERR_CUDA;
    *n_ctas = s->grid;
    *n_marks = s->last_marks;
    return S2D2_OK;
}
