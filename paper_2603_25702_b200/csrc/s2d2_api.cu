// C ABI and host driver of the S2D2 decode step (see include/s2d2.h).
//
// The host keeps the per-sequence decode state (tokens, open block, cache
// length, page list) and, for each pass, builds a small row table that the
// kernels read: which token sits at which position, which rows of the same pass
// a row may attend (a 64-bit mask: the verifier mask and the partially causal
// drafting mask both fit), which rows write their K/V to the cache, and which
// rows need logits.  Everything numerical runs in the kernels.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>

#include "context.h"
#include "attention.h"
#include "gemm.h"
#include "kernels_simt.cuh"
#include "pass.h"
#include "vocab_kernels.cuh"

using namespace s2d2;

#define CUDA_TRY(ctx, call)                                                                      \
    do {                                                                                         \
        cudaError_t e_ = (call);                                                                 \
        if (e_ != cudaSuccess) {                                                                 \
            (ctx)->err = std::string(#call) + ": " + cudaGetErrorString(e_);                     \
            return S2D2_ERR_CUDA;                                                                \
        }                                                                                        \
    } while (0)
#define FAIL(ctx, code, msg)  \
    do {                      \
        (ctx)->err = (msg);   \
        return (code);        \
    } while (0)
#define LAUNCHED(ctx) ((ctx)->cnt.n_kernel_launches++)

// Rows of a wide prefill pass (the activation scratch of every context has at least this many rows).
static constexpr int PREFILL_PASS_ROWS = 1024;

static size_t esize(int dtype) { return dtype == S2D2_DTYPE_BF16 ? 2 : 4; }
static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---------------------------------------------------------------------------------------------
// creation: weight arena layout, KV pool, scratch
// ---------------------------------------------------------------------------------------------
namespace {

struct ArenaPlan {
    size_t cur = 0;
    size_t take(size_t bytes) {
        size_t o = cur;
        cur = align_up(cur + bytes, 256);
        return o;
    }
};

void add_slot(s2d2_ctx* c, const std::string& name, char* base, size_t off, size_t bytes, int dtype) {
    WeightSlot s;
    s.d_ptr = base ? base + off : (void*)off;
    s.bytes = bytes;
    s.dtype = dtype;
    c->slots[name] = s;
}

// Lays the tensors out in one arena.  wq/wk/wv share one [Hq+2Hkv)*hd, d] matrix and
// w_gate/w_up one [2f, d] matrix so that one GEMM serves each group.
size_t plan_weights(s2d2_ctx* c, char* base) {
    const s2d2_model_config& m = c->m;
    ArenaPlan ap;
    size_t es = esize(m.dtype), d = m.d_model, hd = m.head_dim;
    c->slots.clear();
    c->layers.assign(m.n_layers, LayerWeights());
    size_t o = ap.take((size_t)(m.vocab + 1) * d * es);
    add_slot(c, "embed", base, o, (size_t)(m.vocab + 1) * d * es, m.dtype);
    c->embed = base + o;
    for (int l = 0; l < m.n_layers; ++l) {
        std::string p = "layers." + std::to_string(l) + ".";
        LayerWeights& L = c->layers[l];
        auto gain = [&](const char* n, size_t len, float** dst) {
            size_t off = ap.take(len * 4);
            add_slot(c, p + n, base, off, len * 4, S2D2_DTYPE_F32);
            *dst = (float*)(base + off);
        };
        gain("attn_norm", d, &L.attn_norm);
        size_t nq = (size_t)m.n_q_heads * hd, nkv = (size_t)m.n_kv_heads * hd;
        size_t off = ap.take((nq + 2 * nkv) * d * es);
        L.wqkv = base + off;
        add_slot(c, p + "wq", base, off, nq * d * es, m.dtype);
        add_slot(c, p + "wk", base, off + nq * d * es, nkv * d * es, m.dtype);
        add_slot(c, p + "wv", base, off + (nq + nkv) * d * es, nkv * d * es, m.dtype);
        off = ap.take(d * nq * es);
        L.wo = base + off;
        add_slot(c, p + "wo", base, off, d * nq * es, m.dtype);
        if (m.qk_norm) {
            gain("q_norm", hd, &L.q_norm);
            gain("k_norm", hd, &L.k_norm);
        }
        gain("ffn_norm", d, &L.ffn_norm);
        if (m.n_experts > 0) {
            size_t E = m.n_experts, f = m.expert_ffn;
            off = ap.take(E * d * es);
            L.router = base + off;
            add_slot(c, p + "router", base, off, E * d * es, m.dtype);
            off = ap.take(E * f * d * es);
            L.e_gate = base + off;
            add_slot(c, p + "experts.w_gate", base, off, E * f * d * es, m.dtype);
            off = ap.take(E * f * d * es);
            L.e_up = base + off;
            add_slot(c, p + "experts.w_up", base, off, E * f * d * es, m.dtype);
            off = ap.take(E * d * f * es);
            L.e_down = base + off;
            add_slot(c, p + "experts.w_down", base, off, E * d * f * es, m.dtype);
            if (m.n_shared > 0) {
                size_t fs = f * m.n_shared;
                off = ap.take(2 * fs * d * es);
                L.s_gu = base + off;
                add_slot(c, p + "shared.w_gate", base, off, fs * d * es, m.dtype);
                add_slot(c, p + "shared.w_up", base, off + fs * d * es, fs * d * es, m.dtype);
                off = ap.take(d * fs * es);
                L.s_down = base + off;
                add_slot(c, p + "shared.w_down", base, off, d * fs * es, m.dtype);
            }
        } else {
            size_t f = m.ffn;
            off = ap.take(2 * f * d * es);
            L.wgu = base + off;
            add_slot(c, p + "w_gate", base, off, f * d * es, m.dtype);
            add_slot(c, p + "w_up", base, off + f * d * es, f * d * es, m.dtype);
            off = ap.take(d * f * es);
            L.wdown = base + off;
            add_slot(c, p + "w_down", base, off, d * f * es, m.dtype);
        }
    }
    o = ap.take(d * 4);
    add_slot(c, "final_norm", base, o, d * 4, S2D2_DTYPE_F32);
    c->final_norm = (float*)(base + o);
    o = ap.take((size_t)m.vocab * d * es);
    add_slot(c, "lm_head", base, o, (size_t)m.vocab * d * es, m.dtype);
    c->lm_head = base + o;
    return ap.cur;
}

int validate(const s2d2_model_config& m, const s2d2_decode_config& dc, std::string& why) {
    auto bad = [&](const char* s) {
        why = s;
        return S2D2_ERR_INVALID;
    };
    if (m.n_layers < 1 || m.d_model < 32 || m.vocab < 2) return bad("model: n_layers/d_model/vocab");
    if (m.n_q_heads < 1 || m.n_kv_heads < 1 || m.n_q_heads % m.n_kv_heads) return bad("model: heads");
    if (m.head_dim != 32 && m.head_dim != 64 && m.head_dim != 128) return bad("model: head_dim must be 32, 64 or 128");
    if (m.dtype != S2D2_DTYPE_F32 && m.dtype != S2D2_DTYPE_BF16) return bad("model: dtype");
    if (m.n_experts == 0 && m.ffn < 1) return bad("model: ffn");
    if (m.n_experts > 0 && (m.top_k < 1 || m.top_k > m.n_experts || m.top_k > 32 || m.expert_ffn < 1))
        return bad("model: moe");
    if (dc.block_size < 1 || dc.block_size > S2D2_MAX_BLOCK) return bad("decode: block_size");
    if (dc.max_batch < 1 || dc.max_seq_len < 1) return bad("decode: max_batch/max_seq_len");
    int p = dc.kv_page_tokens;
    if (p < 1 || p > 64 || (p & (p - 1))) return bad("decode: kv_page_tokens must be a power of two <= 64");
    if (dc.draft_mode != S2D2_DRAFT_GREEDY && dc.draft_mode != S2D2_DRAFT_SAMPLE) return bad("decode: draft_mode");
    if (dc.verifier_layout != S2D2_VERIFIER_ALIGNED_2L && dc.verifier_layout != S2D2_VERIFIER_RIGHT_SHIFTED) return bad("decode: verifier_layout");
    if (dc.caching != S2D2_CACHE_AR && dc.caching != S2D2_CACHE_BLOCK_END) return bad("decode: caching");
    if (dc.caching == S2D2_CACHE_BLOCK_END && dc.verifier_layout != S2D2_VERIFIER_ALIGNED_2L) return bad("decode: block-end caching needs the aligned verifier layout");
    return S2D2_OK;
}

template <typename T>
int dmalloc(s2d2_ctx* c, T** p, size_t n) {
    CUDA_TRY(c, cudaMalloc((void**)p, std::max<size_t>(n, 1) * sizeof(T)));
    return S2D2_OK;
}

}  // namespace

extern "C" const char* s2d2_last_error(const s2d2_ctx* ctx) { return ctx ? ctx->err.c_str() : "null context"; }

extern "C" int s2d2_create(const s2d2_model_config* m, const s2d2_decode_config* dc, void* cuda_stream,
                           s2d2_ctx** out) {
    if (!m || !dc || !out) return S2D2_ERR_INVALID;
    *out = nullptr;
    std::string why;
    if (validate(*m, *dc, why) != S2D2_OK) {
        fprintf(stderr, "s2d2_create: %s\n", why.c_str());
        return S2D2_ERR_INVALID;
    }
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
        fprintf(stderr, "s2d2_create: no CUDA device (this library has no CPU path)\n");
        return S2D2_ERR_CUDA;
    }
    s2d2_ctx* c = new s2d2_ctx();
    c->m = *m;
    c->dc = *dc;
    c->stream = (cudaStream_t)cuda_stream;
    memset(&c->cnt, 0, sizeof(c->cnt));
    memset(&c->policy, 0, sizeof(c->policy));
    c->policy.policy = S2D2_ROUTE_MIN_SPAN;
    c->policy.p0 = 1.f;
    cudaGetDevice(&c->device);
    *out = c;   // returned even on failure below so that the caller can read last_error and destroy

    // weights arena
    c->w_bytes = plan_weights(c, nullptr);
    CUDA_TRY(c, cudaMalloc((void**)&c->w_arena, c->w_bytes));
    plan_weights(c, c->w_arena);

    // KV pool
    c->page_tokens = dc->kv_page_tokens;
    c->page_shift = 0;
    while ((1 << c->page_shift) < c->page_tokens) ++c->page_shift;
    c->max_pages_per_seq = (dc->max_seq_len + c->page_tokens - 1) / c->page_tokens;
    c->n_pages = dc->n_kv_pages > 0 ? dc->n_kv_pages : dc->max_batch * c->max_pages_per_seq;
    size_t page_elems = (size_t)2 * m->n_kv_heads * c->page_tokens * m->head_dim;
    size_t kv_bytes = (size_t)m->n_layers * c->n_pages * page_elems * esize(m->dtype);
    CUDA_TRY(c, cudaMalloc(&c->kv_base, kv_bytes));
    CUDA_TRY(c, cudaMemsetAsync(c->kv_base, 0, kv_bytes, c->stream));
    for (int p = c->n_pages - 1; p >= 0; --p) c->free_pages.push_back(p);
    c->seqs.assign(dc->max_batch, SeqState());

    // scratch
    int rows_per_seq = std::max(2 * dc->block_size, S2D2_MAX_ROWS_PER_SEQ);
    // A prefill pass carries several 64-row chunks of one prompt (see s2d2_prefill), so even a context for one
    // sequence gets room for a pass wide enough to be tensor-bound.
    c->max_rows = std::max(dc->max_batch * rows_per_seq, (int)PREFILL_PASS_ROWS);
    c->max_logit_rows = dc->max_batch * dc->block_size;
    size_t M = c->max_rows, d = m->d_model, es = esize(m->dtype);
    size_t nqkv = (size_t)(m->n_q_heads + 2 * m->n_kv_heads) * m->head_dim, nq = (size_t)m->n_q_heads * m->head_dim;
    size_t f = m->n_experts > 0 ? (size_t)m->expert_ffn * std::max(1, m->n_shared) : (size_t)m->ffn;
    int rc;
    if ((rc = dmalloc(c, &c->h, M * d))) return rc;
    if ((rc = dmalloc(c, &c->qkv, M * nqkv))) return rc;
    if ((rc = dmalloc(c, &c->gu, M * 2 * f))) return rc;
    if ((rc = dmalloc(c, (char**)&c->xn, M * d * es))) return rc;
    if ((rc = dmalloc(c, (char**)&c->q, M * nq * es))) return rc;
    if ((rc = dmalloc(c, (char**)&c->k_rows, M * m->n_kv_heads * m->head_dim * es))) return rc;
    if ((rc = dmalloc(c, (char**)&c->v_rows, M * m->n_kv_heads * m->head_dim * es))) return rc;
    if ((rc = dmalloc(c, (char**)&c->attn, M * nq * es))) return rc;
    if ((rc = dmalloc(c, (char**)&c->act, M * f * es))) return rc;
    if (m->dtype == S2D2_DTYPE_BF16 && dc->use_tensor_cores) {
        if ((rc = dmalloc(c, (char**)&c->xn_lo, M * d * es))) return rc;
        if ((rc = dmalloc(c, (char**)&c->q_lo, M * nq * es))) return rc;
        if ((rc = dmalloc(c, (char**)&c->attn_lo, M * nq * es))) return rc;
        if ((rc = dmalloc(c, (char**)&c->act_lo, M * f * es))) return rc;
    }
    if ((rc = dmalloc(c, &c->logits_draft, (size_t)c->max_logit_rows * m->vocab))) return rc;
    if ((rc = dmalloc(c, &c->logits_verify, (size_t)c->max_logit_rows * m->vocab))) return rc;
    if (m->n_experts > 0) {
        size_t P = M * m->top_k, fe = m->expert_ffn;
        if ((rc = dmalloc(c, &c->router_logits, M * m->n_experts))) return rc;
        if ((rc = dmalloc(c, &c->moe_gates, P))) return rc;
        if ((rc = dmalloc(c, &c->moe_ids, P))) return rc;
        if ((rc = dmalloc(c, &c->moe_gu, P * 2 * fe))) return rc;
        if ((rc = dmalloc(c, (char**)&c->moe_act, P * fe * es))) return rc;
        if ((rc = dmalloc(c, &c->moe_out, P * d))) return rc;
        if ((rc = dmalloc(c, &c->moe_ids_trace, (size_t)m->n_layers * P))) return rc;
    }
    // RoPE table in fp64 on the host, stored fp32
    {
        int half = m->head_dim / 2;
        size_t n = (size_t)dc->max_seq_len * half;
        std::vector<float> cs(n), sn(n);
        for (int p = 0; p < dc->max_seq_len; ++p)
            for (int i = 0; i < half; ++i) {
                double ang = (double)p * pow((double)m->rope_base, -2.0 * i / m->head_dim);
                cs[(size_t)p * half + i] = (float)cos(ang);
                sn[(size_t)p * half + i] = (float)sin(ang);
            }
        if ((rc = dmalloc(c, &c->rope_cos, n))) return rc;
        if ((rc = dmalloc(c, &c->rope_sin, n))) return rc;
        CUDA_TRY(c, cudaMemcpy(c->rope_cos, cs.data(), n * 4, cudaMemcpyHostToDevice));
        CUDA_TRY(c, cudaMemcpy(c->rope_sin, sn.data(), n * 4, cudaMemcpyHostToDevice));
    }
    // pass metadata staging
    {
        PassMeta& pm = c->meta;
        pm.cap_rows = c->max_rows;
        pm.cap_seqs = dc->max_batch + c->max_rows / S2D2_MAX_ROWS_PER_SEQ;     // sequences plus the chunks of a prefill pass
        pm.max_pages = c->max_pages_per_seq;
        size_t o = 0;
        auto take = [&](size_t b) {
            size_t r = o;
            o = align_up(o + b, 16);
            return r;
        };
        pm.off_mask = take((size_t)pm.cap_rows * 8);
        pm.off_token = take((size_t)pm.cap_rows * 4);
        pm.off_pos = take((size_t)pm.cap_rows * 4);
        pm.off_seq = take((size_t)pm.cap_rows * 4);
        pm.off_flags = take((size_t)pm.cap_rows * 4);
        pm.off_logit_rows = take((size_t)pm.cap_rows * 4);
        pm.off_nctx = take((size_t)pm.cap_seqs * 4);
        pm.off_row0 = take((size_t)pm.cap_seqs * 4);
        pm.off_nrows = take((size_t)pm.cap_seqs * 4);
        pm.off_pages = take((size_t)pm.cap_seqs * pm.max_pages * 4);
        pm.bytes = o;
        CUDA_TRY(c, cudaMallocHost((void**)&pm.h, pm.bytes));
        CUDA_TRY(c, cudaMalloc((void**)&pm.d, pm.bytes));
        memset(pm.h, 0, pm.bytes);
    }
    // draft statistics and acceptance staging
    {
        size_t R = c->max_logit_rows;
        if ((rc = dmalloc(c, &c->d_xhat, R))) return rc;
        if ((rc = dmalloc(c, &c->d_conf, R))) return rc;
        if ((rc = dmalloc(c, &c->d_margin, R))) return rc;
        if ((rc = dmalloc(c, &c->d_entropy, R))) return rc;
        if ((rc = dmalloc(c, &c->d_lse, R))) return rc;
        size_t nch = vocab_chunks(m->vocab), Sq = dc->max_batch;
        if ((rc = dmalloc(c, (ChunkStats**)&c->chunk_d, R * nch))) return rc;
        if ((rc = dmalloc(c, (ChunkStats**)&c->chunk_v, R * nch))) return rc;
        if ((rc = dmalloc(c, (RejectInfo**)&c->rej_info, Sq))) return rc;
        if ((rc = dmalloc(c, &c->res_rsum, Sq * nch))) return rc;
        if ((rc = dmalloc(c, &c->res_vsum, Sq * nch))) return rc;
        CUDA_TRY(c, cudaMallocHost((void**)&c->stats_h, R * 16));
        CUDA_TRY(c, cudaMallocHost((void**)&c->dsamp_h, std::max<size_t>(R, 1) * 12));
        if ((rc = dmalloc(c, &c->dsamp_d, R * 3))) return rc;
        size_t S = dc->max_batch;
        c->acc_bytes = S * 4 * 12 + R * 4 + S * S2D2_MAX_BLOCK * 4 * 3 + 256;      // per sequence, plus the row -> sequence table
        if ((rc = dmalloc(c, &c->acc_tickets, S))) return rc;
        CUDA_TRY(c, cudaMemset(c->acc_tickets, 0, S * 4));
        CUDA_TRY(c, cudaMallocHost((void**)&c->acc_h, c->acc_bytes));
        CUDA_TRY(c, cudaMalloc((void**)&c->acc_d, c->acc_bytes));
    }
    for (int i = 0; i < 8; ++i) CUDA_TRY(c, cudaEventCreate(&c->ev[i]));
    CUDA_TRY(c, cudaMalloc((void**)&c->d_status, 4));
    CUDA_TRY(c, cudaMemset(c->d_status, 0, 4));
    CUDA_TRY(c, cudaMallocHost((void**)&c->h_status, 4));
    *c->h_status = 0;
    int grc = gemm_init(c);
    if (grc != S2D2_OK) return grc;
    if ((grc = attention_init(c)) != S2D2_OK) return grc;
    if ((grc = pass_init(c)) != S2D2_OK) return grc;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return S2D2_OK;
}

extern "C" int s2d2_destroy(s2d2_ctx* c) {
    if (!c) return S2D2_ERR_INVALID;
    cudaStreamSynchronize(c->stream);
    pass_destroy(c);
    attention_destroy(c);
    gemm_destroy(c);
    void* ptrs[] = {c->w_arena, c->kv_base, c->h, c->qkv, c->gu, c->xn, c->q, c->k_rows, c->v_rows, c->attn, c->act, c->xn_lo, c->q_lo, c->attn_lo, c->act_lo,
                    c->logits_draft, c->logits_verify, c->rope_cos, c->rope_sin, c->router_logits, c->moe_gates,
                    c->moe_ids, c->moe_gu, c->moe_act, c->moe_out, c->moe_ids_trace, c->meta.d, c->d_xhat, c->d_conf,
                    c->d_margin, c->d_entropy, c->d_lse, c->acc_d, c->d_status, c->chunk_d, c->chunk_v, c->rej_info,
                    c->res_rsum, c->res_vsum, c->dsamp_d, c->acc_tickets};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    if (c->meta.h) cudaFreeHost(c->meta.h);
    if (c->stats_h) cudaFreeHost(c->stats_h);
    if (c->dsamp_h) cudaFreeHost(c->dsamp_h);
    if (c->acc_h) cudaFreeHost(c->acc_h);
    if (c->h_status) cudaFreeHost(c->h_status);
    for (int i = 0; i < 8; ++i)
        if (c->ev[i]) cudaEventDestroy(c->ev[i]);
    delete c;
    return S2D2_OK;
}

extern "C" int s2d2_load_weights(s2d2_ctx* c, const s2d2_tensor_desc* t, int32_t n) {
    if (!c || (!t && n > 0)) return S2D2_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        auto it = c->slots.find(t[i].name ? t[i].name : "");
        if (it == c->slots.end()) FAIL(c, S2D2_ERR_INVALID, std::string("unknown tensor: ") + (t[i].name ? t[i].name : "(null)"));
        WeightSlot& s = it->second;
        size_t elems = 1;
        for (int k = 0; k < t[i].ndim; ++k) elems *= (size_t)t[i].shape[k];
        if (t[i].dtype != s.dtype || elems * esize(t[i].dtype) != s.bytes || !t[i].data)
            FAIL(c, S2D2_ERR_INVALID, std::string("tensor has wrong dtype or size: ") + t[i].name);
        CUDA_TRY(c, cudaMemcpyAsync(s.d_ptr, t[i].data, s.bytes, cudaMemcpyHostToDevice, c->stream));
        s.loaded = true;
    }
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    c->weights_checked = false;
    return S2D2_OK;
}

// The device status word travels back with the results of every synchronous call.
static int enqueue_status_read(s2d2_ctx* c) {
    CUDA_TRY(c, cudaMemcpyAsync(c->h_status, c->d_status, 4, cudaMemcpyDeviceToHost, c->stream));
    return S2D2_OK;
}
static int check_status(s2d2_ctx* c) {
    if (*c->h_status == 0) return S2D2_OK;
    const int code = *c->h_status;
    *c->h_status = 0;
    cudaMemsetAsync(c->d_status, 0, 4, c->stream);
    gemm_reset_tickets(c);      // a split-K CTA that gave up took no ticket: start the next GEMM from clean counters
    FAIL(c, S2D2_ERR_TIMEOUT, "a kernel gave up on a bounded wait (results of this call are invalid; device status word " +
                                   std::to_string(code) + ")");
}

static int check_weights(s2d2_ctx* c) {
    if (c->weights_checked) return S2D2_OK;
    for (auto& kv : c->slots)
        if (!kv.second.loaded) FAIL(c, S2D2_ERR_MISSING_WEIGHT, "tensor not loaded: " + kv.first);
    c->weights_checked = true;
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// pass construction and execution
// ---------------------------------------------------------------------------------------------
namespace {

struct PassBuild {
    int n_rows = 0, n_seqs = 0, n_logit = 0;
    int max_ctx = 0, max_rows = 0;     // over the sequences of the pass
    long long sum_ctx = 0;             // cached tokens visible to the pass, all sequences
};

int ensure_pages(s2d2_ctx* c, SeqState& s, int n_tokens) {
    int need = (n_tokens + c->page_tokens - 1) / c->page_tokens;
    if (need > c->max_pages_per_seq) FAIL(c, S2D2_ERR_OOM, "sequence longer than max_seq_len");
    while ((int)s.pages.size() < need) {
        if (c->free_pages.empty()) FAIL(c, S2D2_ERR_OOM, "KV page pool exhausted");
        s.pages.push_back(c->free_pages.back());
        c->free_pages.pop_back();
    }
    return S2D2_OK;
}

// Starts the rows of one sequence in the pass being built.
void begin_seq(s2d2_ctx* c, PassBuild& pb, const SeqState& s, int n_ctx) {
    PassMeta& pm = c->meta;
    int q = pb.n_seqs++;
    pb.max_ctx = std::max(pb.max_ctx, n_ctx);
    pb.sum_ctx += n_ctx;
    pm.hp<int>(pm.off_nctx)[q] = n_ctx;
    pm.hp<int>(pm.off_row0)[q] = pb.n_rows;
    pm.hp<int>(pm.off_nrows)[q] = 0;
    int* pg = pm.hp<int>(pm.off_pages) + (size_t)q * pm.max_pages;
    for (size_t i = 0; i < s.pages.size(); ++i) pg[i] = s.pages[i];
}
void add_row(s2d2_ctx* c, PassBuild& pb, int token, int pos, unsigned long long mask, int flags, bool logits) {
    PassMeta& pm = c->meta;
    int r = pb.n_rows++, q = pb.n_seqs - 1;
    pm.hp<int>(pm.off_token)[r] = token;
    pm.hp<int>(pm.off_pos)[r] = pos;
    pm.hp<int>(pm.off_seq)[r] = q;
    pm.hp<int>(pm.off_flags)[r] = flags;
    pm.hp<unsigned long long>(pm.off_mask)[r] = mask;
    pb.max_rows = std::max(pb.max_rows, ++pm.hp<int>(pm.off_nrows)[q]);
    if (logits) pm.hp<int>(pm.off_logit_rows)[pb.n_logit++] = r;
}
PassView make_view(s2d2_ctx* c, const PassBuild& pb) {
    PassMeta& pm = c->meta;
    PassView v;
    v.n_rows = pb.n_rows;
    v.n_seqs = pb.n_seqs;
    v.n_logit_rows = pb.n_logit;
    v.row_token = pm.dp<int>(pm.off_token);
    v.row_pos = pm.dp<int>(pm.off_pos);
    v.row_seq = pm.dp<int>(pm.off_seq);
    v.row_flags = pm.dp<int>(pm.off_flags);
    v.row_mask = pm.dp<unsigned long long>(pm.off_mask);
    v.logit_rows = pm.dp<int>(pm.off_logit_rows);
    v.seq_nctx = pm.dp<int>(pm.off_nctx);
    v.seq_row0 = pm.dp<int>(pm.off_row0);
    v.seq_nrows = pm.dp<int>(pm.off_nrows);
    v.seq_pages = pm.dp<int>(pm.off_pages);
    v.max_pages = pm.max_pages;
    return v;
}

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

// One pass of the network over the rows described by the uploaded metadata.
// Logits of pv.logit_rows go to `logits_out` (row-major [n_logit_rows, vocab]).
template <typename TW, typename TA, typename TKV>
int run_pass_t(s2d2_ctx* c, const PassBuild& pb, float* logits_out) {
    const s2d2_model_config& m = c->m;
    PassView pv = make_view(c, pb);
    cudaStream_t st = c->stream;
    int M = pb.n_rows, d = m.d_model, hd = m.head_dim;
    if (M == 0) return S2D2_OK;
    int nqkv = (m.n_q_heads + 2 * m.n_kv_heads) * hd, nq = m.n_q_heads * hd;
    CUDA_TRY(c, cudaMemcpyAsync(c->meta.d, c->meta.h, c->meta.bytes, cudaMemcpyHostToDevice, st));
    c->cnt.h2d_bytes += c->meta.bytes;
    {   // the persistent kernel runs the whole pass when the shape allows it
        bool taken = false;
        int rc = pass_run(c, pv, pb.max_ctx, pb.max_rows, pb.sum_ctx, logits_out, &taken);
        if (rc) return rc;
        if (taken) {
            CUDA_TRY(c, cudaGetLastError());
            return S2D2_OK;
        }
    }
    embed_kernel<TW><<<M, 256, 0, st>>>((const TW*)c->embed, pv.row_token, c->h, d);
    LAUNCHED(c);
    KvPool<TKV> pool = make_pool<TKV>(c);
    for (int l = 0; l < m.n_layers; ++l) {
        const LayerWeights& L = c->layers[l];
        rmsnorm_kernel<TA><<<M, 256, 0, st>>>(c->h, nullptr, L.attn_norm, (TA*)c->xn, (TA*)c->xn_lo, d, m.rms_eps);
        LAUNCHED(c);
        int rc = gemm(c, c->xn, L.wqkv, c->qkv, M, nqkv, d, nqkv, 1.f, 0, c->xn_lo);
        if (rc) return rc;
        if (M > 64 && hd <= 256)      // wide passes: a warp per (row, head) instead of a block
            qk_rope_kv_rows_kernel<TA, TKV><<<dim3(M, (m.n_q_heads + 2 * m.n_kv_heads + 7) / 8), 256, 0, st>>>(
                c->qkv, pv, L.q_norm, L.k_norm, c->rope_cos, c->rope_sin, (TA*)c->q, (TA*)c->q_lo, (TKV*)c->k_rows, (TKV*)c->v_rows, pool,
                l, m.n_q_heads, m.n_kv_heads, hd, m.rms_eps, m.qk_norm);
        else
            qk_rope_kv_kernel<TA, TKV><<<dim3(M, m.n_q_heads + 2 * m.n_kv_heads), hd / 2, 0, st>>>(
                c->qkv, pv, L.q_norm, L.k_norm, c->rope_cos, c->rope_sin, (TA*)c->q, (TA*)c->q_lo, (TKV*)c->k_rows, (TKV*)c->v_rows, pool,
                l, m.n_q_heads, m.n_kv_heads, hd, m.rms_eps, m.qk_norm);
        LAUNCHED(c);
        if ((rc = attention(c, pv, l, pb.max_ctx, pb.max_rows))) return rc;
        if ((rc = gemm(c, c->attn, L.wo, c->h, M, d, nq, d, 1.f, 1, c->attn_lo))) return rc;
        rmsnorm_kernel<TA><<<M, 256, 0, st>>>(c->h, nullptr, L.ffn_norm, (TA*)c->xn, (TA*)c->xn_lo, d, m.rms_eps);
        LAUNCHED(c);
        if (m.n_experts > 0) {
            int E = m.n_experts, k = m.top_k, fe = m.expert_ffn, P = M * k;
            if ((rc = gemm(c, c->xn, L.router, c->router_logits, M, E, d, E, 1.f, 0, c->xn_lo))) return rc;
            moe_topk_kernel<<<M, 32, 0, st>>>(c->router_logits, M, E, k, c->moe_ids, c->moe_gates);
            LAUNCHED(c);
            CUDA_TRY(c, cudaMemcpyAsync(c->moe_ids_trace + (size_t)l * c->max_rows * k, c->moe_ids, (size_t)P * 4,
                                        cudaMemcpyDeviceToDevice, st));
            moe_gateup_kernel<TW, TA><<<dim3((2 * fe + 3) / 4, P), 128, 0, st>>>(
                (const TA*)c->xn, (const TW*)L.e_gate, (const TW*)L.e_up, c->moe_ids, c->moe_gu, k, fe, d);
            LAUNCHED(c);
            swiglu_kernel<TA><<<(unsigned)(((size_t)P * fe + 255) / 256), 256, 0, st>>>(c->moe_gu, (TA*)c->moe_act, (TA*)nullptr, P, fe);
            LAUNCHED(c);
            moe_down_kernel<TW, TA><<<dim3((d + 3) / 4, P), 128, 0, st>>>((const TA*)c->moe_act, (const TW*)L.e_down,
                                                                         c->moe_ids, c->moe_out, fe, d);
            LAUNCHED(c);
            moe_combine_kernel<<<(unsigned)(((size_t)M * d + 255) / 256), 256, 0, st>>>(c->moe_out, c->moe_gates, c->h, M,
                                                                                       k, d);
            LAUNCHED(c);
            c->cnt.moe_expert_tiles_touched += 0;   // filled by the grouped kernel when it is in use
            if (m.n_shared > 0) {
                int fs = fe * m.n_shared;
                if ((rc = gemm(c, c->xn, L.s_gu, c->gu, M, 2 * fs, d, 2 * fs, 1.f, 0, c->xn_lo))) return rc;
                swiglu_kernel<TA><<<(unsigned)(((size_t)M * fs + 255) / 256), 256, 0, st>>>(c->gu, (TA*)c->act, (TA*)c->act_lo, M, fs);
                LAUNCHED(c);
                if ((rc = gemm(c, c->act, L.s_down, c->h, M, d, fs, d, 1.f, 1, c->act_lo))) return rc;
            }
        } else {
            int f = m.ffn;
            if ((rc = gemm_swiglu(c, c->xn, c->xn_lo, L.wgu, M, f, d, c->act, c->act_lo)) < 0) {      // wide passes: SwiGLU in the GEMM's epilogue
                if ((rc = gemm(c, c->xn, L.wgu, c->gu, M, 2 * f, d, 2 * f, 1.f, 0, c->xn_lo))) return rc;
                swiglu_kernel<TA><<<(unsigned)(((size_t)M * f + 255) / 256), 256, 0, st>>>(c->gu, (TA*)c->act, (TA*)c->act_lo, M, f);
                LAUNCHED(c);
            } else if (rc) {
                return rc;
            }
            if ((rc = gemm(c, c->act, L.wdown, c->h, M, d, f, d, 1.f, 1, c->act_lo))) return rc;
        }
    }
    c->last_pass_rows = M;
    if (pb.n_logit > 0 && logits_out) {
        rmsnorm_kernel<TA><<<pb.n_logit, 256, 0, st>>>(c->h, pv.logit_rows, c->final_norm, (TA*)c->xn, (TA*)c->xn_lo, d, m.rms_eps);
        LAUNCHED(c);
        int rc = gemm(c, c->xn, c->lm_head, logits_out, pb.n_logit, m.vocab, d, m.vocab, m.logit_scale, 0, c->xn_lo);
        if (rc) return rc;
    }
    CUDA_TRY(c, cudaGetLastError());
    return S2D2_OK;
}

int run_pass(s2d2_ctx* c, const PassBuild& pb, float* logits_out) {
    if (c->m.dtype == S2D2_DTYPE_F32) return run_pass_t<float, float, float>(c, pb, logits_out);
    return run_pass_t<bf16, bf16, bf16>(c, pb, logits_out);
}

SeqState* get_seq(s2d2_ctx* c, int id) {
    if (id < 0 || id >= (int)c->seqs.size() || !c->seqs[id].active) return nullptr;
    return &c->seqs[id];
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// prefill
// ---------------------------------------------------------------------------------------------
extern "C" int s2d2_prefill(s2d2_ctx* c, int32_t n, const int32_t* const* prompts, const int32_t* lens,
                            int32_t* ids_out) {
    if (!c || n < 1 || !prompts || !lens || !ids_out) return S2D2_ERR_INVALID;
    int rc = check_weights(c);
    if (rc) return rc;
    std::vector<int> ids;
    for (int i = 0; i < n; ++i) {
        if (lens[i] < 1 || lens[i] + c->dc.block_size > c->dc.max_seq_len) FAIL(c, S2D2_ERR_INVALID, "prompt length");
        for (int t = 0; t < lens[i]; ++t)
            if (prompts[i][t] < 0 || prompts[i][t] >= c->m.vocab) FAIL(c, S2D2_ERR_INVALID, "prompt token out of range");
    }
    for (int i = 0; i < n; ++i) {
        int slot = -1;
        for (int k = 0; k < (int)c->seqs.size(); ++k)
            if (!c->seqs[k].active) {
                slot = k;
                break;
            }
        if (slot < 0) {
            for (int id : ids) s2d2_release_seq(c, id);
            FAIL(c, S2D2_ERR_OOM, "no free sequence slot (max_batch)");
        }
        SeqState& s = c->seqs[slot];
        s = SeqState();
        s.active = true;
        s.rng_stream = (uint32_t)slot;
        s.tok.assign(prompts[i], prompts[i] + lens[i]);
        s.n_final = s.n_prompt = lens[i];
        ids.push_back(slot);
        ids_out[i] = slot;
    }
    CUDA_TRY(c, cudaEventRecord(c->ev[6], c->stream));
    const int CH = S2D2_MAX_ROWS_PER_SEQ;
    std::vector<int> took(ids.size());
    // A row's in-pass mask has 64 bits, so one prompt enters a pass as chunks of at most 64 rows.  The chunks of one
    // prompt may share a pass: each is listed as a sequence of its own whose visible cache ends where the chunk
    // begins and whose page list is the prompt's.  K/V of every row is in the cache before attention starts, so a
    // chunk reads its predecessors of the same pass from the pages and only its own rows through the mask.
    // Which passes: a prompt remainder that one persistent pass can take (and at most four of them) goes through the
    // persistent kernel, which streams the weights once per 64 rows; everything longer goes through wide passes of
    // the per-operation kernels, which are tensor-bound and stream the weights once per PREFILL_PASS_ROWS rows.
    const int pr = pass_max_rows(c);
    // (mixture-of-experts layers have no tensor-core form on the per-operation path: their prompts stay on persistent passes)
    const bool wide_pays = c->m.n_experts == 0;
    for (;;) {
        int n_short = 0, n_long = 0;
        for (size_t k = 0; k < ids.size(); ++k) {
            const SeqState& s = c->seqs[ids[k]];
            const int left = s.n_final - s.n_c;
            if (left > 0) ++(pr > 0 && (left <= pr || !wide_pays) ? n_short : n_long);
        }
        const bool shorts_ride = pr == 0 || n_short > 4;
        const bool wide = n_long > 0 || (n_short > 0 && shorts_ride);
        PassBuild pb;
        int room = wide ? c->max_rows : pr;
        for (size_t k = 0; k < ids.size(); ++k) {
            SeqState& s = c->seqs[ids[k]];
            took[k] = 0;
            const int left = s.n_final - s.n_c;
            if (left <= 0 || room <= 0) continue;
            if (wide && pr > 0 && (left <= pr || !wide_pays) && !shorts_ride) continue;      // waits for the persistent pass
            int rows = std::min(left, room);
            if (rows < left) rows -= rows % CH;                               // whole chunks unless the prompt ends
            if (rows <= 0) continue;
            if ((rc = ensure_pages(c, s, s.n_c + rows))) {
                const std::string why = c->err;
                for (int id : ids) s2d2_release_seq(c, id);      // nothing of this call stays behind: slots and pages go back
                c->err = why;
                return rc;
            }
            for (int r0 = 0; r0 < rows; r0 += CH) {
                const int n = std::min(CH, rows - r0), base = s.n_c + r0;
                begin_seq(c, pb, s, base);
                for (int r = 0; r < n; ++r)
                    add_row(c, pb, s.tok[base + r], base + r, (r == 63) ? ~0ull : ((1ull << (r + 1)) - 1), ROW_WRITE_KV, false);
            }
            took[k] = rows;
            room -= rows;
        }
        if (pb.n_rows == 0) break;
        if ((rc = run_pass(c, pb, nullptr))) {
            const std::string why = c->err;
            for (int id : ids) s2d2_release_seq(c, id);
            c->err = why;
            return rc;
        }
        c->cnt.n_prefill_passes++;
        c->cnt.n_rows_prefill += pb.n_rows;
        // the metadata buffer is reused by the next chunk: wait for this pass to have consumed it
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        for (size_t k = 0; k < ids.size(); ++k) c->seqs[ids[k]].n_c += took[k];
    }
    if ((rc = enqueue_status_read(c))) return rc;
    CUDA_TRY(c, cudaEventRecord(c->ev[7], c->stream));
    CUDA_TRY(c, cudaEventSynchronize(c->ev[7]));
    if ((rc = check_status(c))) {
        const std::string why = c->err;
        for (int id : ids) s2d2_release_seq(c, id);
        c->err = why;
        return rc;
    }
    float ms = 0;
    cudaEventElapsedTime(&ms, c->ev[6], c->ev[7]);
    c->cnt.ms_prefill += ms;
    return S2D2_OK;
}

extern "C" int s2d2_seq_set_rng_stream(s2d2_ctx* c, int32_t id, uint32_t stream) {
    if (!c) return S2D2_ERR_INVALID;
    SeqState* s = get_seq(c, id);
    if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
    s->rng_stream = stream;
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// draft pass
// ---------------------------------------------------------------------------------------------
// SampleFromLogits over n_rows logit rows: per-chunk statistics, per-row merge (greedy proposal, confidence, margin,
// entropy, log-sum-exp) and, in sampling mode, the inverse-CDF draw that replaces proposal and confidence.  The
// Philox words of the rows are taken from dsamp_h (position | stream | step, n_rows each).
static int launch_draft_stats(s2d2_ctx* c, const float* d_logits, int n_rows, int draft_mode) {
    const int nch = vocab_chunks(c->m.vocab);
    DraftStatsOut so{c->d_xhat, c->d_conf, c->d_margin, c->d_entropy, c->d_lse};
    vocab_chunk_stats_kernel<<<dim3(nch, n_rows), VCHUNK_THREADS, 0, c->stream>>>(d_logits, c->m.vocab, (ChunkStats*)c->chunk_d);
    LAUNCHED(c);
    draft_finish_kernel<<<(n_rows + 3) / 4, 128, 0, c->stream>>>((const ChunkStats*)c->chunk_d, nch, n_rows, so);
    LAUNCHED(c);
    if (draft_mode == S2D2_DRAFT_SAMPLE) {
        CUDA_TRY(c, cudaMemcpyAsync(c->dsamp_d, c->dsamp_h, (size_t)n_rows * 12, cudaMemcpyHostToDevice, c->stream));
        c->cnt.h2d_bytes += (size_t)n_rows * 12;
        DraftSampleIn in{d_logits, c->m.vocab, (const ChunkStats*)c->chunk_d, c->dsamp_d, (const unsigned*)(c->dsamp_d + n_rows),
                         c->dsamp_d + 2 * n_rows, c->dc.seed};
        draft_sample_kernel<<<n_rows, VCHUNK_THREADS, 0, c->stream>>>(in, nch, so);
        LAUNCHED(c);
    }
    return S2D2_OK;
}

extern "C" int s2d2_draft_block(s2d2_ctx* c, int32_t n, const int32_t* ids, s2d2_draft_stats* out) {
    if (!c || n < 1 || !ids || !out) return S2D2_ERR_INVALID;
    const int B = c->dc.block_size, MASK = c->m.vocab;
    int rc;
    for (int i = 0; i < n; ++i) {
        SeqState* s = get_seq(c, ids[i]);
        if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
        // a sequence whose draft rows a later draft pass has overwritten may (and must) be drafted again
        if (s->drafted && s->draft_stamp == c->draft_gen) FAIL(c, S2D2_ERR_STATE, "draft_block called twice without accept_and_commit");
        for (int k = 0; k < i; ++k)
            if (ids[k] == ids[i]) FAIL(c, S2D2_ERR_INVALID, "duplicate sequence id");
        if (!s->block_open && s->n_final + B > c->dc.max_seq_len) FAIL(c, S2D2_ERR_OOM, "max_seq_len reached");
    }
    PassBuild pb;
    ++c->draft_gen;
    for (int i = 0; i < n; ++i) {
        SeqState& s = c->seqs[ids[i]];
        s.draft_stamp = c->draft_gen;
        s.verify_in_flight = false;       // a verifier pass made for an overwritten draft is void (its K/V rows lie past the cache length)
        if (!s.block_open) {
            s.tok.resize(s.n_final + B, MASK);
            s.block_open = true;
        }
        int st = s.n_final, j = 0;
        while (j < B && s.tok[st + j] != MASK) ++j;
        // Right-shifted layout: the logits that score in-block position i are those of the row at position i - 1, so the
        // pass starts at the last committed token even when its K/V is cached already (the cache visible to the pass
        // then ends before it, and the cached K/V is kept).
        const bool shifted = c->dc.verifier_layout == S2D2_VERIFIER_RIGHT_SHIFTED;
        if (c->dc.caching == S2D2_CACHE_BLOCK_END) {
            // block-end caching: the whole block, known tokens and MASKs, every row sees every row; nothing is cached
            if ((rc = ensure_pages(c, s, st + B))) return rc;
            begin_seq(c, pb, s, st);
            s.j = j;
            s.n_masked = 0;
            s.draft_row0 = pb.n_logit;
            const unsigned long long all_b = B == 64 ? ~0ull : ((1ull << B) - 1);
            for (int i2 = 0; i2 < B; ++i2) {
                bool masked = s.tok[st + i2] == MASK;
                add_row(c, pb, s.tok[st + i2], st + i2, all_b, 0, masked);
                if (masked) s.masked_idx[s.n_masked++] = i2;
            }
            s.span_len = 1;
            while (j + s.span_len < B && s.tok[st + j + s.span_len] == MASK) ++s.span_len;
            continue;
        }
        int q0 = shifted ? std::min(s.n_c, st + j - 1) : s.n_c;
        int P = st + j - q0;             // committed tokens that run as causal rows (those without K/V get it appended)
        int rows = P + (B - j);
        if (rows > S2D2_MAX_ROWS_PER_SEQ) FAIL(c, S2D2_ERR_UNSUPPORTED, "too many rows for one sequence in a draft pass");
        if ((rc = ensure_pages(c, s, st + B))) return rc;
        begin_seq(c, pb, s, q0);
        unsigned long long all = rows == 64 ? ~0ull : ((1ull << rows) - 1);
        s.j = j;
        s.n_masked = 0;
        s.draft_row0 = pb.n_logit;
        for (int p = 0; p < P; ++p)     // pending rows: causal among themselves, K/V appended
            add_row(c, pb, s.tok[q0 + p], q0 + p, (1ull << (p + 1)) - 1, q0 + p >= s.n_c ? ROW_WRITE_KV : 0, shifted && p == P - 1);
        for (int i2 = j; i2 < B; ++i2) {  // block rows: see the whole pass
            bool masked = s.tok[st + i2] == MASK;
            bool scores_masked = shifted ? (i2 + 1 < B && s.tok[st + i2 + 1] == MASK) : masked;
            add_row(c, pb, s.tok[st + i2], st + i2, all, 0, scores_masked);
            if (masked) s.masked_idx[s.n_masked++] = i2;
        }
        s.span_len = 1;
        while (j + s.span_len < B && s.tok[st + j + s.span_len] == MASK) ++s.span_len;
    }
    if (pb.n_logit > c->max_logit_rows || pb.n_rows > c->max_rows) FAIL(c, S2D2_ERR_UNSUPPORTED, "pass too large");
    CUDA_TRY(c, cudaEventRecord(c->ev[0], c->stream));
    if ((rc = run_pass(c, pb, c->logits_draft))) return rc;
    if (c->dc.draft_mode == S2D2_DRAFT_SAMPLE) {      // Philox words of the logit rows, in row order
        int r = 0;
        for (int i = 0; i < n; ++i) {
            const SeqState& s = c->seqs[ids[i]];
            for (int k = 0; k < s.n_masked; ++k, ++r) {
                c->dsamp_h[r] = s.n_final + s.masked_idx[k];
                c->dsamp_h[pb.n_logit + r] = (int)s.rng_stream;
                c->dsamp_h[2 * pb.n_logit + r] = s.step;
            }
        }
    }
    if ((rc = launch_draft_stats(c, c->logits_draft, pb.n_logit, c->dc.draft_mode))) return rc;
    size_t R = pb.n_logit;
    int* hx = (int*)c->stats_h;
    float* hc = (float*)(c->stats_h + R * 4);
    float* hm = (float*)(c->stats_h + R * 8);
    float* he = (float*)(c->stats_h + R * 12);
    CUDA_TRY(c, cudaMemcpyAsync(hx, c->d_xhat, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(hc, c->d_conf, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(hm, c->d_margin, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(he, c->d_entropy, R * 4, cudaMemcpyDeviceToHost, c->stream));
    c->cnt.d2h_bytes += R * 16;
    if ((rc = enqueue_status_read(c))) return rc;
    CUDA_TRY(c, cudaEventRecord(c->ev[1], c->stream));
    CUDA_TRY(c, cudaEventSynchronize(c->ev[1]));
    if ((rc = check_status(c))) return rc;
    float ms = 0;
    cudaEventElapsedTime(&ms, c->ev[0], c->ev[1]);
    c->cnt.ms_draft += ms;
    c->cnt.n_draft_passes++;
    c->cnt.n_rows_draft += pb.n_rows;
    c->n_draft_logit_rows = pb.n_logit;
    for (int i = 0; i < n; ++i) {
        SeqState& s = c->seqs[ids[i]];
        s2d2_draft_stats& o = out[i];
        memset(&o, 0, sizeof(o));
        if (c->dc.caching == S2D2_CACHE_AR) s.n_c = s.n_final + s.j;         // pending rows are cached now
        o.seq_id = ids[i];
        o.block_start = s.n_final;
        o.first_masked = s.j;
        o.n_masked = s.n_masked;
        o.span_len = s.span_len;
        double sum = 0;
        for (int k = 0; k < s.n_masked; ++k) {
            int r = s.draft_row0 + k;
            o.masked_idx[k] = s.masked_idx[k];
            o.xhat[k] = s.xhat[k] = hx[r];
            o.conf[k] = s.conf[k] = hc[r];
            o.margin[k] = hm[r];
            o.entropy[k] = he[r];
            sum += hc[r];
            if (hc[r] > c->dc.tau_conf) o.n_hi++;
        }
        o.mean_conf = (float)(sum / std::max(1, s.n_masked));
        s.drafted = true;
    }
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// routing (host)
// ---------------------------------------------------------------------------------------------
extern "C" int s2d2_set_router(s2d2_ctx* c, s2d2_route_fn fn, void* user) {
    if (!c) return S2D2_ERR_INVALID;
    c->route_fn = fn;
    c->route_user = user;
    return S2D2_OK;
}
extern "C" int s2d2_set_route_policy(s2d2_ctx* c, const s2d2_route_policy* p) {
    if (!c || !p || p->policy < 0 || p->policy > S2D2_ROUTE_UCB) return S2D2_ERR_INVALID;
    if (p->policy == S2D2_ROUTE_UCB && (p->p1 < 0.f || p->p1 > 16.f)) FAIL(c, S2D2_ERR_INVALID, "route policy: bins per context dimension must be 0..16");
    c->policy = *p;
    for (auto& s : c->seqs) {
        s.hyst_on = true;
        s.ucb_bucket = -1;
    }
    c->ucb_t = 0;
    c->ucb_n.clear();
    c->ucb_sum.clear();
    return S2D2_OK;
}

// Expected accepted prefix length K_hat = sum_k prod_{i<=k} alpha_i over the span (Eq. khat)
// and the static / dynamic verification score.
static double route_score(const s2d2_ctx* c, const s2d2_draft_stats* st) {
    const s2d2_route_policy& p = c->policy;
    double khat = 0, prod = 1;
    for (int i = 0; i < st->span_len; ++i) {     // masked_idx[0..span_len) is the span
        double alpha = p.alpha_entropy ? exp(-(double)p.alpha_param * st->entropy[i] / log((double)c->m.vocab))
                                       : (st->margin[i] >= p.alpha_param ? 1.0 : 0.0);
        prod *= alpha;
        khat += prod;
    }
    return p.dynamic_cost ? khat - (double)p.cost * st->n_hi : khat - (double)p.cost;
}

// Contextual-bandit router (Appendix "Contextual-bandit routing policy", Eq. (ucb)).
static int ucb_bins(const s2d2_ctx* c) { return c->policy.p1 >= 1.f ? (int)c->policy.p1 : 2; }
static int ucb_bucket_of(const s2d2_ctx* c, const s2d2_draft_stats* st) {
    const int nb = ucb_bins(c), B = c->dc.block_size;
    const int b_span = std::min(nb - 1, (st->span_len - 1) * nb / B);
    const int b_prog = std::min(nb - 1, (B - st->n_masked) * nb / B);
    double h = 0;
    for (int i = 0; i < st->span_len; ++i) h += st->entropy[i];
    h /= (double)st->span_len * log((double)c->m.vocab);
    const int b_ent = std::min(nb - 1, std::max(0, (int)floor(h * nb)));
    return (b_span * nb + b_prog) * nb + b_ent;
}
static double ucb_index(const s2d2_ctx* c, int action, int bucket) {
    const long long n = c->ucb_n[2 * bucket + action];
    if (n == 0) return INFINITY;
    return c->ucb_sum[2 * bucket + action] / (double)n + (double)c->policy.p0 * sqrt(log((double)c->ucb_t) / (double)n);
}

extern "C" int s2d2_route(s2d2_ctx* c, int32_t n, const s2d2_draft_stats* st, uint8_t* flags) {
    if (!c || n < 1 || !st || !flags) return S2D2_ERR_INVALID;
    for (int i = 0; i < n; ++i) {
        if (c->route_fn) {
            flags[i] = c->route_fn(c->route_user, &st[i]) ? 1 : 0;
            continue;
        }
        const s2d2_route_policy& p = c->policy;
        switch (p.policy) {
            case S2D2_ROUTE_MIN_SPAN: flags[i] = st[i].span_len >= (int)p.p0; break;
            case S2D2_ROUTE_SCORE: flags[i] = route_score(c, &st[i]) >= p.p0; break;
            case S2D2_ROUTE_HYSTERESIS: {
                SeqState* s = get_seq(c, st[i].seq_id);
                if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id in stats");
                double sc = route_score(c, &st[i]);
                if (s->hyst_on && sc < p.p1) s->hyst_on = false;
                else if (!s->hyst_on && sc >= p.p0) s->hyst_on = true;
                flags[i] = s->hyst_on;
                break;
            }
            case S2D2_ROUTE_MEAN_CONF: flags[i] = st[i].mean_conf < p.p0; break;
            case S2D2_ROUTE_UCB: {
                SeqState* s = get_seq(c, st[i].seq_id);
                if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id in stats");
                if (st[i].span_len < 1 || st[i].span_len > c->dc.block_size || st[i].n_masked < st[i].span_len)
                    FAIL(c, S2D2_ERR_INVALID, "draft stats: span");
                const int nb = ucb_bins(c);
                if (c->ucb_n.empty()) {
                    c->ucb_n.assign((size_t)2 * nb * nb * nb, 0);
                    c->ucb_sum.assign((size_t)2 * nb * nb * nb, 0.0);
                }
                ++c->ucb_t;
                const int b = ucb_bucket_of(c, &st[i]);
                flags[i] = ucb_index(c, 1, b) >= ucb_index(c, 0, b);
                s->ucb_bucket = b;
                break;
            }
            default: flags[i] = 0;
        }
    }
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// verifier pass
// ---------------------------------------------------------------------------------------------
extern "C" int s2d2_verify_block(s2d2_ctx* c, int32_t n, const int32_t* ids, const uint8_t* flags) {
    if (!c || n < 1 || !ids || !flags) return S2D2_ERR_INVALID;
    const int MASK = c->m.vocab;
    int rc;
    PassBuild pb;
    for (int i = 0; i < n; ++i) {
        SeqState* s = get_seq(c, ids[i]);
        if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
        if (!s->drafted) FAIL(c, S2D2_ERR_STATE, "verify_block without a draft pass");
        if (s->draft_stamp != c->draft_gen)
            FAIL(c, S2D2_ERR_STATE, "the draft pass of this sequence was overwritten by a later draft_block: draft it again");
        if (s->verify_in_flight) FAIL(c, S2D2_ERR_STATE, "verify_block called twice");
        for (int k = 0; k < i; ++k)
            if (ids[k] == ids[i]) FAIL(c, S2D2_ERR_INVALID, "duplicate sequence id");
    }
    // one verifier pass per step: sequences verified by an earlier call of this step would lose their rows
    for (auto& other : c->seqs)
        if (other.active && other.verify_in_flight && other.verify_stamp == c->verify_gen && other.draft_stamp == c->draft_gen) {
            bool flagged_now = false;
            for (int i = 0; i < n; ++i) flagged_now = flagged_now || (flags[i] != 0);
            if (flagged_now) FAIL(c, S2D2_ERR_STATE, "a second verify_block before accept_and_commit would overwrite the first one's logits");
            break;
        }
    {
        bool any = false;
        for (int i = 0; i < n; ++i) any = any || flags[i];
        if (any) ++c->verify_gen;
    }
    for (int i = 0; i < n; ++i) {
        if (!flags[i]) continue;
        SeqState& s = c->seqs[ids[i]];
        int L = s.span_len, p0 = s.n_final + s.j;
        if ((rc = ensure_pages(c, s, p0 + L))) return rc;
        s.verify_stamp = c->verify_gen;
        if (c->dc.verifier_layout == S2D2_VERIFIER_RIGHT_SHIFTED) {
            // L causal rows: the last committed token (its K/V is in the cache since the draft pass; the cache visible
            // to this pass ends before it), then the drafted tokens but the last; row k scores drafted token k + 1
            begin_seq(c, pb, s, p0 - 1);
            s.verify_row0 = pb.n_logit;
            add_row(c, pb, s.tok[p0 - 1], p0 - 1, 1ull, 0, true);
            for (int k = 1; k < L; ++k) add_row(c, pb, s.xhat[k - 1], p0 + k - 1, (1ull << (k + 1)) - 1, ROW_WRITE_KV, true);
            s.verify_in_flight = true;
            continue;
        }
        if (c->dc.caching == S2D2_CACHE_BLOCK_END) {
            // the block's committed prefix has no K/V in the cache: it rides along as causal rows in front of the drafted
            // tokens (one causal run of j + L rows, nothing written); MASK copy i sees the token rows to its left and itself
            const int jj = s.j, st0 = s.n_final;
            if (jj + 2 * L > S2D2_MAX_ROWS_PER_SEQ) FAIL(c, S2D2_ERR_UNSUPPORTED, "too many rows for one sequence in a verifier pass");
            begin_seq(c, pb, s, st0);
            s.verify_row0 = pb.n_logit;
            for (int k = 0; k < jj; ++k) add_row(c, pb, s.tok[st0 + k], st0 + k, (1ull << (k + 1)) - 1, 0, false);
            for (int k = 0; k < L; ++k) add_row(c, pb, s.xhat[k], p0 + k, (1ull << (jj + k + 1)) - 1, 0, false);
            for (int k = 0; k < L; ++k) add_row(c, pb, MASK, p0 + k, ((1ull << (jj + k)) - 1) | (1ull << (jj + L + k)), 0, true);
            s.verify_in_flight = true;
            continue;
        }
        begin_seq(c, pb, s, s.n_c);
        s.verify_row0 = pb.n_logit;
        // drafted tokens: causal block A_L; their K/V goes to the cache speculatively
        for (int k = 0; k < L; ++k) add_row(c, pb, s.xhat[k], p0 + k, (1ull << (k + 1)) - 1, ROW_WRITE_KV, false);
        // MASK copies at the same positions: strictly-left drafted tokens plus itself
        for (int k = 0; k < L; ++k)
            add_row(c, pb, MASK, p0 + k, ((1ull << k) - 1) | (1ull << (L + k)), 0, true);
        s.verify_in_flight = true;
    }
    c->n_verify_logit_rows = pb.n_logit;
    if (pb.n_rows == 0) return S2D2_OK;
    CUDA_TRY(c, cudaEventRecord(c->ev[2], c->stream));
    if ((rc = run_pass(c, pb, c->logits_verify))) return rc;
    CUDA_TRY(c, cudaEventRecord(c->ev[3], c->stream));
    c->verify_timing_pending = true;
    c->cnt.n_verify_passes++;
    c->cnt.n_rows_verify += pb.n_rows;
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// acceptance + commit
// ---------------------------------------------------------------------------------------------
namespace {
struct AccStage {     // layout of acc_h / acc_d for S sequences
    size_t S;
    size_t o_draft0, o_verify0, o_len, o_pos0, o_stream, o_step, o_mode, o_row_seq;     // inputs (row_seq: per verifier logit row)
    size_t o_nacc, o_rej, o_res, o_near, o_bits, o_u, o_a, o_v;              // outputs
    size_t in_bytes, total;
    AccStage(size_t s, size_t verify_rows) : S(s) {
        size_t o = 0;
        auto t = [&](size_t b) { size_t r = o; o += b; return r; };
        o_draft0 = t(S * 4); o_verify0 = t(S * 4); o_len = t(S * 4); o_pos0 = t(S * 4);
        o_stream = t(S * 4); o_step = t(S * 4); o_mode = t(S * 4); o_row_seq = t(verify_rows * 4);
        in_bytes = o;
        o_nacc = t(S * 4); o_rej = t(S * 4); o_res = t(S * 4); o_near = t(S * 4); o_bits = t(S * 4);
        o_u = t(S * S2D2_MAX_BLOCK * 4); o_a = t(S * S2D2_MAX_BLOCK * 4); o_v = t(S * S2D2_MAX_BLOCK * 4);
        total = o;
    }
};

// n_draft_rows / n_verify_rows: logit rows of the two buffers that the sequences refer to.
int launch_accept(s2d2_ctx* c, const AccStage& a, int n, const float* d_draft, const float* d_verify, const int* d_xhat,
                  const double* d_lse, const float* d_conf, int n_draft_rows, int n_verify_rows) {
    {   // verifier logit row -> index of its sequence in this call (-1: a row of a sequence that is not part of it)
        int* row_seq = (int*)(c->acc_h + a.o_row_seq);
        const int *v0 = (const int*)(c->acc_h + a.o_verify0), *len = (const int*)(c->acc_h + a.o_len), *mode = (const int*)(c->acc_h + a.o_mode);
        for (int r = 0; r < n_verify_rows; ++r) row_seq[r] = -1;
        for (int i = 0; i < n; ++i)
            if (mode[i])
                for (int k = 0; k < len[i] && v0[i] + k < n_verify_rows; ++k) row_seq[v0[i] + k] = i;
    }
    CUDA_TRY(c, cudaMemcpyAsync(c->acc_d, c->acc_h, a.in_bytes, cudaMemcpyHostToDevice, c->stream));
    c->cnt.h2d_bytes += a.in_bytes;
    c->cnt.d2h_bytes += a.total - a.in_bytes;
    AcceptIn in;
    in.draft_logits = d_draft;
    in.verify_logits = d_verify;
    in.V = c->m.vocab;
    in.seq_draft_row0 = (const int*)(c->acc_d + a.o_draft0);
    in.seq_verify_row0 = (const int*)(c->acc_d + a.o_verify0);
    in.seq_len = (const int*)(c->acc_d + a.o_len);
    in.seq_pos0 = (const int*)(c->acc_d + a.o_pos0);
    in.seq_stream = (const unsigned*)(c->acc_d + a.o_stream);
    in.seq_step = (const int*)(c->acc_d + a.o_step);
    in.seq_mode = (const int*)(c->acc_d + a.o_mode);
    in.xhat = d_xhat;
    in.draft_lse = d_lse;
    in.conf = d_conf;
    in.tau_conf = c->dc.tau_conf;
    in.seed = c->dc.seed;
    in.gamma = c->dc.ratio_gamma;
    in.accept_override = c->accept_override;
    in.resample = c->dc.resample;
    in.l_cap = S2D2_MAX_BLOCK;
    AcceptOut out;
    out.n_accepted = (int*)(c->acc_d + a.o_nacc);
    out.first_reject = (int*)(c->acc_d + a.o_rej);
    out.resampled = (int*)(c->acc_d + a.o_res);
    out.n_near = (int*)(c->acc_d + a.o_near);
    out.commit_bits = (unsigned*)(c->acc_d + a.o_bits);
    out.u = (float*)(c->acc_d + a.o_u);
    out.a = (float*)(c->acc_d + a.o_a);
    out.v = (float*)(c->acc_d + a.o_v);
    const int nch = vocab_chunks(c->m.vocab);
    in.verify_chunks = (const ChunkStats*)c->chunk_v;
    in.draft_chunks = (const ChunkStats*)c->chunk_d;
    if (!d_lse && n_draft_rows > 0) {      // stand-alone entry without draft statistics: the drafter's chunk statistics first
        vocab_chunk_stats_kernel<<<dim3(nch, n_draft_rows), VCHUNK_THREADS, 0, c->stream>>>(d_draft, c->m.vocab, (ChunkStats*)c->chunk_d);
        LAUNCHED(c);
    }
    // chunk statistics + scan in one launch, the residual draw in a second (see accept_fused_kernel)
    accept_fused_kernel<<<dim3(nch, n_verify_rows + n), VCHUNK_THREADS, 0, c->stream>>>(
        in, out, (RejectInfo*)c->rej_info, (ChunkStats*)c->chunk_v, (const int*)(c->acc_d + a.o_row_seq), c->acc_tickets, n_verify_rows);
    LAUNCHED(c);
    if (c->dc.resample && n_verify_rows > 0) {
        residual_fused_kernel<<<dim3(nch, n), VCHUNK_THREADS, 0, c->stream>>>(in, (const RejectInfo*)c->rej_info, c->res_rsum, c->res_vsum,
                                                                              c->acc_tickets, out.resampled);
        LAUNCHED(c);
    }
    CUDA_TRY(c, cudaMemcpyAsync(c->acc_h + a.in_bytes, c->acc_d + a.in_bytes, a.total - a.in_bytes,
                                cudaMemcpyDeviceToHost, c->stream));
    return S2D2_OK;
}
}  // namespace

extern "C" int s2d2_accept_and_commit(s2d2_ctx* c, int32_t n, const int32_t* ids, const uint8_t* flags,
                                      s2d2_step_result* res) {
    if (!c || n < 1 || !ids || !flags || !res) return S2D2_ERR_INVALID;
    if (n > c->dc.max_batch) return S2D2_ERR_INVALID;
    const int B = c->dc.block_size, MASK = c->m.vocab;
    for (int i = 0; i < n; ++i) {
        SeqState* s = get_seq(c, ids[i]);
        if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
        if (!s->drafted) FAIL(c, S2D2_ERR_STATE, "accept_and_commit without a draft pass");
        if (s->draft_stamp != c->draft_gen)
            FAIL(c, S2D2_ERR_STATE, "the draft pass of this sequence was overwritten by a later draft_block: draft it again");
        if (flags[i] && s->verify_in_flight && s->verify_stamp != c->verify_gen)
            FAIL(c, S2D2_ERR_STATE, "the verifier pass of this sequence was overwritten by a later verify_block");
        if (flags[i] && !s->verify_in_flight) FAIL(c, S2D2_ERR_STATE, "sequence flagged verified but verify_block did not run for it");
        if (!flags[i] && s->verify_in_flight) FAIL(c, S2D2_ERR_STATE, "verify flags differ from those given to verify_block");
    }
    AccStage a(n, c->n_verify_logit_rows);
    for (int i = 0; i < n; ++i) {
        SeqState& s = c->seqs[ids[i]];
        ((int*)(c->acc_h + a.o_draft0))[i] = s.draft_row0;
        ((int*)(c->acc_h + a.o_verify0))[i] = flags[i] ? s.verify_row0 : 0;
        ((int*)(c->acc_h + a.o_len))[i] = flags[i] ? s.span_len : s.n_masked;
        ((int*)(c->acc_h + a.o_pos0))[i] = s.n_final + s.j;
        ((unsigned*)(c->acc_h + a.o_stream))[i] = s.rng_stream;
        ((int*)(c->acc_h + a.o_step))[i] = s.step;
        ((int*)(c->acc_h + a.o_mode))[i] = flags[i] ? 1 : 0;
    }
    CUDA_TRY(c, cudaEventRecord(c->ev[4], c->stream));
    int rc = launch_accept(c, a, n, c->logits_draft, c->logits_verify, c->d_xhat, c->d_lse, c->d_conf, c->n_draft_logit_rows,
                           c->n_verify_logit_rows);
    if (rc) return rc;
    if ((rc = enqueue_status_read(c))) return rc;
    CUDA_TRY(c, cudaEventRecord(c->ev[5], c->stream));
    CUDA_TRY(c, cudaEventSynchronize(c->ev[5]));
    if ((rc = check_status(c))) return rc;
    float ms = 0;
    cudaEventElapsedTime(&ms, c->ev[4], c->ev[5]);
    c->cnt.ms_accept += ms;
    if (c->verify_timing_pending) {
        cudaEventElapsedTime(&ms, c->ev[2], c->ev[3]);
        c->cnt.ms_verify += ms;
        c->verify_timing_pending = false;
    }
    const int* h_nacc = (const int*)(c->acc_h + a.o_nacc);
    const int* h_rej = (const int*)(c->acc_h + a.o_rej);
    const int* h_res = (const int*)(c->acc_h + a.o_res);
    const int* h_near = (const int*)(c->acc_h + a.o_near);
    const unsigned* h_bits = (const unsigned*)(c->acc_h + a.o_bits);
    for (int i = 0; i < n; ++i) {
        SeqState& s = c->seqs[ids[i]];
        s2d2_step_result& o = res[i];
        memset(&o, 0, sizeof(o));
        o.seq_id = ids[i];
        o.verified = flags[i] ? 1 : 0;
        o.first_reject = -1;
        o.resampled_id = -1;
        int st = s.n_final;
        if (flags[i]) {
            int na = h_nacc[i];
            o.n_accepted = na;
            o.first_reject = h_rej[i];
            o.resampled_id = h_res[i];
            o.n_near_boundary = h_near[i];
            int scanned = h_rej[i] >= 0 ? h_rej[i] + 1 : na;
            for (int k = 0; k < scanned; ++k) {
                o.u[k] = ((const float*)(c->acc_h + a.o_u))[(size_t)i * S2D2_MAX_BLOCK + k];
                o.a[k] = ((const float*)(c->acc_h + a.o_a))[(size_t)i * S2D2_MAX_BLOCK + k];
                o.v[k] = ((const float*)(c->acc_h + a.o_v))[(size_t)i * S2D2_MAX_BLOCK + k];
            }
            for (int k = 0; k < na; ++k) {
                s.tok[st + s.j + k] = s.xhat[k];
                o.committed_idx[o.n_committed] = s.j + k;
                o.committed_tok[o.n_committed++] = s.xhat[k];
            }
            // accepted drafted rows keep their K/V; rows past them are rolled back by length (the right-shifted
            // verifier has no row for the last drafted token: it gets its K/V in the next draft pass)
            if (c->dc.caching == S2D2_CACHE_AR)
                s.n_c += c->dc.verifier_layout == S2D2_VERIFIER_RIGHT_SHIFTED ? std::min(na, s.span_len - 1) : na;
            if (h_rej[i] >= 0 && c->dc.resample) {
                s.tok[st + s.j + na] = h_res[i];
                o.committed_idx[o.n_committed] = s.j + na;
                o.committed_tok[o.n_committed++] = h_res[i];
                c->cnt.n_resampled++;
            }
            c->cnt.n_accepted_tokens += na;
            c->cnt.accepted_len_hist[std::min(na, S2D2_MAX_BLOCK)]++;
            c->cnt.n_near_boundary += h_near[i];
        } else {
            for (int k = 0; k < s.n_masked; ++k)
                if (h_bits[i] >> k & 1) {
                    s.tok[st + s.masked_idx[k]] = s.xhat[k];
                    o.committed_idx[o.n_committed] = s.masked_idx[k];
                    o.committed_tok[o.n_committed++] = s.xhat[k];
                }
        }
        if (c->policy.policy == S2D2_ROUTE_UCB && !c->route_fn && s.ucb_bucket >= 0 && !c->ucb_n.empty()) {
            // reward of the step: tokens it committed / its cost (2 forward passes when verified, else 1)
            const int a = flags[i] ? 1 : 0;
            c->ucb_n[2 * s.ucb_bucket + a] += 1;
            c->ucb_sum[2 * s.ucb_bucket + a] += (double)o.n_committed / (a ? 2.0 : 1.0);
            s.ucb_bucket = -1;
        }
        c->cnt.n_committed_tokens += o.n_committed;
        c->cnt.n_steps++;
        s.step++;
        s.drafted = false;
        s.verify_in_flight = false;
        bool done = true;
        for (int k = 0; k < B; ++k)
            if (s.tok[st + k] == MASK) done = false;
        if (done) {
            s.n_final += B;
            s.block_open = false;
        }
        o.block_done = done;
    }
    if (c->dc.caching == S2D2_CACHE_BLOCK_END) {
        // K^b, V^b <- x_theta(x^b) (Algorithm "Block-wise autoregressive decoding"): one pass over every block that was
        // finished by this step, full attention inside the block, K/V appended
        PassBuild pb;
        std::vector<int> finished;
        for (int i = 0; i < n; ++i) {
            SeqState& s = c->seqs[ids[i]];
            if (!res[i].block_done) continue;
            const int st = s.n_final - B;
            int rc2;
            if ((rc2 = ensure_pages(c, s, s.n_final))) return rc2;
            begin_seq(c, pb, s, st);
            const unsigned long long all_b = B == 64 ? ~0ull : ((1ull << B) - 1);
            for (int k = 0; k < B; ++k) add_row(c, pb, s.tok[st + k], st + k, all_b, ROW_WRITE_KV, false);
            finished.push_back(ids[i]);
        }
        if (pb.n_rows > 0) {
            int rc2 = run_pass(c, pb, nullptr);
            if (rc2) return rc2;
            if ((rc2 = enqueue_status_read(c))) return rc2;
            CUDA_TRY(c, cudaStreamSynchronize(c->stream));      // the row table is reused by the next pass
            if ((rc2 = check_status(c))) return rc2;
            c->cnt.n_cache_passes++;
            for (int id : finished) c->seqs[id].n_c = c->seqs[id].n_final;
        }
    }
    return S2D2_OK;
}

extern "C" int s2d2_accept_logits(s2d2_ctx* c, const float* d_draft, const float* d_verify, int32_t n, int32_t l_max,
                                  const int32_t* span_len, const int32_t* xhat, const int32_t* pos0,
                                  const uint32_t* rng_stream, const int32_t* step, s2d2_step_result* res) {
    if (!c || !d_draft || !d_verify || n < 1 || l_max < 1 || l_max > S2D2_MAX_BLOCK || !span_len || !xhat || !pos0 ||
        !rng_stream || !step || !res)
        return S2D2_ERR_INVALID;
    if (n > c->dc.max_batch || n * l_max > c->max_logit_rows) FAIL(c, S2D2_ERR_INVALID, "accept_logits: batch larger than the context");
    AccStage a(n, (size_t)n * l_max);
    for (int i = 0; i < n; ++i) {
        if (span_len[i] < 0 || span_len[i] > l_max) FAIL(c, S2D2_ERR_INVALID, "accept_logits: span_len");
        for (int k = 0; k < span_len[i]; ++k)
            if (xhat[i * l_max + k] < 0 || xhat[i * l_max + k] >= c->m.vocab) FAIL(c, S2D2_ERR_INVALID, "accept_logits: xhat out of range");
        ((int*)(c->acc_h + a.o_draft0))[i] = i * l_max;
        ((int*)(c->acc_h + a.o_verify0))[i] = i * l_max;
        ((int*)(c->acc_h + a.o_len))[i] = span_len[i];
        ((int*)(c->acc_h + a.o_pos0))[i] = pos0[i];
        ((unsigned*)(c->acc_h + a.o_stream))[i] = rng_stream[i];
        ((int*)(c->acc_h + a.o_step))[i] = step[i];
        ((int*)(c->acc_h + a.o_mode))[i] = 1;
    }
    CUDA_TRY(c, cudaMemcpyAsync(c->d_xhat, xhat, (size_t)n * l_max * 4, cudaMemcpyHostToDevice, c->stream));
    int rc = launch_accept(c, a, n, d_draft, d_verify, c->d_xhat, nullptr, nullptr, n * l_max, n * l_max);
    if (rc) return rc;
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int i = 0; i < n; ++i) {
        s2d2_step_result& o = res[i];
        memset(&o, 0, sizeof(o));
        o.seq_id = i;
        o.verified = 1;
        o.n_accepted = ((const int*)(c->acc_h + a.o_nacc))[i];
        o.first_reject = ((const int*)(c->acc_h + a.o_rej))[i];
        o.resampled_id = ((const int*)(c->acc_h + a.o_res))[i];
        o.n_near_boundary = ((const int*)(c->acc_h + a.o_near))[i];
        int scanned = o.first_reject >= 0 ? o.first_reject + 1 : o.n_accepted;
        for (int k = 0; k < scanned; ++k) {
            o.u[k] = ((const float*)(c->acc_h + a.o_u))[(size_t)i * S2D2_MAX_BLOCK + k];
            o.a[k] = ((const float*)(c->acc_h + a.o_a))[(size_t)i * S2D2_MAX_BLOCK + k];
            o.v[k] = ((const float*)(c->acc_h + a.o_v))[(size_t)i * S2D2_MAX_BLOCK + k];
        }
    }
    return S2D2_OK;
}

extern "C" int s2d2_sample_logits(s2d2_ctx* c, const float* d_logits, int32_t n_rows, int32_t draft_mode, const int32_t* position,
                                  const uint32_t* rng_stream, const int32_t* step, int32_t* xhat_out, float* conf_out,
                                  float* margin_out, float* entropy_out) {
    if (!c || !d_logits || n_rows < 1 || !xhat_out || !conf_out || !margin_out || !entropy_out) return S2D2_ERR_INVALID;
    if (draft_mode != S2D2_DRAFT_GREEDY && draft_mode != S2D2_DRAFT_SAMPLE) FAIL(c, S2D2_ERR_INVALID, "sample_logits: draft_mode");
    if (n_rows > c->max_logit_rows) FAIL(c, S2D2_ERR_INVALID, "sample_logits: more rows than the context holds");
    if (draft_mode == S2D2_DRAFT_SAMPLE) {
        if (!position || !rng_stream || !step) FAIL(c, S2D2_ERR_INVALID, "sample_logits: Philox words missing");
        for (int r = 0; r < n_rows; ++r) {
            c->dsamp_h[r] = position[r];
            c->dsamp_h[n_rows + r] = (int)rng_stream[r];
            c->dsamp_h[2 * n_rows + r] = step[r];
        }
    }
    int rc = launch_draft_stats(c, d_logits, n_rows, draft_mode);
    if (rc) return rc;
    const size_t R = n_rows;
    CUDA_TRY(c, cudaMemcpyAsync(xhat_out, c->d_xhat, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(conf_out, c->d_conf, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(margin_out, c->d_margin, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(entropy_out, c->d_entropy, R * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    return S2D2_OK;
}

// ---------------------------------------------------------------------------------------------
// convenience loop, accessors, test taps
// ---------------------------------------------------------------------------------------------
extern "C" int s2d2_generate(s2d2_ctx* c, int32_t n, const int32_t* ids, int32_t n_new) {
    if (!c || n < 1 || !ids || n_new < 1) return S2D2_ERR_INVALID;
    if (n_new % c->dc.block_size) FAIL(c, S2D2_ERR_INVALID, "n_new_tokens must be a multiple of the block size");
    std::vector<int> target(n);
    for (int i = 0; i < n; ++i) {
        SeqState* s = get_seq(c, ids[i]);
        if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
        target[i] = s->n_final + n_new;
    }
    std::vector<int> live;
    std::vector<s2d2_draft_stats> st(n);
    std::vector<s2d2_step_result> rs(n);
    std::vector<uint8_t> fl(n);
    for (;;) {
        live.clear();
        for (int i = 0; i < n; ++i)
            if (c->seqs[ids[i]].n_final < target[i]) live.push_back(ids[i]);
        if (live.empty()) break;
        int k = (int)live.size(), rc;
        if ((rc = s2d2_draft_block(c, k, live.data(), st.data()))) return rc;
        if ((rc = s2d2_route(c, k, st.data(), fl.data()))) return rc;
        if ((rc = s2d2_verify_block(c, k, live.data(), fl.data()))) return rc;
        if ((rc = s2d2_accept_and_commit(c, k, live.data(), fl.data(), rs.data()))) return rc;
    }
    return S2D2_OK;
}

extern "C" int s2d2_get_tokens(s2d2_ctx* c, int32_t id, int32_t* out, int32_t cap, int32_t* n_out) {
    if (!c || !n_out) return S2D2_ERR_INVALID;
    SeqState* s = get_seq(c, id);
    if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
    *n_out = s->n_final;
    if (out) {
        if (cap < s->n_final) FAIL(c, S2D2_ERR_INVALID, "token buffer too small");
        memcpy(out, s->tok.data(), (size_t)s->n_final * 4);
    }
    return S2D2_OK;
}

extern "C" int s2d2_release_seq(s2d2_ctx* c, int32_t id) {
    if (!c) return S2D2_ERR_INVALID;
    SeqState* s = get_seq(c, id);
    if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
    cudaStreamSynchronize(c->stream);
    for (int p : s->pages) c->free_pages.push_back(p);
    *s = SeqState();
    return S2D2_OK;
}

extern "C" int s2d2_get_counters(s2d2_ctx* c, s2d2_counters* out) {
    if (!c || !out) return S2D2_ERR_INVALID;
    c->cnt.kv_pages_total = c->n_pages;
    c->cnt.kv_pages_in_use = c->n_pages - (int64_t)c->free_pages.size();
    *out = c->cnt;
    return S2D2_OK;
}
extern "C" int s2d2_reset_counters(s2d2_ctx* c) {
    if (!c) return S2D2_ERR_INVALID;
    memset(&c->cnt, 0, sizeof(c->cnt));
    return S2D2_OK;
}

extern "C" int s2d2_set_accept_override(s2d2_ctx* c, float prob) {
    if (!c || !(prob >= 0.f && prob <= 1.f)) return S2D2_ERR_INVALID;
    c->accept_override = prob;
    return S2D2_OK;
}

extern "C" int s2d2_set_profiling(s2d2_ctx* c, int32_t on) {
    if (!c) return S2D2_ERR_INVALID;
    int rc = gemm_prof_collect(c);
    if (rc) return rc;
    if (on && !c->profiling) {
        c->prof_bytes = c->prof_ms_done = 0;
        c->prof_launches = 0;
    }
    c->profiling = on != 0;
    c->tracing = on >= 2;
    return S2D2_OK;
}
extern "C" int s2d2_get_gemm_profile(s2d2_ctx* c, int64_t* n, double* ms, double* bytes) {
    if (!c || !n || !ms || !bytes) return S2D2_ERR_INVALID;
    int rc = gemm_prof_collect(c);
    if (rc) return rc;
    *n = c->prof_launches;
    *ms = c->prof_ms_done;
    *bytes = c->prof_bytes;
    return S2D2_OK;
}

extern "C" int s2d2_debug_copy_logits(s2d2_ctx* c, int32_t which, float* out, int64_t cap, int64_t* n_rows) {
    if (!c || !out || !n_rows || (which != 0 && which != 1)) return S2D2_ERR_INVALID;
    int64_t rows = which == 0 ? c->n_draft_logit_rows : c->n_verify_logit_rows;
    if (cap < rows * c->m.vocab) FAIL(c, S2D2_ERR_INVALID, "logit buffer too small");
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    CUDA_TRY(c, cudaMemcpy(out, which == 0 ? c->logits_draft : c->logits_verify, (size_t)rows * c->m.vocab * 4,
                           cudaMemcpyDeviceToHost));
    *n_rows = rows;
    return S2D2_OK;
}

extern "C" int s2d2_debug_copy_kv(s2d2_ctx* c, int32_t id, int32_t layer, int32_t n_tokens, float* k_out, float* v_out) {
    if (!c || !k_out || !v_out || layer < 0 || layer >= c->m.n_layers) return S2D2_ERR_INVALID;
    SeqState* s = get_seq(c, id);
    if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
    if (n_tokens < 1 || n_tokens > (int)s->pages.size() * c->page_tokens) FAIL(c, S2D2_ERR_INVALID, "n_tokens beyond the allocated pages");
    size_t elems = (size_t)n_tokens * c->m.n_kv_heads * c->m.head_dim;
    float *dk = nullptr, *dv = nullptr;
    int* dp = nullptr;
    CUDA_TRY(c, cudaMalloc(&dk, elems * 4));
    CUDA_TRY(c, cudaMalloc(&dv, elems * 4));
    CUDA_TRY(c, cudaMalloc(&dp, s->pages.size() * 4));
    CUDA_TRY(c, cudaMemcpyAsync(dp, s->pages.data(), s->pages.size() * 4, cudaMemcpyHostToDevice, c->stream));
    if (c->m.dtype == S2D2_DTYPE_F32)
        kv_export_kernel<float><<<dim3(n_tokens, c->m.n_kv_heads), 64, 0, c->stream>>>(make_pool<float>(c), dp, layer, n_tokens, dk, dv);
    else
        kv_export_kernel<bf16><<<dim3(n_tokens, c->m.n_kv_heads), 64, 0, c->stream>>>(make_pool<bf16>(c), dp, layer, n_tokens, dk, dv);
    CUDA_TRY(c, cudaMemcpyAsync(k_out, dk, elems * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(v_out, dv, elems * 4, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    cudaFree(dk);
    cudaFree(dv);
    cudaFree(dp);
    return S2D2_OK;
}

extern "C" int s2d2_debug_seq_state(s2d2_ctx* c, int32_t id, int32_t* n_cached, int32_t* block_start,
                                    int32_t* block_tokens, int32_t* step_index) {
    if (!c) return S2D2_ERR_INVALID;
    SeqState* s = get_seq(c, id);
    if (!s) FAIL(c, S2D2_ERR_INVALID, "bad sequence id");
    if (n_cached) *n_cached = s->n_c;
    if (block_start) *block_start = s->n_final;
    if (step_index) *step_index = s->step;
    if (block_tokens)
        for (int k = 0; k < c->dc.block_size; ++k)
            block_tokens[k] = s->block_open ? s->tok[s->n_final + k] : c->m.vocab;
    return S2D2_OK;
}

extern "C" int s2d2_debug_gemm(s2d2_ctx* c, const void* x, const void* w, int32_t M, int32_t N, int32_t K, float* y) {
    if (!c || !x || !w || !y || M < 1 || N < 1 || K < 1) return S2D2_ERR_INVALID;
    size_t es = esize(c->m.dtype);
    void *dx = nullptr, *dw = nullptr;
    float* dy = nullptr;
    CUDA_TRY(c, cudaMalloc(&dx, (size_t)M * K * es));
    CUDA_TRY(c, cudaMalloc(&dw, (size_t)N * K * es));
    CUDA_TRY(c, cudaMalloc((void**)&dy, (size_t)M * N * 4));
    CUDA_TRY(c, cudaMemcpyAsync(dx, x, (size_t)M * K * es, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(dw, w, (size_t)N * K * es, cudaMemcpyHostToDevice, c->stream));
    int rc = gemm(c, dx, dw, dy, M, N, K, N, 1.f, 0);
    if (!rc) rc = enqueue_status_read(c);
    if (!rc) {
        CUDA_TRY(c, cudaMemcpyAsync(y, dy, (size_t)M * N * 4, cudaMemcpyDeviceToHost, c->stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        rc = check_status(c);
    }
    gemm_forget(c, dx);
    gemm_forget(c, dw);
    cudaFree(dx);
    cudaFree(dw);
    cudaFree(dy);
    return rc;
}

extern "C" int s2d2_debug_gemm2(s2d2_ctx* c, const void* x_hi, const void* x_lo, const void* w, int32_t M, int32_t N, int32_t K,
                                float scale, int32_t accumulate, float* y) {
    if (!c || !x_hi || !w || !y || M < 1 || N < 1 || K < 1) return S2D2_ERR_INVALID;
    if (c->m.dtype != S2D2_DTYPE_BF16) FAIL(c, S2D2_ERR_UNSUPPORTED, "debug_gemm2: bf16 models only");
    void *dx = nullptr, *dl = nullptr, *dw = nullptr;
    float* dy = nullptr;
    CUDA_TRY(c, cudaMalloc(&dx, (size_t)M * K * 2));
    CUDA_TRY(c, cudaMalloc(&dl, (size_t)M * K * 2));
    CUDA_TRY(c, cudaMalloc(&dw, (size_t)N * K * 2));
    CUDA_TRY(c, cudaMalloc((void**)&dy, (size_t)M * N * 4));
    CUDA_TRY(c, cudaMemcpyAsync(dx, x_hi, (size_t)M * K * 2, cudaMemcpyHostToDevice, c->stream));
    if (x_lo) CUDA_TRY(c, cudaMemcpyAsync(dl, x_lo, (size_t)M * K * 2, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(dw, w, (size_t)N * K * 2, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(dy, y, (size_t)M * N * 4, cudaMemcpyHostToDevice, c->stream));
    int rc = gemm(c, dx, dw, dy, M, N, K, N, scale, accumulate, x_lo ? dl : nullptr);
    if (!rc) rc = enqueue_status_read(c);
    if (!rc) {
        CUDA_TRY(c, cudaMemcpyAsync(y, dy, (size_t)M * N * 4, cudaMemcpyDeviceToHost, c->stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        rc = check_status(c);
    }
    gemm_forget(c, dx);
    gemm_forget(c, dl);
    gemm_forget(c, dw);
    cudaFree(dx);
    cudaFree(dl);
    cudaFree(dw);
    cudaFree(dy);
    return rc;
}

extern "C" int s2d2_debug_gemm_swiglu(s2d2_ctx* c, const void* x_hi, const void* x_lo, const void* w, int32_t M, int32_t f, int32_t K,
                                      uint16_t* act_hi, uint16_t* act_lo) {
    if (!c || !x_hi || !x_lo || !w || !act_hi || !act_lo || M < 1 || f < 1 || K < 1) return S2D2_ERR_INVALID;
    if (c->m.dtype != S2D2_DTYPE_BF16) FAIL(c, S2D2_ERR_UNSUPPORTED, "debug_gemm_swiglu: bf16 models only");
    void *dx = nullptr, *dl = nullptr, *dw = nullptr, *dh = nullptr, *dlo = nullptr;
    CUDA_TRY(c, cudaMalloc(&dx, (size_t)M * K * 2));
    CUDA_TRY(c, cudaMalloc(&dl, (size_t)M * K * 2));
    CUDA_TRY(c, cudaMalloc(&dw, (size_t)2 * f * K * 2));
    CUDA_TRY(c, cudaMalloc(&dh, (size_t)M * f * 2));
    CUDA_TRY(c, cudaMalloc(&dlo, (size_t)M * f * 2));
    CUDA_TRY(c, cudaMemcpyAsync(dx, x_hi, (size_t)M * K * 2, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(dl, x_lo, (size_t)M * K * 2, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(dw, w, (size_t)2 * f * K * 2, cudaMemcpyHostToDevice, c->stream));
    int rc = gemm_swiglu(c, dx, dl, dw, M, f, K, dh, dlo);
    if (rc < 0) {
        c->err = "debug_gemm_swiglu: this shape takes the separate GEMM and SwiGLU kernels (needs M > 64, f % 128 == 0, K % 64 == 0)";
        rc = S2D2_ERR_UNSUPPORTED;
    }
    if (!rc) rc = enqueue_status_read(c);
    if (!rc) {
        CUDA_TRY(c, cudaMemcpyAsync(act_hi, dh, (size_t)M * f * 2, cudaMemcpyDeviceToHost, c->stream));
        CUDA_TRY(c, cudaMemcpyAsync(act_lo, dlo, (size_t)M * f * 2, cudaMemcpyDeviceToHost, c->stream));
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        rc = check_status(c);
    }
    gemm_forget(c, dx);
    gemm_forget(c, dl);
    gemm_forget(c, dw);
    cudaFree(dx);
    cudaFree(dl);
    cudaFree(dw);
    cudaFree(dh);
    cudaFree(dlo);
    return rc;
}

extern "C" int s2d2_debug_copy_expert_ids(s2d2_ctx* c, int32_t* out, int64_t cap, int32_t* n_rows) {
    if (!c || !out || !n_rows) return S2D2_ERR_INVALID;
    if (c->m.n_experts == 0) FAIL(c, S2D2_ERR_UNSUPPORTED, "not a MoE model");
    int M = c->last_pass_rows, k = c->m.top_k;
    if (cap < (int64_t)c->m.n_layers * M * k) FAIL(c, S2D2_ERR_INVALID, "buffer too small");
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
    for (int l = 0; l < c->m.n_layers; ++l)
        CUDA_TRY(c, cudaMemcpy(out + (size_t)l * M * k, c->moe_ids_trace + (size_t)l * c->max_rows * k, (size_t)M * k * 4,
                               cudaMemcpyDeviceToHost));
    *n_rows = M;
    return S2D2_OK;
}

extern "C" int s2d2_debug_pass_trace(s2d2_ctx* c, uint64_t* out, int64_t cap, int32_t* n_ctas, int32_t* n_marks) {
    if (!c || !out || !n_ctas || !n_marks) return S2D2_ERR_INVALID;
    return pass_copy_trace(c, (unsigned long long*)out, cap, n_ctas, n_marks);
}

extern "C" int s2d2_debug_wait_timeout(s2d2_ctx* c, uint32_t target, uint32_t limit_polls) {
    if (!c || limit_polls == 0 || limit_polls > (1u << 20)) return S2D2_ERR_INVALID;
    // the word polled is the status word's neighbour in a zeroed 8-byte allocation: nothing ever sets it
    unsigned* word = nullptr;
    CUDA_TRY(c, cudaMalloc((void**)&word, 8));
    CUDA_TRY(c, cudaMemsetAsync(word, 0, 8, c->stream));
    bounded_wait_probe_kernel<<<1, 1, 0, c->stream>>>(word, target, limit_polls, c->d_status);
    LAUNCHED(c);
    int rc = enqueue_status_read(c);
    if (!rc) {
        CUDA_TRY(c, cudaStreamSynchronize(c->stream));
        rc = check_status(c);
    }
    cudaFree(word);
    return rc;
}
