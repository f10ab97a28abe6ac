// Host-side state of an S2D2 context: configuration, device buffers, the paged
// KV allocator and the per-sequence decode state.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/s2d2.h"
#include "common.cuh"

namespace s2d2 {

struct WeightSlot {
    void* d_ptr = nullptr;      // destination on the device
    size_t bytes = 0;
    int dtype = 0;
    bool loaded = false;
};

struct LayerWeights {
    float *attn_norm = nullptr, *ffn_norm = nullptr, *q_norm = nullptr, *k_norm = nullptr;
    void *wqkv = nullptr, *wo = nullptr, *wgu = nullptr, *wdown = nullptr;            // dense
    void *router = nullptr, *e_gate = nullptr, *e_up = nullptr, *e_down = nullptr;    // routed experts
    void *s_gu = nullptr, *s_down = nullptr;                                          // shared expert
};

struct SeqState {
    bool active = false;
    uint32_t rng_stream = 0;
    std::vector<int> tok;       // finalised tokens followed by the open block (vocab = MASK)
    int n_final = 0;            // finalised tokens = start of the open block
    int n_prompt = 0;
    bool block_open = false;
    int n_c = 0;                // tokens whose K/V is committed in the cache
    int step = 0;               // draft passes so far (Philox step word)
    std::vector<int> pages;
    // result of the last draft pass
    bool drafted = false;
    int j = 0, n_masked = 0, span_len = 0;
    int masked_idx[S2D2_MAX_BLOCK];
    int xhat[S2D2_MAX_BLOCK];
    float conf[S2D2_MAX_BLOCK];
    int draft_row0 = 0;         // first row of this sequence in the draft-logit buffer
    bool verify_in_flight = false;
    int verify_row0 = 0;        // first row in the verifier-logit buffer
    bool hyst_on = true;
    // which draft / verifier pass of the context produced the logit rows this sequence refers to
    unsigned long long draft_stamp = 0, verify_stamp = 0;
    int ucb_bucket = -1;        // context bucket of the bandit router's last decision for this sequence (-1: none pending)
};

// Fixed-layout staging area for the metadata of one pass (pinned host mirror and
// device copy have the same layout, so pointers into the device copy never change).
struct PassMeta {
    int cap_rows = 0, cap_seqs = 0, max_pages = 0;
    size_t bytes = 0;
    char* h = nullptr;          // pinned
    char* d = nullptr;
    size_t off_token, off_pos, off_seq, off_flags, off_mask, off_logit_rows, off_nctx, off_row0, off_nrows, off_pages;
    template <typename T> T* hp(size_t off) const { return reinterpret_cast<T*>(h + off); }
    template <typename T> T* dp(size_t off) const { return reinterpret_cast<T*>(d + off); }
};

}  // namespace s2d2

struct s2d2_ctx {
    s2d2_model_config m;
    s2d2_decode_config dc;
    cudaStream_t stream = nullptr;
    std::string err;
    int device = 0;

    // weights
    char* w_arena = nullptr;
    size_t w_bytes = 0;
    std::unordered_map<std::string, s2d2::WeightSlot> slots;
    std::vector<s2d2::LayerWeights> layers;
    void* embed = nullptr;
    void* lm_head = nullptr;
    float* final_norm = nullptr;
    bool weights_checked = false;

    // KV pool
    void* kv_base = nullptr;
    int n_pages = 0, page_tokens = 64, page_shift = 6, max_pages_per_seq = 0;
    std::vector<int> free_pages;

    // sequences
    std::vector<s2d2::SeqState> seqs;

    // scratch (device)
    int max_rows = 0, max_logit_rows = 0;
    float *h = nullptr, *qkv = nullptr, *gu = nullptr, *tmp = nullptr;
    void *xn = nullptr, *q = nullptr, *k_rows = nullptr, *v_rows = nullptr, *attn = nullptr, *act = nullptr;
    // low halves of the two-term activations (bf16 models): x = hi + lo
    void *xn_lo = nullptr, *q_lo = nullptr, *attn_lo = nullptr, *act_lo = nullptr;
    float *logits_draft = nullptr, *logits_verify = nullptr;
    float *rope_cos = nullptr, *rope_sin = nullptr;
    // MoE scratch
    float *router_logits = nullptr, *moe_gates = nullptr, *moe_gu = nullptr, *moe_out = nullptr;
    int* moe_ids = nullptr;
    void* moe_act = nullptr;
    int* moe_ids_trace = nullptr;   // [n_layers, max_rows, top_k]
    int last_pass_rows = 0;

    s2d2::PassMeta meta;

    // draft statistics and acceptance outputs (device + pinned host mirrors)
    int *d_xhat = nullptr;
    float *d_conf = nullptr, *d_margin = nullptr, *d_entropy = nullptr;
    double* d_lse = nullptr;
    void *chunk_d = nullptr, *chunk_v = nullptr;   // per (logit row, vocabulary chunk) statistics of the two passes
    void* rej_info = nullptr;                      // per sequence: the rejected position to resample
    double *res_rsum = nullptr, *res_vsum = nullptr;   // per (sequence, chunk) residual and pi_v mass
    char *acc_h = nullptr, *acc_d = nullptr;      // staging for the acceptance kernel's inputs and outputs
    size_t acc_bytes = 0;
    unsigned* acc_tickets = nullptr;               // per sequence of an acceptance launch: CTAs done so far (zero between launches)
    char* stats_h = nullptr;                       // pinned mirror of the draft statistics
    int *dsamp_h = nullptr, *dsamp_d = nullptr;    // draft sampling: per logit row position, Philox stream, step (pinned / device)
    int n_draft_logit_rows = 0, n_verify_logit_rows = 0;
    // The logits of a pass live in per-context buffers that the next pass of the same kind overwrites; the passes
    // are numbered so that a sequence whose rows have been overwritten is recognised (S2D2_ERR_STATE).
    unsigned long long draft_gen = 0, verify_gen = 0;

    // routing
    s2d2_route_fn route_fn = nullptr;
    void* route_user = nullptr;
    s2d2_route_policy policy;
    // contextual-bandit router: decisions so far, and per (bucket, action) the count and the summed reward
    long long ucb_t = 0;
    std::vector<long long> ucb_n;
    std::vector<double> ucb_sum;

    // counters / timing
    s2d2_counters cnt;
    cudaEvent_t ev[8];
    bool verify_timing_pending = false;
    // per-GEMM profiling (off by default)
    bool profiling = false;
    float accept_override = 0.f;            // > 0: every accept test is u < accept_override (throughput studies)
    bool tracing = false;                   // in-kernel phase marks of the persistent pass
    std::vector<cudaEvent_t> prof_events;   // pairs
    size_t prof_used = 0;
    double prof_bytes = 0, prof_ms_done = 0;
    int64_t prof_launches = 0;
    void* gemm_state = nullptr;             // owned by gemm.cu
    void* attn_state = nullptr;             // owned by attention.cu
    void* pass_state = nullptr;             // owned by pass.cu
    int* d_status = nullptr;                // raised by a kernel whose bounded wait ran out
    int* h_status = nullptr;                // pinned mirror
};
