/*
 * s2d2.h - C ABI of the B200-native S2D2 decode step.
 *
 * S2D2 (training-free self-speculation for block-diffusion language models)
 * decodes a block of B masked tokens by repeating: one *draft* pass of the
 * network over the block (bidirectional inside the block, attending to the
 * cached prefix), a host-side *routing* decision, one *verify* pass of the same
 * weights in block-size-1 (autoregressive) mode over the first contiguous masked
 * span, speculative *acceptance* left to right with residual resampling at the
 * first rejection, and *commit* of the accepted prefix to the KV cache
 * (Algorithm "Block-wise autoregressive decoding", Algorithm "SampleBlock for
 * S2D2").  Naming: pi_d is the drafter's distribution (the paper's P_l, with
 * p_i for the drafted token), pi_v the verifier's (P_l^ver, q_i).
 *
 * Conventions
 *   - Every call returns 0 (S2D2_OK) or a negative s2d2_status; the text of the
 *     last error of a context is given by s2d2_last_error().  Nothing aborts.
 *   - All pointers are HOST pointers unless the name starts with d_ (device).
 *   - The caller owns every buffer it passes; the library copies what it keeps.
 *     The library owns the device copy of the weights, the KV page pool, its
 *     scratch memory and the per-sequence state, all released by s2d2_destroy().
 *   - All device work of a context runs on the CUDA stream given at creation.
 *     Calls that return results to the host synchronise that stream.
 *   - One context is not thread safe; use one context per thread.
 */
#ifndef S2D2_H
#define S2D2_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define S2D2_MAX_BLOCK 32          /* largest block size B                       */
#define S2D2_MAX_ROWS_PER_SEQ 64   /* rows one sequence contributes to one pass  */

typedef enum {
    S2D2_OK = 0,
    S2D2_ERR_INVALID = -1,      /* bad argument or handle                        */
    S2D2_ERR_CUDA = -2,         /* a CUDA call failed (text in last_error)       */
    S2D2_ERR_OOM = -3,          /* KV page pool or sequence slots exhausted      */
    S2D2_ERR_STATE = -4,        /* call out of order for this sequence           */
    S2D2_ERR_TIMEOUT = -5,      /* a bounded device-side wait ran out            */
    S2D2_ERR_UNSUPPORTED = -6,  /* shape outside what the kernels support        */
    S2D2_ERR_MISSING_WEIGHT = -7
} s2d2_status;

enum { S2D2_DTYPE_F32 = 0, S2D2_DTYPE_BF16 = 1 };
/* SampleFromLogits: GREEDY proposes the argmax (ties -> lowest id); SAMPLE draws the proposal from pi_d by
 * inverse CDF in vocabulary order with one uniform of the draft-sampling Philox stream (only then is the
 * output law of the speculative step exactly the verifier's: Section "Background", speculative decoding).
 * In both modes the confidence is pi_d(proposal); margin and entropy describe pi_d itself. */
enum { S2D2_DRAFT_GREEDY = 0, S2D2_DRAFT_SAMPLE = 1 };
/* How the verifier pass is laid out (Section "Self-Verification Mode").
 * ALIGNED_2L: position-aligned models; 2L rows [drafted span ; L MASK copies] under Eq. (ver_mask), the logits
 *   of the row at position i score position i.
 * RIGHT_SHIFTED: models whose logits at position i - 1 score the token at position i; "the standard causal
 *   mask already provides the verifier view": L causal rows [last committed token, drafted tokens but the
 *   last], row k scores drafted token k + 1.  The draft pass reads its logits one row to the left in the same
 *   way, and every pass starts with the row of the last committed token. */
enum { S2D2_VERIFIER_ALIGNED_2L = 0, S2D2_VERIFIER_RIGHT_SHIFTED = 1 };
/* When the K/V of a block enter the cache (Algorithm "Block-wise autoregressive decoding"; Section
 * "Self-Verification Mode", Eq. (draft_mask)).
 * AR: the partially causal drafting/caching mask: committed tokens are causal rows, their K/V is final and enters
 *   the cache as they are committed (accepted drafted tokens keep the K/V of their verifier rows).
 * BLOCK_END: the standard block-diffusion pattern: every row of the block sees the whole block in the draft
 *   pass, nothing of the block is cached while it is decoded (the verifier pass carries the block's committed
 *   prefix as causal rows), and when the block has no MASK left s2d2_accept_and_commit runs one more pass over
 *   it, with full attention inside the block, whose K/V are appended.  Aligned verifier layout only. */
enum { S2D2_CACHE_AR = 0, S2D2_CACHE_BLOCK_END = 1 };

/* The network (the paper treats x_theta as given; these fields describe the
 * decoder shapes of the synthetic workloads). Matrices are [out, in], y = x W^T. */
typedef struct {
    int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim;
    int32_t ffn;                /* dense SwiGLU width; 0 for MoE models          */
    int32_t vocab;              /* [MASK] is embedding row `vocab`               */
    int32_t dtype;              /* S2D2_DTYPE_*: storage type of the matrices    */
    int32_t qk_norm;            /* per-head RMSNorm on q and k before RoPE       */
    int32_t n_experts, top_k, expert_ffn, n_shared;   /* MoE; n_experts = 0: dense */
    float rope_base, rms_eps, logit_scale;
} s2d2_model_config;

/* Decoding parameters (Algorithm "SampleBlock for S2D2": B, tau; Appendix
 * "ratio tempering": gamma). */
typedef struct {
    int32_t block_size;         /* B, 1..S2D2_MAX_BLOCK                          */
    int32_t max_batch;          /* sequences alive at once                       */
    int32_t max_seq_len;        /* prompt + generated tokens per sequence        */
    int32_t kv_page_tokens;     /* tokens per KV page (power of two, <= 64)      */
    int32_t n_kv_pages;         /* pool size; 0 = max_batch*ceil(max_seq_len/page) */
    int32_t draft_mode;         /* S2D2_DRAFT_GREEDY | S2D2_DRAFT_SAMPLE         */
    int32_t resample;           /* 1: draw from the residual at a rejection      */
    float tau_conf;             /* threshold of the confidence branch            */
    float ratio_gamma;          /* accept iff u < min(1, (v/d)^gamma)            */
    uint32_t seed;              /* Philox key                                    */
    int32_t use_tensor_cores;   /* 1: default. 0: portable SIMT kernels only (debug).
                                   2: tensor-core kernels, one per operation (no persistent pass kernel).
                                   3: as 1, with every GEMM of the persistent pass kernel cut into sub-GEMMs wherever
                                   its tile counts allow (test setting: a small model then runs the same
                                   tile-by-tile hand-overs between GEMMs that a large one runs by default) */
    int32_t verifier_layout;    /* S2D2_VERIFIER_*                               */
    int32_t caching;            /* S2D2_CACHE_*                                  */
} s2d2_decode_config;

typedef struct {
    const char* name;           /* e.g. "layers.3.wq", "embed", "lm_head"        */
    int32_t dtype;              /* S2D2_DTYPE_*; must match the model for matrices; gains are fp32 */
    int32_t ndim;
    int64_t shape[4];
    const void* data;           /* host pointer, row-major                       */
} s2d2_tensor_desc;

/* Per-sequence result of a draft pass: SampleFromLogits on every masked
 * position of the block plus the quantities routing needs (Section
 * "Verification Routing Policies"). Arrays are indexed 0..n_masked-1. */
typedef struct {
    int32_t seq_id;
    int32_t block_start;        /* absolute position of the block's first token  */
    int32_t first_masked;       /* j: first masked in-block index                */
    int32_t n_masked;           /* |M_t|                                         */
    int32_t span_len;           /* |C_t|: first contiguous masked span           */
    int32_t n_hi;               /* #{i in M_t : conf_i > tau_conf}               */
    float mean_conf;            /* mean of conf over M_t                         */
    int32_t masked_idx[S2D2_MAX_BLOCK];   /* in-block indices of M_t, ascending  */
    int32_t xhat[S2D2_MAX_BLOCK];         /* proposed token                      */
    float conf[S2D2_MAX_BLOCK];           /* d_i = pi_d,i(xhat_i)                */
    float margin[S2D2_MAX_BLOCK];         /* top-1 minus top-2 draft probability */
    float entropy[S2D2_MAX_BLOCK];        /* entropy of pi_d,i in nats           */
} s2d2_draft_stats;

/* Per-sequence result of one step (accept scan or confidence branch). */
typedef struct {
    int32_t seq_id;
    int32_t verified;           /* 1: acceptance scan ran; 0: confidence branch  */
    int32_t n_accepted;         /* accepted drafted tokens (prefix of the span)  */
    int32_t first_reject;       /* index in the span, -1 if none                 */
    int32_t resampled_id;       /* token drawn from the residual, -1 if none     */
    int32_t n_committed;        /* tokens written to the block this step         */
    int32_t block_done;         /* 1: the block has no MASK left                 */
    int32_t n_near_boundary;    /* scanned positions with |u - a| < 1e-4         */
    int32_t committed_idx[S2D2_MAX_BLOCK];   /* in-block indices written         */
    int32_t committed_tok[S2D2_MAX_BLOCK];
    float u[S2D2_MAX_BLOCK];    /* accept uniforms of the scanned positions      */
    float a[S2D2_MAX_BLOCK];    /* min(1,(v/d)^gamma) of the scanned positions   */
    float v[S2D2_MAX_BLOCK];    /* verifier probability of the drafted token     */
} s2d2_step_result;

typedef struct {
    int64_t n_draft_passes, n_verify_passes, n_prefill_passes;
    int64_t n_steps, n_committed_tokens, n_accepted_tokens, n_resampled, n_near_boundary;
    int64_t n_kernel_launches;      /* kernels of this library launched so far   */
    int64_t accepted_len_hist[S2D2_MAX_BLOCK + 1];
    double ms_draft, ms_verify, ms_accept, ms_prefill;  /* device time, CUDA events */
    int64_t kv_pages_in_use, kv_pages_total;
    int64_t moe_expert_tiles_touched;                   /* (layer, expert) pairs streamed */
    int64_t h2d_bytes, d2h_bytes;                       /* host<->device copies made by the calls */
    int64_t n_rows_draft, n_rows_verify, n_rows_prefill; /* token rows the passes of each kind carried, summed */
    int64_t n_cache_passes;                             /* end-of-block cache passes (S2D2_CACHE_BLOCK_END) */
} s2d2_counters;

typedef struct s2d2_ctx s2d2_ctx;

/* Create a context: allocates the KV page pool, scratch and tables on the
 * current device. `cuda_stream` is a cudaStream_t (NULL = default stream). */
int s2d2_create(const s2d2_model_config* m, const s2d2_decode_config* dc, void* cuda_stream, s2d2_ctx** out);
int s2d2_destroy(s2d2_ctx* ctx);
const char* s2d2_last_error(const s2d2_ctx* ctx);

/* Copy the network's tensors to the device (names as produced by the weight
 * generator: embed [(V+1), d]; layers.N.{attn_norm,wq,wk,wv,wo,q_norm,k_norm,
 * ffn_norm,w_gate,w_up,w_down | router, experts.w_gate [E,f,d], experts.w_up,
 * experts.w_down [E,d,f], shared.w_*}; final_norm; lm_head [V, d]).  May be
 * called several times with disjoint subsets; every tensor must have arrived
 * before the first s2d2_prefill (else S2D2_ERR_MISSING_WEIGHT). */
int s2d2_load_weights(s2d2_ctx* ctx, const s2d2_tensor_desc* tensors, int32_t n_tensors);

/* Algorithm "Block-wise autoregressive decoding", first line: x <- prompt and
 * the KV cache of the prompt.  Runs a causal pass over each prompt (in chunks)
 * and fills KV pages; returns one sequence id per prompt. Synchronous. */
int s2d2_prefill(s2d2_ctx* ctx, int32_t n_seqs, const int32_t* const* prompt_ids,
                 const int32_t* prompt_lens, int32_t* seq_ids_out);

/* The sequence-stream word of the Philox counter (default: the sequence id). */
int s2d2_seq_set_rng_stream(s2d2_ctx* ctx, int32_t seq_id, uint32_t stream);

/* Draft pass (Algorithm "SampleBlock for S2D2": "draft forward" and
 * SampleFromLogits; mask of Eq. (draft_mask)).  Opens a new block of B MASKs
 * for a sequence that has none.  Rows per sequence: committed tokens not yet in
 * the cache (causal; their K/V is appended) followed by the block from its
 * first masked position (these see the whole pass).  Fills stats_out[n_seqs].
 * Synchronous (routing needs the stats on the host).  With S2D2_VERIFIER_RIGHT_SHIFTED the logits
 * that score in-block position i are those of the row at position i - 1, so the pass always carries
 * the last committed token as its first row (run again if its K/V is cached already).
 * The logits of a draft pass and of a verifier pass live in per-context buffers, so one step uses one id
 * list: every draft_block overwrites the previous one's rows.  A sequence drafted by an earlier call that has
 * not been through accept_and_commit since is refused by verify_block and accept_and_commit (S2D2_ERR_STATE)
 * and has to be drafted again, which is allowed (the repeated draft uses the same uniforms).  Likewise a
 * second verify_block with a flagged sequence before accept_and_commit is refused. */
int s2d2_draft_block(s2d2_ctx* ctx, int32_t n_seqs, const int32_t* seq_ids, s2d2_draft_stats* stats_out);

/* Routing hook (Algorithm "DoVerify"): return non-zero to verify the span. */
typedef int (*s2d2_route_fn)(void* user, const s2d2_draft_stats* st);
enum {
    S2D2_ROUTE_MIN_SPAN = 0,      /* |C_t| >= p0 (default, p0 = 1: always verify)              */
    S2D2_ROUTE_SCORE = 1,         /* K_hat - c[*N_hi] >= tau_score                              */
    S2D2_ROUTE_HYSTERESIS = 2,    /* on/off thresholds on the same score, state per sequence    */
    S2D2_ROUTE_MEAN_CONF = 3,     /* mean draft confidence over M_t < p0                        */
    S2D2_ROUTE_NEVER = 4,
    S2D2_ROUTE_UCB = 5            /* contextual bandit (Appendix "Contextual-bandit routing policy", Eq. (ucb)):
                                     p0 = beta, p1 = bins per context dimension (0: the paper's default, 2).  Context
                                     bucket = (span-length bin over 1..B, fraction of the block already unmasked,
                                     mean over the span of H_i / log V); per bucket and action the mean reward
                                     (tokens committed by the step / cost, cost 2 for a verified step, 1 otherwise)
                                     and the count; the action maximises mean + beta * sqrt(log t / count), an
                                     action not yet taken in the bucket goes first, ties verify.  One table per
                                     context; s2d2_accept_and_commit feeds the rewards back (with the flags it is
                                     given as the action taken).  s2d2_set_route_policy clears the table. */
};
typedef struct {
    int32_t policy;
    float p0;                     /* tau_span | tau_score | tau_on | confidence threshold       */
    float p1;                     /* tau_off (hysteresis)                                       */
    float cost;                   /* c                                                          */
    int32_t dynamic_cost;         /* 1: s = K_hat - c * N_hi                                    */
    int32_t alpha_entropy;        /* 0: margin proxy 1[m_i >= alpha_param]; 1: exp(-alpha_param * H_i / log V) */
    float alpha_param;            /* tau_margin | beta                                          */
} s2d2_route_policy;
int s2d2_set_router(s2d2_ctx* ctx, s2d2_route_fn fn, void* user);      /* fn = NULL: built-in policy */
int s2d2_set_route_policy(s2d2_ctx* ctx, const s2d2_route_policy* p);
/* Evaluate the router (hook or built-in policy) on stats: flags_out[i] = 1 to verify. */
int s2d2_route(s2d2_ctx* ctx, int32_t n_seqs, const s2d2_draft_stats* stats, uint8_t* flags_out);

/* Verifier pass (Section "Self-Verification Mode", the 2L construction and
 * Eq. (ver_mask)): for every flagged sequence 2L rows [drafted span ; L MASK
 * copies at the same positions]; K/V of the drafted rows is appended
 * speculatively to the cache pages.  With S2D2_VERIFIER_RIGHT_SHIFTED: L causal rows
 * [last committed token ; drafted tokens but the last], K/V of the drafted rows appended
 * speculatively (the last drafted token gets its K/V in the next draft pass). Asynchronous. */
int s2d2_verify_block(s2d2_ctx* ctx, int32_t n_seqs, const int32_t* seq_ids, const uint8_t* verify_flags);

/* Acceptance and commit (Algorithm "SampleBlock for S2D2", the left-to-right
 * loop and the else-branch): verified sequences accept drafted token i iff
 * u_i < min(1, (v_i/d_i)^gamma), stop at the first rejection and resample it from
 * (pi_v - pi_d)_+; the accepted prefix's K/V stays in the cache, the rest is
 * rolled back.  Other sequences commit {i: d_i > tau_conf} plus the most
 * confident masked position.  Fills res_out[n_seqs]. Synchronous. */
int s2d2_accept_and_commit(s2d2_ctx* ctx, int32_t n_seqs, const int32_t* seq_ids,
                           const uint8_t* verify_flags, s2d2_step_result* res_out);

/* Convenience loop draft -> route -> verify -> accept until every listed
 * sequence has n_new_tokens generated tokens (a multiple of B). */
int s2d2_generate(s2d2_ctx* ctx, int32_t n_seqs, const int32_t* seq_ids, int32_t n_new_tokens);

/* Finalised tokens of a sequence (prompt included), without the open block. */
int s2d2_get_tokens(s2d2_ctx* ctx, int32_t seq_id, int32_t* out, int32_t cap, int32_t* n_out);
int s2d2_release_seq(s2d2_ctx* ctx, int32_t seq_id);
int s2d2_get_counters(s2d2_ctx* ctx, s2d2_counters* out);
int s2d2_reset_counters(s2d2_ctx* ctx);

/* Throughput studies on models whose acceptance profile is not the one of interest (random
 * weights accept far fewer tokens than the trained models of the paper's Table "Per-token
 * draft-confidence versus verifier-ratio analysis", whose quadrants average to 0.77 per verified
 * token).  prob in (0, 1]: the accept test of every scanned position becomes u_i < prob, whatever
 * the two distributions say; a rejected position is still resampled from the residual.  The
 * output no longer follows the verifier's law, so such a run measures speed only.  prob = 0
 * restores the rule of Algorithm "SampleBlock for S2D2".  S2D2_ERR_INVALID outside [0, 1]. */
int s2d2_set_accept_override(s2d2_ctx* ctx, float prob);

/* Kernel-level timing for roofline reports.  on >= 1: the dominant launches of the forward
 * pass (the persistent pass kernel; on the one-kernel-per-operation path every GEMM) are
 * bracketed by a CUDA event pair on the context's stream.  on >= 2: the persistent kernel also
 * records its phase marks (s2d2_debug_pass_trace), which costs it a few percent.
 * s2d2_get_gemm_profile synchronises and returns the bracketed launches, their summed device
 * time and their summed algorithmic bytes (every weight matrix read once, the cached K/V of the
 * pass's sequences read once, K/V rows and logits written; for a single GEMM: weights +
 * activations read + output written) since profiling was switched on. */
int s2d2_set_profiling(s2d2_ctx* ctx, int32_t on);
int s2d2_get_gemm_profile(s2d2_ctx* ctx, int64_t* n_launches, double* total_ms, double* total_bytes);

/* Stand-alone entry to the fused acceptance kernel on caller-supplied device
 * logits (Algorithm "SampleBlock for S2D2", ScoreFromLogits and the scan).
 * d_draft_logits / d_verify_logits: fp32 [n_seqs * L_max, vocab], row
 * s*L_max + i = position i of sequence s; span_len[s] <= L_max rows are used;
 * xhat [n_seqs*L_max] proposals; position0[s] absolute position of the span's
 * first token; rng_stream[s], step[s] Philox counter words.  Host outputs:
 * res_out[n_seqs] (committed_* fields not filled). Synchronous. */
int s2d2_accept_logits(s2d2_ctx* ctx, const float* d_draft_logits, const float* d_verify_logits,
                       int32_t n_seqs, int32_t l_max, const int32_t* span_len, const int32_t* xhat,
                       const int32_t* position0, const uint32_t* rng_stream, const int32_t* step,
                       s2d2_step_result* res_out);

/* Stand-alone entry to the SampleFromLogits kernels on caller-supplied device logits (Algorithm
 * "SampleBlock for S2D2", SampleFromLogits; Section "Verification Routing Policies" for margin and
 * entropy).  d_logits: fp32 [n_rows, vocab]; draft_mode S2D2_DRAFT_*; position[r], rng_stream[r], step[r]:
 * Philox counter words of row r (read in SAMPLE mode only, may be NULL for GREEDY).  Host outputs, each
 * [n_rows]: proposal, its probability, top-1 minus top-2 probability, entropy in nats.  n_rows is at most
 * max_batch * block_size of the context.  Synchronous. */
int s2d2_sample_logits(s2d2_ctx* ctx, const float* d_logits, int32_t n_rows, int32_t draft_mode,
                       const int32_t* position, const uint32_t* rng_stream, const int32_t* step,
                       int32_t* xhat_out, float* conf_out, float* margin_out, float* entropy_out);

/* Test taps. which: 0 = logits of the last draft pass (rows = masked positions
 * of the listed sequences in call order), 1 = last verify pass (rows = span
 * positions of the verified sequences in call order). */
int s2d2_debug_copy_logits(s2d2_ctx* ctx, int32_t which, float* out, int64_t cap_floats, int64_t* n_rows_out);
/* K and V of cache positions [0, n_tokens) of one layer, widened to fp32,
 * each [n_tokens, n_kv_heads, head_dim]. */
int s2d2_debug_copy_kv(s2d2_ctx* ctx, int32_t seq_id, int32_t layer, int32_t n_tokens, float* k_out, float* v_out);
/* Cache length (tokens whose K/V is committed) and open-block state. */
int s2d2_debug_seq_state(s2d2_ctx* ctx, int32_t seq_id, int32_t* n_cached, int32_t* block_start,
                         int32_t* block_tokens /* [B], vocab = MASK, may be NULL */, int32_t* step_index);
/* One GEMM of the forward pass on host data (test tap): y[M,N] = x[M,K] w[N,K]^T with
 * x and w in the model's storage type (bf16 bit patterns or fp32), y fp32. Uses the
 * same kernel selection as the forward pass. Allocates temporaries. */
int s2d2_debug_gemm(s2d2_ctx* ctx, const void* x, const void* w, int32_t M, int32_t N, int32_t K, float* y);
/* The same with the token operand as two bf16 terms, x = x_hi + x_lo (x_lo may be NULL), an output scale and, with
 * accumulate != 0, y_inout[M,N] += scale * x w^T (y_inout is read, then overwritten with the result). bf16 models only. */
int s2d2_debug_gemm2(s2d2_ctx* ctx, const void* x_hi, const void* x_lo, const void* w, int32_t M, int32_t N, int32_t K,
                     float scale, int32_t accumulate, float* y_inout);
/* The gate/up GEMM of a wide pass with SwiGLU in its epilogue (test tap): w is [2f, K] = gate rows then up rows,
 * act = silu(x w_gate^T) * (x w_up^T) with x = x_hi + x_lo, returned as two bf16 terms (bit patterns, [M, f] each).
 * S2D2_ERR_UNSUPPORTED for shapes the forward pass would not give to this kernel (M <= 64, f % 128, K % 64). */
int s2d2_debug_gemm_swiglu(s2d2_ctx* ctx, const void* x_hi, const void* x_lo, const void* w, int32_t M, int32_t f, int32_t K,
                           uint16_t* act_hi, uint16_t* act_lo);

/* Expert ids chosen in the last pass, [n_layers, n_rows, top_k] (MoE models). */
int s2d2_debug_copy_expert_ids(s2d2_ctx* ctx, int32_t* out, int64_t cap, int32_t* n_rows_out);

/* Phase timeline of the last pass that ran as the persistent kernel: for every CTA a row of n_marks + 1
 * values, GPU global-timer readings (ns) at named points of the pass followed by the id of the SM the CTA
 * ran on.  Slots 0, 1: entry to and exit from the grid barrier behind the embedding (slot 2 unused).  Then
 * per layer, for dense models 12 slots: QKV accumulators drained; entry, exit of the barrier behind q/k-norm +
 * RoPE + K/V write; entry, exit of the barrier behind the attention items (a pass of one sequence has no barrier
 * there: items done, first combine pair's items counted complete); key splits combined; O accumulators
 * drained; residual add done; gate/up accumulators drained; SwiGLU done; down accumulators drained; residual
 * add done (from the combine on, the GEMMs of a dense layer follow each other without a grid barrier).  For
 * mixture-of-experts models 27 slots: (entry, exit, last accumulator drained before it or 0) for each of the
 * layer's nine grid barriers.  Then two slots: LM-head accumulators drained, logits written.  Then, for every
 * sub-GEMM of the pass in execution order (a GEMM may run as up to four), two slots: the CTA's first unit of it
 * ready to be multiplied, its last unit issued (0, 0 if the CTA has no unit of it); then, again per sub-GEMM,
 * four slots of the two producers: first weight tile requested, token-row producer arrived at the sub-GEMM,
 * its input counted complete, first token-row slice about to be requested.  Marks are
 * recorded only while s2d2_set_profiling is at level 2.  S2D2_ERR_STATE if no such pass has run. */
int s2d2_debug_pass_trace(s2d2_ctx* ctx, uint64_t* out, int64_t cap, int32_t* n_ctas, int32_t* n_marks);

/* Failure-path tap: runs the kernels' bounded-wait pattern on a word that nothing sets.  With
 * target > 0 the wait runs out after limit_polls polls (<= 2^20, about 0.1 us each), the kernel raises
 * the status word and returns normally, and the call returns S2D2_ERR_TIMEOUT; the context stays
 * usable.  With target == 0 the wait is satisfied at once and the call returns S2D2_OK. */
int s2d2_debug_wait_timeout(s2d2_ctx* ctx, uint32_t target, uint32_t limit_polls);

/* y[M, N] = x[M, K] w[N, K]^T on device buffers, without any allocation.
 * (The paper has no counterpart: this is a service entry for hosts that must not
 * allocate.)  Some callers cannot call cudaMalloc: a serving process whose framework
 * has already reserved the whole GPU for its own arena, so that any further driver
 * allocation fails or fragments it, and latency-critical loops, because cudaMalloc
 * and cudaFree synchronise the device and stall every stream.  This variant of the
 * tensor-core split-K GEMM keeps its scratch (partial tiles, ticket counters, status
 * word) in a fixed region that is part of the library image: S2D2_NOALLOC_WS_BYTES +
 * 16 KiB of device memory, held by every GPU that loads the library until exit.
 *   d_x  bf16 [M, K], d_w  bf16 [N, K], d_y  fp32 [M, N]: device pointers, row-major,
 *   16-byte aligned, owned by the caller.  1 <= M <= 256, 1 <= N <= 1048576,
 *   K a multiple of 64 with 64 <= K <= 65536; anything else returns S2D2_ERR_INVALID
 *   (text from s2d2_noalloc_last_error()).  The K split is lowered until the partial
 *   tiles fit the fixed scratch, so every shape inside these limits runs.
 * The call is synchronous on `cuda_stream` (it reads back the status word) and calls
 * no cudaMalloc, cudaFree or allocating library routine.  The first call on a device
 * looks up the address of the scratch region and raises the kernel's shared-memory
 * limit (host threads that arrive there together take their turn); make that first
 * call before any stream capture begins.  All calls on a
 * device share the one scratch region, which keeps the previous call's contents (the
 * counters are cleared at the start of every call): two calls that overlap on the
 * GPU, from different streams or threads, race and give wrong results. */
#define S2D2_NOALLOC_WS_BYTES (8u << 20)
int s2d2_gemm_bf16_noalloc(const void* d_x, const void* d_w, float* d_y, int32_t M, int32_t N, int32_t K,
                           void* cuda_stream);
const char* s2d2_noalloc_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* S2D2_H */
