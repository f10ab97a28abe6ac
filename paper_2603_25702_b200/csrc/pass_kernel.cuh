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
//             stages as soon as the phase that writes them has counted their columns complete.
//   warp 2    issues tcgen05.mma (weight tile = M operand, token rows = N operand, fp32
//             accumulators double-buffered in tensor memory).
//   warps 4-7 everything else: drain accumulators to split-K partials, then between grid barriers
//             the element-wise phases (partial sums + RMSNorm scale, q/k norm + RoPE + K/V write,
//             residual adds, SwiGLU, logits), the two-mask attention items and their combine.
//
// Work split of a GEMM (stream-K): its (weight tile, k-block) units, tile-major, are cut into
// gridDim equal contiguous ranges; a CTA's range yields one partial accumulator per tile it
// touches.  The element-wise phase behind the GEMM sums the partials of a tile in a fixed order, so
// results do not depend on timing.  A GEMM of a dense layer is cut into up to four sub-GEMMs (SubDesc)
// so that consecutive GEMMs overlap: the first output tiles are complete, reduced and turned into
// the next GEMM's input while the rest still streams, and the next GEMM begins with exactly those
// k-blocks.  Between the attention block of one layer and the next, no grid barrier is left on
// that path; every hand-over is a counted input tile or a counted partial.  RMSNorm is folded around the GEMM: the GEMM input is bf16(h * gain) and
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
constexpr int ACC_COLS = 256;        // tensor-memory columns of the GEMM accumulators: a ring of 2..8 buffers of 2 T columns
                                     // (high and low halves), rounded up to a power of two
constexpr int MAX_ACC = 8;
constexpr int TMEM_COLS = 512;       // the accumulator ring, then 64 columns of attention scores and 128 of attention output
constexpr int MAX_T = 64;            // most token rows of a pass
constexpr int W_TILE_BYTES = tc::BLOCK_N * 128;
constexpr uint32_t SPIN_LIMIT = 1u << 24;
constexpr int MAX_PARTS = 30;        // most split-K partials of one weight tile (the list of a tile is held one entry per lane)
constexpr int MAX_SUBS = 4;          // most sub-GEMMs of one GEMM
// GEMM kinds of a pass.  Dense layers run QKV, O, GU, DOWN; mixture-of-experts layers run QKV, O,
// ROUTER, SGU (shared expert gate/up), EGU (gate/up of the touched routed experts), SDOWN, EDOWN.
enum : int { K_QKV = 0, K_O = 1, K_GU = 2, K_DOWN = 3, K_LM = 4, K_ROUTER = 5, K_SGU = 6, K_EGU = 7, K_SDOWN = 8, K_EDOWN = 9, N_KINDS = 10 };
constexpr int MAX_EXPERTS = 256;

// A GEMM runs as one to four sub-GEMMs, each a set of weight tiles times a range of k-blocks with its
// own stream-K split over the CTAs.  The order of the sub-GEMMs is what lets consecutive GEMMs overlap:
// a GEMM whose output feeds the next one finishes a first group of tiles early (the element-wise work
// on them then runs while the remaining tiles stream), and the next GEMM starts with the k-blocks that
// this first group produces.
struct SubDesc {
    int t0, nt;          // first weight tile and number of tiles
    int t_split, t_jump; // local tile i is global tile t0 + i for i < t_split, else t0 + t_jump + (i - t_split)
                         // (the gate and the up rows that make the same columns of the SwiGLU output)
    int kb0, nkb;        // k-block range
    int seg_base;        // first workspace segment (per CTA) of this sub-GEMM
    int ew_t0, ew_t1;    // output tiles that are complete once this sub-GEMM is drained everywhere: the
                         // element-wise phase over them follows its drain (for gate/up: tiles of the SwiGLU output)
};

struct LayerGains {
    const float *attn_norm, *ffn_norm, *q_norm, *k_norm;
};

struct PassParams {
    int n_layers, d, Hq, Hkv, hd, f, V;
    int moe, n_experts, top_k, fe, fs;   // mixture of experts: routed experts of width fe, shared width fs (f = fs)
    int maps_per_layer;                  // weight tensor maps per layer (4 dense, 8 mixture of experts)
    int qk_norm;
    float eps, logit_scale;
    PassView pv;
    int M, T, n_logit;
    const bf16* embed;
    const LayerGains* gains;
    const float* final_norm;
    float* h;                 // [M, d] residual stream
    bf16 *xn, *q, *k_rows, *v_rows, *attn, *act;
    bf16 *xn_lo, *attn_lo, *act_lo;   // low halves of the GEMM inputs: x = hi + lo, both bf16
    bf16 *xn_b, *xn_b_lo;             // input of the GEMMs behind the attention block (gate/up, router): a buffer of its
                                      // own, so that writing it never meets a late reader of the QKV input and vice versa
    bf16* q_lo;                       // low halves of q, same split, for the attention items
    int map_lo_off;                   // tensor map of a buffer's low half = that of its high half + this
    float* ws;                // split-K partials, one region per GEMM kind: [grid][max_segs][T][128]
    long long ws_off[N_KINDS];   // region offsets in floats
    int max_segs[N_KINDS];
    bf16 *act_e, *act_e_lo;   // SwiGLU outputs of the touched experts [expert slot][T][fe], hi and lo halves
    int map_act_e;
    int* moe_ids;             // [M, top_k] chosen experts of the current layer
    float* moe_gates;         // [M, top_k] renormalised gates
    int* moe_ids_trace;       // [n_layers][trace_stride] copy of the ids of every layer (test tap)
    int trace_stride;
    int* n_touched_out;       // [n_layers] touched experts per layer (for byte accounting)
    float *ssq_a, *ssq_b;     // per-tile sums of squares of h rows [d/128][MAX_T]
    float* logits;            // [n_logit, V]
    const float *rope_cos, *rope_sin;
    KvPool<bf16> pool;
    const CUtensorMap* maps;  // device array: weights [n_layers*4 + 1], then the entries below
    int map_xn, map_xn_b, map_attn, map_act, map_kv;
    int map_q;                  // first of the two 3D maps of q (high, low halves) for the attention items, or -1
    att::AttnParams ap;       // attention geometry of this pass (layer filled in per layer)
    unsigned* barrier;        // grid barrier counter, zero at launch
    unsigned* tile_cnt[N_KINDS];    // per GEMM kind and weight tile: partials published so far (zero at launch)
    unsigned* x_cnt[4];       // per 128-column tile of xn / attn / act / xn_b: (tile, row) pairs written so far (zero at launch)
    unsigned* attn_cnt;       // per (sequence, kv head, query tile): attention items finished so far (zero at launch)
    SubDesc subs[N_KINDS][MAX_SUBS];
    int n_subs[N_KINDS];
    int acc_stride, n_acc;    // tensor-memory columns per accumulator buffer and buffers in the ring
    int* status;
    int S;                    // ring stages
    const int* parts[N_KINDS];      // per GEMM kind: [n_tiles][1 + MAX_PARTS] = count, then workspace slots in CTA order
    unsigned long long* trace;   // [grid][trace_cap] per grid barrier: globaltimer at entry, at exit, and when the
                                 // CTA's last accumulator of the phase had been drained (0 if the phase has no GEMM)
    int trace_cap;
    int trace_mma0;              // first of the per-sub-GEMM slot pairs written by the MMA issuer
    int trace_n_sub;             // sub-GEMMs of a pass with logits; behind the MMA issuer's pairs come four producer marks per sub-GEMM
    // Dense models: host-made schedule.  segs[cta * seg_stride + i] = i-th segment of the CTA: x = kind | sub << 8 |
    // workspace slot << 16, y = row coordinate of the weight tile, z = first k-block | k-blocks << 16, w = weight tile;
    // a layer's segments first (the same list for every layer), then the LM head's.  seg_sub_begin[cta * (n_layer_subs +
    // n_lm_subs + 1) + j] = first segment of sub-GEMM j in that order; the last entry is the total.  Null: the unit
    // ranges are computed in the kernel (mixture-of-experts models, whose routed-expert GEMMs are sized at run time).
    const int4* segs;
    const int* seg_sub_begin;
    int seg_stride, n_layer_subs, n_lm_subs;
};

__host__ __device__ inline size_t stage_bytes(int T) { return (size_t)W_TILE_BYTES + (size_t)2 * T * 128; }
__host__ __device__ inline size_t misc_bytes() { return 4096; }
__host__ __device__ inline size_t smem_bytes(int T, int S, int hd) {
    return 1024 + (size_t)S * stage_bytes(T) + att::attn_tiles_bytes(hd) + misc_bytes();
}

struct GemmShape {
    int n_tiles, kbt, map_w, map_x;      // tiles and k-blocks of this sub-GEMM (local numbering)
    int tpe;           // weight tiles per expert for the two routed-expert GEMMs, else 0
    int Geff;          // CTAs that share the sub-GEMM's units: all of them, or fewer for a small one so that
                       // no CTA gets less than an eighth of a tile's k-blocks and a tile has few parts
    int t0, t_split, t_jump, kb0, seg_base;     // placement inside the whole GEMM (SubDesc)
    long long U;
    __device__ __forceinline__ int tile_global(int i) const { return i < t_split ? t0 + i : t0 + t_jump + (i - t_split); }
};
__host__ __device__ inline int effective_ctas(long long U, int kbt, int G) {
    const long long min_units = kbt / 8 > 1 ? kbt / 8 : 1;
    const long long n = U / min_units;
    return (int)(n < 1 ? 1 : (n < G ? n : G));
}
// Shape of sub-GEMM `sub` of one GEMM of layer l; n_touched: touched routed experts of that layer (K_EGU, K_EDOWN).
__device__ __forceinline__ GemmShape gemm_shape(const PassParams& p, int l, int kind, int sub, int n_touched) {
    int mx, mw;
    GemmShape g;
    g.tpe = 0;
    switch (kind) {
        case K_QKV: mx = p.map_xn; mw = 0; break;
        case K_O: mx = p.map_attn; mw = 1; break;
        case K_GU: mx = p.map_xn_b; mw = 2; break;
        case K_DOWN: mx = p.map_act; mw = 3; break;
        case K_ROUTER: mx = p.map_xn_b; mw = 2; break;
        case K_SGU: mx = p.map_xn_b; mw = 3; break;
        case K_EGU: g.tpe = 2 * p.fe / tc::BLOCK_N; mx = p.map_xn_b; mw = 4; break;   // gate map 4, up map 5
        case K_SDOWN: mx = p.map_act; mw = 6; break;
        case K_EDOWN: g.tpe = p.d / tc::BLOCK_N; mx = p.map_act_e; mw = 7; break;
        default: mx = p.map_xn; mw = 0; break;
    }
    const SubDesc& sd = p.subs[kind][sub];
    g.n_tiles = sd.nt;
    g.kbt = sd.nkb;
    g.t0 = sd.t0;
    g.t_split = sd.t_split;
    g.t_jump = sd.t_jump;
    g.kb0 = sd.kb0;
    g.seg_base = sd.seg_base;
    if (kind == K_EGU || kind == K_EDOWN) {      // tile count known at run time only; one sub-GEMM
        g.n_tiles = n_touched * g.tpe;
        g.t_split = g.n_tiles;
    }
    g.map_w = kind == K_LM ? p.n_layers * p.maps_per_layer : l * p.maps_per_layer + mw;
    g.map_x = mx;
    g.U = (long long)g.n_tiles * g.kbt;
    g.Geff = effective_ctas(g.U, g.kbt, (int)gridDim.x);
    return g;
}
// GEMM kinds of a layer in the order they run.
__device__ __forceinline__ int layer_kind(const PassParams& p, int j) { return !p.moe ? j : (j < 2 ? j : K_ROUTER + (j - 2)); }
// Sub-GEMMs of one layer.
__device__ __forceinline__ int subs_per_layer(const PassParams& p) {
    int n = 0;
    for (int j = 0; j < (p.moe ? 7 : 4); ++j) n += p.n_subs[layer_kind(p, j)];
    return n;
}
// The gi-th sub-GEMM of the pass: its layer, kind and index inside the GEMM.
__device__ __forceinline__ void gemm_at(const PassParams& p, int gi, int spl, int& l, int& kind, int& sub) {
    if (gi >= p.n_layers * spl) {
        l = p.n_layers;
        kind = K_LM;
        sub = gi - p.n_layers * spl;
        return;
    }
    l = gi / spl;
    int r = gi - l * spl;
    for (int j = 0;; ++j) {
        kind = layer_kind(p, j);
        if (r < p.n_subs[kind]) break;
        r -= p.n_subs[kind];
    }
    sub = r;
}
// What the routed-expert GEMMs of the current layer need to know; lives in shared memory, written by
// the compute warps after the layer's routing, read by every role (layer_ready says for which layer).
struct Routing {
    volatile int layer_ready;      // 1 + the layer whose list is valid
    volatile int n_touched;
    int mask[MAX_EXPERTS / 32];
    short list[MAX_EXPERTS];       // touched expert ids, ascending
    short slot_of[MAX_EXPERTS];    // expert id -> position in list
};
__device__ __forceinline__ bool wait_routing(const PassParams& p, const Routing* r, int l, volatile int* abort_flag) {
    for (uint32_t it = 0; it < SPIN_LIMIT; ++it) {
        if (r->layer_ready > l) return true;
        if ((it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) return false;
        __nanosleep(50);
    }
    return false;
}
// Tensor map and row coordinate of (local) weight tile `tile` of a sub-GEMM.
__device__ __forceinline__ void weight_tile_coord(const PassParams& p, const GemmShape& g, int kind, int tile, const Routing* r,
                                                  int& map_w, int& y) {
    map_w = g.map_w;
    if (kind == K_EGU) {
        const int e = r->list[tile / g.tpe], t = tile % g.tpe, half = g.tpe / 2;
        map_w += t >= half;                                   // gate rows, then up rows
        y = e * p.fe + (t % half) * tc::BLOCK_N;
    } else if (kind == K_EDOWN) {
        y = r->list[tile / g.tpe] * p.d + (tile % g.tpe) * tc::BLOCK_N;
    } else {
        y = g.tile_global(tile) * tc::BLOCK_N;
    }
}
// First unit of CTA c: the units are cut into Geff equal contiguous ranges, CTAs past Geff get none.
__device__ __forceinline__ long long unit_begin(const GemmShape& g, int c) { return c >= g.Geff ? g.U : g.U * c / g.Geff; }

// Calls f(tile, kb0, kb1, local_segment) for the segments of this CTA's unit range (local tile and k-block numbers).
template <class F>
__device__ __forceinline__ void for_each_segment(const GemmShape& g, int cta, int G, F f) {
    long long u = unit_begin(g, cta), u1 = unit_begin(g, cta + 1);
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
__device__ __forceinline__ unsigned ld_relaxed(const unsigned* p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
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

// Walks the weight tiles (unit by unit) that one CTA streams during a pass, in order.  The
// per-unit step is two compares; divisions happen once per GEMM.  Before a layer's routed-expert
// GEMMs the cursor waits for that layer's routing.
struct UnitCursor {
    int gi, n_gemms, cta, G, spl;
    int left, kb, tile, kind;
    GemmShape g;
    const Routing* routing;
    volatile int* abort_flag;
    bool failed, opened;
    __device__ __forceinline__ void init(const PassParams&, int n_gemms_, int spl_, int cta_, int G_, const Routing* r, volatile int* abort) {
        gi = 0;
        spl = spl_;
        n_gemms = n_gemms_;
        cta = cta_;
        G = G_;
        routing = r;
        abort_flag = abort;
        failed = false;
        opened = false;
    }
    // Next unit: weight map index, k-block and row coordinate; false when the pass is through (or a
    // wait gave up: `failed`).  A GEMM is opened only when its first unit is asked for, so the wait for a
    // layer's routing never holds back a unit of an earlier GEMM.
    __device__ __forceinline__ bool next(const PassParams& p, int& map_w_, int& kb_, int& y_) {
        while (!opened) {
            if (gi >= n_gemms) return false;
            int l, sub;
            gemm_at(p, gi, spl, l, kind, sub);
            int n_touched = 0;
            if (kind == K_EGU || kind == K_EDOWN) {
                if (!wait_routing(p, routing, l, abort_flag)) {
                    failed = true;
                    return false;
                }
                n_touched = routing->n_touched;
            }
            g = gemm_shape(p, l, kind, sub, n_touched);
            const long long u = unit_begin(g, cta), u1 = unit_begin(g, cta + 1);
            if (u < u1) {
                left = (int)(u1 - u);
                tile = (int)(u / g.kbt);
                kb = (int)(u - (long long)tile * g.kbt);
                opened = true;
            } else {
                ++gi;
            }
        }
        weight_tile_coord(p, g, kind, tile, routing, map_w_, y_);
        kb_ = g.kb0 + kb;
        if (--left == 0) {
            ++gi;
            opened = false;
        } else if (++kb == g.kbt) {
            kb = 0;
            ++tile;
        }
        return true;
    }
};
// Sum over the split-K partials (in CTA order) of 4 consecutive columns of (tile, row): every
// lane of a warp takes columns 4*lane .. 4*lane+3.  tile_row_tab fetches the tile's slot list
// (count, then slots; one entry per lane) ahead of time.
__device__ __forceinline__ int tile_row_tab(const PassParams& p, int kind, int tile, int lane) {
    return lane <= MAX_PARTS ? __ldg(p.parts[kind] + (size_t)tile * (1 + MAX_PARTS) + lane) : 0;
}
// The same list for a GEMM whose tile count is only known at run time (routed experts): the
// contiguous unit ranges of the CTAs that touch the tile, by the arithmetic of for_each_segment
// (CTAs whose range is empty are skipped).  Returns -1 in lane 0 when the tile has more parts than
// the list holds.
__device__ __forceinline__ int dyn_tab(const GemmShape& g, int tile, int G, int max_segs, int lane) {
    const long long ua = (long long)tile * g.kbt, ub = ua + g.kbt - 1;
    int c_lo = (int)(ua * g.Geff / g.U);
    while (unit_begin(g, c_lo + 1) <= ua) ++c_lo;
    int c_hi = (int)(ub * g.Geff / g.U);
    while (unit_begin(g, c_hi + 1) <= ub) ++c_hi;
    const int c = c_lo + lane;                       // lane i looks at the i-th CTA from c_lo
    long long b0 = 0;
    bool valid = c <= c_hi;
    if (valid) {
        b0 = unit_begin(g, c);
        valid = unit_begin(g, c + 1) > b0;
    }
    const unsigned have = __ballot_sync(0xffffffffu, valid);
    const int cnt = __popc(have);
    const int mine = c * max_segs + (tile - (int)(b0 / g.kbt));
    // entry j (lane j >= 1) is the slot of the (j-1)-th valid CTA
    const int src = lane >= 1 && lane <= cnt ? (int)__fns(have, 0, lane) : 0;
    const int got = __shfl_sync(0xffffffffu, mine, src & 31);
    if (lane == 0) return (cnt > MAX_PARTS || c_hi - c_lo > 31) ? -1 : cnt;
    return lane <= cnt ? got : 0;
}
// NS such sums at once (tab_lane[s] = 0 marks an unused one).  Before reading, the warp waits
// (bounded) until all `cnt * round` partials of each tile have been published by the CTAs that
// drained them (round = layer + 1: the counters only grow).  Then the loads of up to PC parts of
// every sum are issued together, and each sum is accumulated in part order.
// published[s] == nullptr: no wait (a grid barrier already ordered the partials).
// after(dep) runs once the counts have arrived and before the partials are requested: loads issued there whose
// addresses include `dep` (always 0) are ordered behind the polls in the same way, which is how a phase reads
// what the writers of the GEMM's input had stored before they counted (the sums of squares of the rows).
template <int NS, int PC, class After>
__device__ __forceinline__ bool tile_row_sums(const PassParams& p, const float* ws, const int (&tab_lane)[NS], const int (&row)[NS],
                                              const unsigned* const (&published)[NS], unsigned round, int lane,
                                              volatile int* abort_flag, float4 (&out)[NS], After&& after) {
    int cnt[NS], max_cnt = 0;
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        cnt[s] = __shfl_sync(0xffffffffu, tab_lane[s], 0);
        if (cnt[s] < 0) {      // a tile split into more parts than the lists hold
            atomicCAS(p.status, 0, 9);
            *abort_flag = 1;
            cnt[s] = 0;
        }
        max_cnt = max(max_cnt, cnt[s]);
        out[s] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // Relaxed polls of all counters at once (acquire loads would complete one after the other).
    // The partials are then read by L2 loads whose addresses depend on the polled values: such a
    // load is issued after the counts it depends on have arrived, and the writers made their
    // partials visible in L2 before they counted, so no fence is needed between the two.
    unsigned dep = 0;
    {
        bool ready = false;
        unsigned low = 0xffffffffu;
        for (uint32_t it = 0; it < SPIN_LIMIT && !ready; ++it) {
            unsigned seen[NS];
#pragma unroll
            for (int s = 0; s < NS; ++s) seen[s] = cnt[s] > 0 && published[s] ? ld_relaxed(published[s]) : 0xffffffffu;
            ready = true;
            low = 0xffffffffu;
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                if (cnt[s] > 0 && seen[s] < (unsigned)cnt[s] * round) ready = false;
                low = min(low, seen[s] + 0x7fffffffu);        // wraps for the "no counter" value; never 0 for a real count
            }
            if (!ready && (it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) break;
        }
        if (!ready) {
            atomicCAS(p.status, 0, 8);
            *abort_flag = 1;
            return false;
        }
        dep = low == 0u ? 1u : 0u;     // always 0, but only known once every poll has returned
    }
    after(dep);
    for (int j0 = 0; j0 < max_cnt; j0 += PC) {
        float4 v[NS][PC];
#pragma unroll
        for (int s = 0; s < NS; ++s)
#pragma unroll
            for (int j = 0; j < PC; ++j) {
                const int slot = __shfl_sync(0xffffffffu, tab_lane[s], (j0 + j + 1) & 31);
                v[s][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (j0 + j < cnt[s])
                    v[s][j] = __ldcg(reinterpret_cast<const float4*>(ws + ((size_t)slot * p.T + row[s]) * tc::BLOCK_N) + lane + dep);
            }
#pragma unroll
        for (int s = 0; s < NS; ++s)
#pragma unroll
            for (int j = 0; j < PC; ++j) {
                out[s].x += v[s][j].x;
                out[s].y += v[s][j].y;
                out[s].z += v[s][j].z;
                out[s].w += v[s][j].w;
            }
    }
    return true;
}
template <int NS, int PC>
__device__ __forceinline__ bool tile_row_sums(const PassParams& p, const float* ws, const int (&tab_lane)[NS], const int (&row)[NS],
                                              const unsigned* const (&published)[NS], unsigned round, int lane,
                                              volatile int* abort_flag, float4 (&out)[NS]) {
    return tile_row_sums<NS, PC>(p, ws, tab_lane, row, published, round, lane, abort_flag, out, [](unsigned) {});
}
// 1/rms of a row from the per-tile sums of squares of h, in two steps: the loads (lanes take
// the tiles; nothing consumes them here, so they stay in flight with whatever the caller loads
// next), and later the sum.  Up to 128 tiles (d <= 16384).
struct SsqLane {
    float v[4];
};
__device__ __forceinline__ SsqLane row_ssq_lane(const float* ssq, int d_tiles, int row, int lane, unsigned dep = 0u) {
    SsqLane r;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int t = lane + 32 * k;
        r.v[k] = t < d_tiles ? __ldcg(ssq + (size_t)t * MAX_T + row + dep) : 0.f;
    }
    return r;
}
__device__ __forceinline__ float inv_rms_from(const SsqLane& r, int d, float eps) {
    return 1.0f / sqrtf(warp_sum((r.v[0] + r.v[1]) + (r.v[2] + r.v[3])) / (float)d + eps);
}
__device__ __forceinline__ void store_bf16x4(bf16* dst, float a, float b, float c, float d);
// x = q * d + r for 0 <= x < 2^22 and a run-time d: one multiplication by the precomputed 1/d
// instead of an integer division (about 40 dependent instructions, which a warp that has its
// scheduler to itself pays in full).
struct FastDiv {
    int d;
    float inv;
    __device__ __forceinline__ explicit FastDiv(int d_) : d(d_), inv(1.0f / (float)d_) {}
    __device__ __forceinline__ void divmod(int x, int& q, int& r) const {
        q = (int)(((float)x + 0.5f) * inv);
        r = x - q * d;
        if (r < 0) {
            --q;
            r += d;
        } else if (r >= d) {
            ++q;
            r -= d;
        }
    }
};
// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): the GEMMs take both halves as token rows, so
// their inputs carry 16 significant bits instead of 8 (the tensor pipe is nearly idle in this
// kernel; the second half costs 2 KB of shared memory per stage).
__device__ __forceinline__ void store_hi_lo_x4(bf16* hi, bf16* lo, float a, float b, float c, float d) {
    const float ha = __bfloat162float(__float2bfloat16_rn(a)), hb = __bfloat162float(__float2bfloat16_rn(b));
    const float hc = __bfloat162float(__float2bfloat16_rn(c)), hd = __bfloat162float(__float2bfloat16_rn(d));
    store_bf16x4(hi, ha, hb, hc, hd);
    store_bf16x4(lo, a - ha, b - hb, c - hc, d - hd);
}
__device__ __forceinline__ void store_bf16x4(bf16* dst, float a, float b, float c, float d) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst) = u;
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
    uint64_t* acc_empty = acc_full + MAX_ACC;
    uint64_t* kv_full = acc_empty + MAX_ACC;
    uint32_t* tmem_slot = (uint32_t*)(kv_full + att::STAGES + 3);     // + the "scores ready" and "output ready" barriers of the tcgen05 attention items
    volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
    volatile int* w_issued = abort_flag + 1;
    volatile int* x_issued = w_issued + 1;
    volatile int* consumed = x_issued + 1;
    Routing* routing = (Routing*)(misc + 1024);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int spl = subs_per_layer(p);
    const int n_gemms = p.n_layers * spl + (p.n_logit > 0 ? p.n_subs[K_LM] : 0);
    const int NACC = p.n_acc, ACC_STRIDE = p.acc_stride;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            tc::mbar_init(&full[s], 2);
            tc::mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < MAX_ACC; ++b) {
            tc::mbar_init(&acc_full[b], 1);
            tc::mbar_init(&acc_empty[b], 4);
        }
        for (int s = 0; s < att::STAGES + 3; ++s) tc::mbar_init(&kv_full[s], 1);
        *abort_flag = 0;
        *w_issued = 0;
        *x_issued = 0;
        *consumed = 0;
        routing->layer_ready = 0;
        routing->n_touched = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 2) {
        tc::tmem_alloc(tmem_slot, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Dense models: this CTA's segments (one weight tile times a k-block range each) come from a host-made table,
    // a layer's list (the same for every layer) and the LM head's; sb[j] is the first segment of sub-GEMM j.
    const bool tabled = p.segs != nullptr;
    const int4* my_segs = tabled ? p.segs + (size_t)cta * p.seg_stride : nullptr;
    const int* sb = tabled ? p.seg_sub_begin + (size_t)cta * (p.n_layer_subs + p.n_lm_subs + 1) : nullptr;
    // per-sub-GEMM trace slots (only while tracing): MMA issuer {first unit ready, last unit issued}; producers
    // {first weight tile requested, token-row producer arrived, input counted complete, first slice about to be requested}
    auto trace_slot = [&](int k) -> unsigned long long* {
        return p.trace && k >= 0 && k + 3 < p.trace_cap - 1 ? p.trace + (size_t)cta * p.trace_cap + k : nullptr;
    };
    auto stamp = [](unsigned long long* dst) {
        if (dst) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(*dst));
    };

    if (warp == 0) {
        if (lane == 0) {
            // ---------------- W producer: free-running over every GEMM of the pass ----------------
            uint64_t policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
            bool ok = true;
            if (tabled) {
                // One iteration per streamed unit is a wait for the stage, an expect and a copy: the stage index and
                // its parity advance by increments, the coordinates come from the segment's table entry.
                int s = 0;
                uint32_t par = 0, issued = 0;      // par: parity of the stage's use count; the first use of a stage waits for nothing
                bool first_round = true;
                uint8_t* dst = ring;
                auto run = [&](int seg_a, int seg_b, int map_base, int gi_base, int sub_a) {
                    int sub = sub_a;
                    int4 d = seg_a < seg_b ? __ldg(my_segs + seg_a) : make_int4(0, 0, 0, 0);
                    for (int si = seg_a; si < seg_b && ok; ++si) {
                        const int4 dn = si + 1 < seg_b ? __ldg(my_segs + si + 1) : d;      // next entry requested ahead of this segment's copies
                        const int kind = d.x & 255;
                        if (p.trace) {
                            while (sb[sub + 1] <= si) ++sub;
                            if (sb[sub] == si) stamp(trace_slot(p.trace_mma0 + 2 * p.trace_n_sub + 4 * (gi_base + sub - sub_a)));
                        }
                        const CUtensorMap* map = p.maps + map_base + (kind == K_LM ? 0 : kind);      // dense kinds 0..3 are the layer's map order
                        int x = (d.z & 0xffff) * tc::BLOCK_K;
                        const int y = d.y;
                        for (int n = d.z >> 16; n > 0; --n, x += tc::BLOCK_K) {
                            if (!first_round && !tc::mbar_wait(&empty[s], par ^ 1u, abort_flag)) {
                                ok = false;
                                break;
                            }
                            tc::mbar_expect_tx(&full[s], W_TILE_BYTES);
                            tc::tma_load_2d_hint(dst, map, x, y, &full[s], policy);
                            *w_issued = (int)++issued;
                            dst += sbytes;
                            if (++s == S) {
                                s = 0;
                                dst = ring;
                                par ^= 1u;
                                first_round = false;
                            }
                        }
                        d = dn;
                    }
                };
                for (int l = 0; l < p.n_layers && ok; ++l) run(0, sb[p.n_layer_subs], l * p.maps_per_layer, l * p.n_layer_subs, 0);
                if (ok && p.n_logit > 0)
                    run(sb[p.n_layer_subs], sb[p.n_layer_subs + p.n_lm_subs], p.n_layers * p.maps_per_layer, p.n_layers * p.n_layer_subs, p.n_layer_subs);
            } else {
                UnitCursor ld;
                ld.init(p, n_gemms, spl, cta, G, routing, abort_flag);
                uint32_t i = 0;
                int mw, kb, y;
                while (ld.next(p, mw, kb, y)) {
                    const int s = (int)(i % (uint32_t)S);
                    if (i >= (uint32_t)S && !tc::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) {
                        ok = false;
                        break;
                    }
                    if (*abort_flag) {
                        ok = false;
                        break;
                    }
                    tc::mbar_expect_tx(&full[s], W_TILE_BYTES);
                    tc::tma_load_2d_hint(ring + s * sbytes, p.maps + mw, kb * tc::BLOCK_K, y, &full[s], policy);
                    *w_issued = (int)i + 1;
                    ++i;
                }
                if (ld.failed) ok = false;
            }
            if (!ok) {
                atomicCAS(p.status, 0, 7);
                *abort_flag = 1;
            }
        }
    } else if (warp == 1) {
        // ---------------- X producer: token-row slices, as soon as their columns are written ----------------
        // The phases that write a GEMM's input count the finished (128-column tile, row) pairs per
        // tile; the lanes of this warp poll the tiles a segment needs in parallel, lane 0 issues the
        // copies.  The inputs are therefore fetched without waiting for the grid barrier, which only
        // guards buffer reuse.
        bool ok = true;
        if (tabled) {
            int s = 0;
            uint32_t par = 0, issued = 0;
            bool first_round = true;
            uint8_t* dst = ring + W_TILE_BYTES;
            auto run = [&](int seg_a, int seg_b, int l, int gi_base, int sub_a) {
                int sub = sub_a;
                int4 d = seg_a < seg_b ? __ldg(my_segs + seg_a) : make_int4(0, 0, 0, 0);
                for (int si = seg_a; si < seg_b && ok; ++si) {
                    const int4 dn = si + 1 < seg_b ? __ldg(my_segs + si + 1) : d;
                    const int kind = d.x & 255;
                    unsigned long long* tx = nullptr;
                    if (p.trace) {
                        while (sb[sub + 1] <= si) ++sub;
                        if (sb[sub] == si && lane == 0) tx = trace_slot(p.trace_mma0 + 2 * p.trace_n_sub + 4 * (gi_base + sub - sub_a));
                    }
                    stamp(tx ? tx + 1 : nullptr);
                    // which counter set, and how many pairs make a tile complete for this GEMM
                    const unsigned* cnt;
                    unsigned target = (unsigned)p.M * (unsigned)(l + 1);
                    int mx;
                    switch (kind) {
                        case K_QKV: cnt = p.x_cnt[0]; mx = p.map_xn; break;
                        case K_O: cnt = p.x_cnt[1]; mx = p.map_attn; target *= (unsigned)(tc::BLOCK_N / HD); break;
                        case K_GU: cnt = p.x_cnt[3]; mx = p.map_xn_b; break;
                        case K_DOWN: cnt = p.x_cnt[2]; mx = p.map_act; break;
                        default: cnt = p.x_cnt[0]; mx = p.map_xn; break;      // LM head: l == n_layers
                    }
                    const int kb0 = d.z & 0xffff, kb1 = kb0 + (d.z >> 16);
                    // tiles of 128 columns = 2 k-blocks
                    for (int t0 = kb0 >> 1; t0 <= (kb1 - 1) >> 1; t0 += 32) {
                        const int t = t0 + lane;
                        bool ready = t > ((kb1 - 1) >> 1);
                        for (uint32_t it = 0; !ready && it < SPIN_LIMIT; ++it) {
                            ready = ld_acquire(cnt + t) >= target;
                            if (!ready && (it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) break;
                        }
                        if (!__all_sync(0xffffffffu, ready)) ok = false;
                    }
                    if (!ok) break;
                    stamp(tx ? tx + 2 : nullptr);
                    if (lane == 0) {
                        const CUtensorMap* m_hi = p.maps + mx;
                        const CUtensorMap* m_lo = m_hi + p.map_lo_off;
                        const uint32_t bytes = (uint32_t)T * 256u;
                        bool fine = true;
                        int x = kb0 * tc::BLOCK_K;
                        for (int n = kb1 - kb0; n > 0; --n, x += tc::BLOCK_K) {
                            if (!first_round && !tc::mbar_wait(&empty[s], par ^ 1u, abort_flag)) {
                                fine = false;
                                break;
                            }
                            if (tx) {
                                stamp(tx + 3);
                                tx = nullptr;
                            }
                            tc::mbar_expect_tx(&full[s], bytes);
                            tc::tma_load_2d(dst, m_hi, x, 0, &full[s]);
                            tc::tma_load_2d(dst + T * 128, m_lo, x, 0, &full[s]);
                            ++issued;
                            dst += sbytes;
                            if (++s == S) {
                                s = 0;
                                dst = ring + W_TILE_BYTES;
                                par ^= 1u;
                                first_round = false;
                            }
                        }
                        *x_issued = (int)issued;
                        if (!fine) ok = false;
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    d = dn;
                }
            };
            for (int l = 0; l < p.n_layers && ok; ++l) run(0, sb[p.n_layer_subs], l, l * p.n_layer_subs, 0);
            if (ok && p.n_logit > 0) run(sb[p.n_layer_subs], sb[p.n_layer_subs + p.n_lm_subs], p.n_layers, p.n_layers * p.n_layer_subs, p.n_layer_subs);
        } else {
            uint32_t i = 0;
            for (int gi = 0; gi < n_gemms && ok; ++gi) {
                int l, kind, sub;
                gemm_at(p, gi, spl, l, kind, sub);
                int n_touched = 0;
                if (kind == K_EGU || kind == K_EDOWN) {
                    if (!wait_routing(p, routing, l, abort_flag)) {
                        ok = false;
                        break;
                    }
                    n_touched = routing->n_touched;
                }
                const GemmShape g = gemm_shape(p, l, kind, sub, n_touched);
                const CUtensorMap* mx = p.maps + g.map_x;
                // which counter set, and how many pairs make a tile complete for this GEMM
                const unsigned* cnt = nullptr;
                unsigned target = 0;
                switch (kind) {
                    case K_QKV: cnt = p.x_cnt[0]; target = (unsigned)p.M * (l + 1u); break;
                    case K_O: cnt = p.x_cnt[1]; target = (unsigned)p.M * (unsigned)(tc::BLOCK_N / HD) * (l + 1u); break;
                    case K_GU: case K_ROUTER: case K_SGU: case K_EGU: cnt = p.x_cnt[3]; target = (unsigned)p.M * (l + 1u); break;
                    case K_DOWN: case K_SDOWN: cnt = p.x_cnt[2]; target = (unsigned)p.M * (l + 1u); break;
                    case K_EDOWN: break;     // its input is published by the grid barrier that follows the experts' SwiGLU
                    default: cnt = p.x_cnt[0]; target = (unsigned)p.M * (p.n_layers + 1u); break;
                }
                if (kind == K_EDOWN && unit_begin(g, cta + 1) > unit_begin(g, cta)) {
                    if (!wait_counter(p, (2u + 9u * l + 6u) * (unsigned)G, abort_flag)) {
                        ok = false;
                        break;
                    }
                }
                for_each_segment(g, cta, G, [&](int tile, int kb0, int kb1, int) {
                    const int x_row = kind == K_EDOWN ? (tile / g.tpe) * T : 0;     // the expert slot's rows of act_e
                    kb0 += g.kb0;                                                    // k-blocks of the whole GEMM from here on
                    kb1 += g.kb0;
                    // tiles of 128 columns = 2 k-blocks
                    for (int t0 = kb0 >> 1; cnt && t0 <= (kb1 - 1) >> 1; t0 += 32) {
                        const int t = t0 + lane;
                        bool ready = t > ((kb1 - 1) >> 1);
                        for (uint32_t it = 0; !ready && it < SPIN_LIMIT; ++it) {
                            ready = ld_acquire(cnt + t) >= target;
                            if (!ready && (it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) break;
                        }
                        if (!__all_sync(0xffffffffu, ready)) return ok = false;
                    }
                    asm volatile("fence.proxy.async;" ::: "memory");
                    for (int kb = kb0; kb < kb1; ++kb, ++i) {
                        int s = (int)(i % (uint32_t)S);
                        bool fine = true;
                        if (lane == 0) {
                            if (i >= (uint32_t)S && !tc::mbar_wait(&empty[s], ((i / S) - 1) & 1, abort_flag)) fine = false;
                            if (*abort_flag) fine = false;
                            if (fine) {
                                tc::mbar_expect_tx(&full[s], (uint32_t)T * 256u);
                                tc::tma_load_2d(ring + s * sbytes + W_TILE_BYTES, mx, kb * tc::BLOCK_K, x_row, &full[s]);
                                tc::tma_load_2d(ring + s * sbytes + W_TILE_BYTES + T * 128, mx + (kind == K_EDOWN ? 4 : p.map_lo_off), kb * tc::BLOCK_K,
                                                x_row, &full[s]);
                                *x_issued = (int)i + 1;
                            }
                        }
                        if (!__all_sync(0xffffffffu, fine)) return ok = false;
                    }
                    return true;
                });
            }
        }
        if (!ok && lane == 0) {
            atomicCAS(p.status, 0, 3);
            *abort_flag = 1;
        }
    } else if (warp == 2) {
        if (lane == 0) {
            // ---------------- MMA issuer ----------------
            const uint32_t idesc = tc::instr_desc_bf16(2 * T);     // token rows twice: high halves, then low halves
            uint32_t seg = 0;
            bool ok = true;
            if (tabled) {
                int s = 0;
                uint32_t par = 0, done = 0;
                uint32_t b = 0, use_par = 0;       // accumulator buffer of the segment and the parity of its use count
                bool first_acc_round = true;
                const uint64_t desc0 = tc::smem_desc_sw128(tc::smem_u32(ring));
                const uint64_t desc_step = (uint64_t)(sbytes >> 4), desc_b = (uint64_t)(W_TILE_BYTES >> 4);      // descriptor addresses count 16-byte units
                uint64_t a_desc = desc0;
                auto run = [&](int seg_a, int seg_b, int gi_base, int sub_a) {
                    int sub = sub_a;
                    int4 d = seg_a < seg_b ? __ldg(my_segs + seg_a) : make_int4(0, 0, 0, 0);
                    for (int si = seg_a; si < seg_b && ok; ++si) {
                        const int4 dn = si + 1 < seg_b ? __ldg(my_segs + si + 1) : d;
                        unsigned long long* tm = nullptr;
                        bool last_of_sub = false;
                        if (p.trace) {
                            while (sb[sub + 1] <= si) ++sub;
                            tm = trace_slot(p.trace_mma0 + 2 * (gi_base + sub - sub_a));
                            last_of_sub = sb[sub + 1] == si + 1;
                            if (sb[sub] != si) tm = last_of_sub ? tm : nullptr;
                        }
                        const bool first_of_sub = p.trace && sb[sub] == si;
                        if (!first_acc_round && !tc::mbar_wait(&acc_empty[b], use_par ^ 1u, abort_flag)) {
                            ok = false;
                            break;
                        }
                        tc::tc_fence_after();
                        const uint32_t d_tmem = tmem_base + b * ACC_STRIDE;
                        uint32_t acc = 0;
                        for (int n = d.z >> 16; n > 0; --n) {
                            if (!tc::mbar_wait(&full[s], par, abort_flag)) {
                                ok = false;
                                break;
                            }
                            tc::tc_fence_after();
                            if (first_of_sub && acc == 0) stamp(tm);
                            const uint64_t b_desc = a_desc + desc_b;
#pragma unroll
                            for (int k = 0; k < tc::BLOCK_K / tc::UMMA_K; ++k) {
                                tc::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, acc);
                                acc = 1;
                            }
                            tc::umma_commit(&empty[s]);
                            *consumed = (int)++done;
                            a_desc += desc_step;
                            if (++s == S) {
                                s = 0;
                                a_desc = desc0;
                                par ^= 1u;
                            }
                        }
                        if (!ok) break;
                        tc::umma_commit(&acc_full[b]);
                        if (last_of_sub && tm) stamp(tm + 1);
                        if (++b == (uint32_t)NACC) {
                            b = 0;
                            use_par ^= 1u;
                            first_acc_round = false;
                        }
                        ++seg;
                        d = dn;
                    }
                };
                for (int l = 0; l < p.n_layers && ok; ++l) run(0, sb[p.n_layer_subs], l * p.n_layer_subs, 0);
                if (ok && p.n_logit > 0) run(sb[p.n_layer_subs], sb[p.n_layer_subs + p.n_lm_subs], p.n_layers * p.n_layer_subs, p.n_layer_subs);
            } else {
                uint32_t i = 0;
                for (int gi = 0; gi < n_gemms && ok; ++gi) {
                    int l, kind, sub;
                    gemm_at(p, gi, spl, l, kind, sub);
                    int n_touched = 0;
                    if (kind == K_EGU || kind == K_EDOWN) {
                        if (!wait_routing(p, routing, l, abort_flag)) {
                            ok = false;
                            break;
                        }
                        n_touched = routing->n_touched;
                    }
                    const GemmShape g = gemm_shape(p, l, kind, sub, n_touched);
                    for_each_segment(g, cta, G, [&](int, int kb0, int kb1, int) {
                        const uint32_t b = seg % (uint32_t)NACC, use = seg / (uint32_t)NACC;
                        if (use >= 1 && !tc::mbar_wait(&acc_empty[b], (use - 1) & 1, abort_flag)) return ok = false;
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
        uint32_t seg = 0, kv_ring = 0, attn_s_cnt = 0, attn_o_cnt = 0, attn_q_cnt = 0;
        bool ok = true;
        const int M = p.M, d = p.d;
        const int d_tiles = d / tc::BLOCK_N;

        // Grid barrier.  tma_out: this phase wrote data that other CTAs read through TMA (GEMM
        // inputs, K/V pages), which needs the generic-to-async proxy fence on the writer side.
        // One thread publishes for the CTA: its release covers the writes the CTA barrier ordered
        // before it.
        unsigned long long t_drained = 0;
        // Phase marks (only while tracing): the GPU timer at a named point of the pass, one slot each.
        auto mark = [&](int k) {
            if (p.trace && tid == 0 && k >= 0 && k < p.trace_cap - 1) {
                unsigned long long t;
                asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
                p.trace[(size_t)cta * p.trace_cap + k] = t;
            }
        };
        // k: trace slot of the barrier's entry mark (exit at k + 1; with_drained: k + 2 gets the time the
        // CTA's last accumulator before the barrier had been drained)
        auto grid_sync = [&](bool tma_out, int k, bool with_drained) {
            ++epoch;
            if (tma_out) asm volatile("fence.proxy.async;" ::: "memory");
            att::group_sync(BAR_COMPUTE, CTHREADS);
            if (tid == 0) {
                mark(k);
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.barrier) : "memory");
                if (!wait_counter(p, epoch * (unsigned)G, abort_flag)) {
                    atomicCAS(p.status, 0, 5);
                    *abort_flag = 1;
                }
                mark(k + 1);
                if (with_drained && p.trace && k + 2 < p.trace_cap - 1) {
                    p.trace[(size_t)cta * p.trace_cap + k + 2] = t_drained;
                    t_drained = 0;
                }
            }
            att::group_sync(BAR_COMPUTE, CTHREADS);
            if (*abort_flag) ok = false;
        };
        // accumulators of this CTA's segments of one sub-GEMM -> split-K partials
        uint32_t acc_b = 0, acc_par = 0;      // accumulator buffer of the next segment and the parity of its use count
        auto drain_segment = [&](int kind, int slot, int tile_global) {
            if (!tc::mbar_wait(&acc_full[acc_b], acc_par, abort_flag)) return ok = false;
            tc::tc_fence_after();
            float* mine = p.ws + p.ws_off[kind] + ((size_t)cta * p.max_segs[kind] + slot) * (size_t)T * tc::BLOCK_N + tid;
            const uint32_t taddr = tmem_base + ((uint32_t)(cw * 32) << 16) + acc_b * ACC_STRIDE;
            for (int c0 = 0; c0 < T; c0 += 16) {
                float v[16], w[16];
                tc::tmem_ld16(taddr + c0, v);          // W x_hi
                tc::tmem_ld16(taddr + T + c0, w);      // W x_lo
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (c0 + j < M) mine[(size_t)(c0 + j) * tc::BLOCK_N] = v[j] + w[j];
            }
            tc::tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[acc_b]);
            // publish: every thread's part of the partial is stored, then one release for the CTA
            att::group_sync(BAR_COMPUTE, CTHREADS);
            if (tid == 0 && p.tile_cnt[kind])
                asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.tile_cnt[kind] + tile_global) : "memory");
            if (++acc_b == (uint32_t)NACC) {
                acc_b = 0;
                acc_par ^= 1u;
            }
            ++seg;
            return true;
        };
        // first sub-GEMM of each dense kind in the table's order
        const int jb_o = p.n_subs[K_QKV], jb_gu = jb_o + p.n_subs[K_O], jb_down = jb_gu + p.n_subs[K_GU];
        auto drain_sub = [&](int l, int kind, int sub) {
            if (tabled) {
                const int j = (kind == K_QKV ? 0 : kind == K_O ? jb_o : kind == K_GU ? jb_gu : kind == K_DOWN ? jb_down : p.n_layer_subs) + sub;
                const int a = __ldg(sb + j), b = __ldg(sb + j + 1);
                for (int si = a; si < b && ok; ++si) {
                    const int4 d = __ldg(my_segs + si);
                    drain_segment(kind, d.x >> 16, d.w);
                }
            } else {
                const GemmShape g = gemm_shape(p, l, kind, sub, routing->n_touched);
                for_each_segment(g, cta, G, [&](int tile, int, int, int local) { return drain_segment(kind, g.seg_base + local, g.tile_global(tile)); });
            }
            if (!ok) {
                atomicCAS(p.status, 0, 6);
                *abort_flag = 1;
            }
            if (p.trace && tid == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_drained));
        };
        auto drain = [&](int l, int kind) {
            for (int sub = 0; sub < p.n_subs[kind] && ok; ++sub) drain_sub(l, kind, sub);
        };
        // The element-wise phases work warp by warp on (tile, row) pairs: 128 output columns of one
        // row, 4 per lane.  A pair's loads (its partials, its residual row, the sums of squares) are
        // all in flight together, so a phase costs about one round trip to L2.
        const int gw = cta * 4 + cw, GW = G * 4;
        const FastDiv by_M(M), by_Hq(p.Hq);

        // A (tile, row) pair of a GEMM input is written: count it.  Each writing thread first orders its
        // generic-proxy stores before later async-proxy (TMA) reads of global memory, then the release orders the
        // warp's stores before the count; the reader (the X producer) acquires the count and issues its TMA loads.
        // The proxy fence sits with the writers because a writer has no copies in flight when it runs it, whereas
        // the X producer always has: there the same fence waited for them, about two microseconds per segment.
        auto publish_x = [&](unsigned* counter) {
            asm volatile("fence.proxy.async.global;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
        };
        // h update shared by the embedding and the residual phases, over the tiles [t_a, t_b) of the row: writes h,
        // the next GEMM's input bf16(h * gain) (two terms) and the (tile, row) sum of squares.  The pair
        // (t, m) always belongs to warp (t * M + m) mod GW, whatever the tile range, so the same warp reads
        // and rewrites a given piece of h in every phase of the pass.
        auto h_phase = [&](const float* gain, float* ssq, bf16* x_hi, bf16* x_lo, unsigned* x_counter, int t_a, int t_b, auto&& value) {
            const int lo_pair = t_a * M;
            int r0 = (gw - lo_pair) % GW;
            if (r0 < 0) r0 += GW;
            for (int pair = lo_pair + r0; pair < t_b * M; pair += GW) {
                int t, m;
                by_M.divmod(pair, t, m);
                const int col = t * tc::BLOCK_N + 4 * lane;
                const float4 gn = *reinterpret_cast<const float4*>(gain + col);
                const float4 x = value(t, m, col);
                *reinterpret_cast<float4*>(p.h + (size_t)m * d + col) = x;
                store_hi_lo_x4(x_hi + (size_t)m * d + col, x_lo + (size_t)m * d + col, x.x * gn.x, x.y * gn.y, x.z * gn.z, x.w * gn.w);
                const float sq = warp_sum(x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w);
                if (lane == 0) ssq[(size_t)t * MAX_T + m] = sq;
                publish_x(x_counter + t);
            }
        };
        // h += GEMM output over the output tiles [t_a, t_b); to_b: the result feeds the GEMMs behind the attention block
        auto residual_phase = [&](int kind, unsigned round, const float* gain, float* ssq, bool to_b, int t_a, int t_b) {
            h_phase(gain, ssq, to_b ? p.xn_b : p.xn, to_b ? p.xn_b_lo : p.xn_lo, p.x_cnt[to_b ? 3 : 0], t_a, t_b, [&](int t, int m, int col) {
                const int tab = tile_row_tab(p, kind, t, lane);
                const float4 hv = __ldcg(reinterpret_cast<const float4*>(p.h + (size_t)m * d + col));
                const int tabs[1] = {tab}, rows[1] = {m};
                const unsigned* const pubs[1] = {p.tile_cnt[kind] + t};
                float4 sums[1];
                tile_row_sums<1, 16>(p, p.ws + p.ws_off[kind], tabs, rows, pubs, round, lane, abort_flag, sums);
                float4 x = sums[0];
                x.x += hv.x;
                x.y += hv.y;
                x.z += hv.z;
                x.w += hv.w;
                return x;
            });
        };

        if (tid == 0 && p.trace) {
            unsigned smid;
            asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
            p.trace[(size_t)cta * p.trace_cap + p.trace_cap - 1] = smid;
        }
        // ---- embedding ----
        h_phase(p.gains[0].attn_norm, p.ssq_a, p.xn, p.xn_lo, p.x_cnt[0], 0, d_tiles, [&](int, int m, int col) {
            const uint2 u = *reinterpret_cast<const uint2*>(p.embed + (size_t)p.pv.row_token[m] * d + col);
            const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&u.x), hi = *reinterpret_cast<const __nv_bfloat162*>(&u.y);
            return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
        });
        grid_sync(true, 0, true);
        // trace slots: 3 for the embedding barrier; then per dense layer 12 named marks, per mixture-of-experts
        // layer 9 barrier triples; then two marks of the LM-head phase
        const int marks_per_layer = p.moe ? 27 : 12;

        for (int l = 0; l < p.n_layers && ok; ++l) {
            const LayerGains lg = p.gains[l];
            const int tb = 3 + marks_per_layer * l;        // this layer's first trace slot
            // First attention item of this CTA in this layer: its first K/V page is in the cache already, so the
            // copies are started now and land behind the QKV GEMM (tcgen05 items only).
            bool attn_first_requested = false;
            int attn_first = -1;
            if constexpr (HD == 128) {
                if (p.ap.page_tokens == 64) {
                    att::AttnParams ap0 = p.ap;
                    ap0.layer = l;
                    const int n_splits0 = ap0.n_cache_splits + 1;
                    const int total0 = ap0.pv.n_seqs * ap0.Hkv * ap0.n_qtiles * n_splits0;
                    if (ap0.sched_off) {
                        const int i0 = __ldg(ap0.sched_off + cta);
                        if (i0 < __ldg(ap0.sched_off + cta + 1)) attn_first = __ldg(ap0.sched_items + i0);
                    } else if (cta < total0) {
                        attn_first = cta;
                    }
                    if (attn_first >= 0) {
                        const int r0 = attn_first / n_splits0;
                        attn_first_requested = att::attn_umma_request_first(p.maps + p.map_kv, ap0, attn_first % n_splits0, r0 % ap0.n_qtiles,
                                                                            r0 / ap0.n_qtiles, attn_s, kv_full, kv_ring, tid);
                    }
                }
            }
            // ---- QKV GEMM ----
            drain(l, K_QKV);
            if (!ok) break;
            if (!p.moe) mark(tb);
            // ---- 1/rms, q/k norm, RoPE, K/V write: one warp per (128-column tile, row) ----
            {
                constexpr int half = HD / 2, PART = half / 4;     // PART: lane distance of a RoPE pair
                const int n_tiles = (p.Hq + 2 * p.Hkv) * HD / tc::BLOCK_N;
                const int c_tile = 4 * lane;                        // column inside the tile
                const int n_pairs = n_tiles * M;
                // two pairs per step; everything a step reads is requested before anything is used
                for (int pair0 = gw; pair0 < n_pairs; pair0 += 2 * GW) {
                    int tt[2], mm[2], tabs[2], pos[2], flags[2], page[2];
                    SsqLane sq_l[2];
                    float4 cs[2], sn[2], gq[2];
                    bool on[2];
                    const unsigned* pubs[2];
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const int pr = pair0 + q * GW;
                        on[q] = pr < n_pairs;
                        by_M.divmod(on[q] ? pr : 0, tt[q], mm[q]);
                        const int head = (tt[q] * tc::BLOCK_N + c_tile) / HD, ch = c_tile % HD;
                        const bool is_q = head < p.Hq, is_k = !is_q && head < p.Hq + p.Hkv;
                        tabs[q] = on[q] ? tile_row_tab(p, 0, tt[q], lane) : 0;
                        pubs[q] = p.tile_cnt[0] + tt[q];
                        pos[q] = __ldg(p.pv.row_pos + mm[q]);
                        flags[q] = __ldg(p.pv.row_flags + mm[q]);
                        const int sq = __ldg(p.pv.row_seq + mm[q]);
                        const int i0 = ch - (ch >= half ? half : 0);
                        cs[q] = __ldg(reinterpret_cast<const float4*>(p.rope_cos + (size_t)pos[q] * half + i0));
                        sn[q] = __ldg(reinterpret_cast<const float4*>(p.rope_sin + (size_t)pos[q] * half + i0));
                        page[q] = (flags[q] & ROW_WRITE_KV) ? __ldg(p.pv.seq_pages + (size_t)sq * p.pv.max_pages + (pos[q] >> p.pool.page_shift)) : 0;
                        gq[q] = make_float4(1.f, 1.f, 1.f, 1.f);
                        if (p.qk_norm && (is_q || is_k)) gq[q] = __ldg(reinterpret_cast<const float4*>((is_q ? lg.q_norm : lg.k_norm) + ch));
                    }
                    // The sums of squares of the rows were stored by the writers of this GEMM's input before they
                    // counted it; no grid barrier lies in between, so they are read behind the polls of the partials.
                    float4 sums[2];
                    const unsigned* const pubs_c[2] = {pubs[0], pubs[1]};
                    tile_row_sums<2, 8>(p, p.ws + p.ws_off[K_QKV], tabs, mm, pubs_c, (unsigned)l + 1u, lane, abort_flag, sums, [&](unsigned dep) {
                        sq_l[0] = row_ssq_lane(p.ssq_a, d_tiles, mm[0], lane, dep);
                        sq_l[1] = row_ssq_lane(p.ssq_a, d_tiles, mm[1], lane, dep);
                    });
                    const float inv_q[2] = {inv_rms_from(sq_l[0], d, p.eps), inv_rms_from(sq_l[1], d, p.eps)};
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        const float inv = inv_q[q];
                        if (!on[q]) continue;                          // warp-uniform
                        const int t = tt[q], m = mm[q];
                        const int head = (t * tc::BLOCK_N + c_tile) / HD, ch = c_tile % HD;
                        const bool is_q = head < p.Hq, is_k = !is_q && head < p.Hq + p.Hkv;
                        const bool second = ch >= half;
                        float x[4] = {inv * sums[q].x, inv * sums[q].y, inv * sums[q].z, inv * sums[q].w};
                        if (p.qk_norm) {
                            float ss = x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3];
#pragma unroll
                            for (int o = HD / 8; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);   // over the head's lanes
                            if (is_q || is_k) {
                                const float hinv = 1.0f / sqrtf(ss / (float)HD + p.eps);
                                x[0] *= hinv * gq[q].x;
                                x[1] *= hinv * gq[q].y;
                                x[2] *= hinv * gq[q].z;
                                x[3] *= hinv * gq[q].w;
                            }
                        }
                        {   // rotate-half RoPE: element i of the first half pairs with i + half
                            const float c4[4] = {cs[q].x, cs[q].y, cs[q].z, cs[q].w}, s4r[4] = {sn[q].x, sn[q].y, sn[q].z, sn[q].w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float other = __shfl_xor_sync(0xffffffffu, x[e], PART);
                                const float y = second ? x[e] * c4[e] + other * s4r[e] : x[e] * c4[e] - other * s4r[e];
                                if (is_q || is_k) x[e] = y;
                            }
                        }
                        if (is_q) {
                            const size_t o = ((size_t)m * p.Hq + head) * HD + ch;
                            store_hi_lo_x4(p.q + o, p.q_lo + o, x[0], x[1], x[2], x[3]);
                        } else {
                            const int kvh = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
                            store_bf16x4((is_k ? p.k_rows : p.v_rows) + ((size_t)m * p.Hkv + kvh) * HD + ch, x[0], x[1], x[2], x[3]);
                            if (flags[q] & ROW_WRITE_KV)
                                store_bf16x4(p.pool.ptr(l, page[q], is_k ? 0 : 1, kvh, pos[q] & (p.pool.page_tokens - 1)) + ch, x[0], x[1], x[2],
                                             x[3]);
                        }
                    }
                }
            }
            grid_sync(true, p.moe ? tb : tb + 1, p.moe);
            if (!ok) break;
            // ---- attention items ----
            {
                att::AttnParams ap = p.ap;
                ap.layer = l;
                const int n_splits = ap.n_cache_splits + 1;
                const int total = ap.pv.n_seqs * ap.Hkv * ap.n_qtiles * n_splits;
                const FastDiv by_splits(n_splits), by_qtiles(ap.n_qtiles);
                // One sequence, dense model: the combine does not wait for a grid barrier behind the items but, pair by
                // pair, for the count of finished items of its (sequence, kv head, query tile), every item of which is
                // counted by the CTA that ran it.  (Several sequences: items are dealt out from a host-made list that
                // leaves out the splits without keys, and the barrier stays.)
                const bool counted = !p.moe && !ap.sched_off;
                // Items of this CTA: a host-made list when the pass has several sequences (their context
                // lengths differ, so items are dealt out by cost), else every G-th item.
                const int i_end = ap.sched_off ? __ldg(ap.sched_off + cta + 1) : total;
                for (int i = ap.sched_off ? __ldg(ap.sched_off + cta) : cta; i < i_end && ok; i += ap.sched_off ? 1 : G) {
                    const int idx = ap.sched_off ? __ldg(ap.sched_items + i) : i;
                    int r, split, z_i, qt_i;
                    by_splits.divmod(idx, r, split);
                    by_qtiles.divmod(r, z_i, qt_i);
                    bool fine;
                    if constexpr (HD == 128) {
                        // 64-token pages: the work item runs on tcgen05 (scores and output in tensor memory)
                        fine = ap.page_tokens == 64
                                   ? att::attn_item_umma<true>(p.maps + p.map_kv, ap, split, qt_i, z_i, attn_s, kv_full,
                                                               tmem_base + ACC_COLS, kv_ring, attn_s_cnt, attn_o_cnt, tid, BAR_COMPUTE,
                                                               attn_first_requested && idx == attn_first,
                                                               p.map_q >= 0 ? p.maps + p.map_q : nullptr, &attn_q_cnt)
                                   : att::attn_item<HD, true>(p.maps + p.map_kv, ap, split, qt_i, z_i, attn_s, kv_full,
                                                              kv_ring, tid, BAR_COMPUTE);
                    } else {
                        fine = att::attn_item<HD, true>(p.maps + p.map_kv, ap, split, qt_i, z_i, attn_s, kv_full, kv_ring,
                                                        tid, BAR_COMPUTE);
                    }
                    if (!fine) {
                        ok = false;
                        *abort_flag = 1;
                    }
                    if (counted) {
                        att::group_sync(BAR_COMPUTE, CTHREADS);      // every thread's part of the partial is stored
                        if (tid == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.attn_cnt + r) : "memory");
                    }
                }
                if (!ok) break;
                // the row table entries of this warp's first combine pair are fetched before the barrier, not behind it
                int pre_seq = 0, pre_row0 = 0, pre_nctx = 0;
                if (gw < M * p.Hq) {
                    int r, hq;
                    by_Hq.divmod(gw, r, hq);
                    pre_seq = __ldg(p.pv.row_seq + r);
                    pre_row0 = __ldg(p.pv.seq_row0 + pre_seq);
                    pre_nctx = __ldg(p.pv.seq_nctx + pre_seq);
                }
                if (counted) {
                    mark(tb + 3);
                } else {
                    grid_sync(false, tb + 3, p.moe);
                    if (!ok) break;
                }
                // ---- combine the key splits of every (row, query head) ----
                bool first_pair = true;
                for (int pair = gw; pair < M * p.Hq; pair += GW) {
                    int r, hq;
                    by_Hq.divmod(pair, r, hq);
                    const bool first = pair == gw;
                    const int seq = first ? pre_seq : __ldg(p.pv.row_seq + r), kvh = hq / ap.group;
                    const int qv = (r - (first ? pre_row0 : __ldg(p.pv.seq_row0 + seq))) * ap.group + hq % ap.group;
                    const int qt = qv / att::QT, qi = qv % att::QT;
                    const int n_ctx = first ? pre_nctx : __ldg(p.pv.seq_nctx + seq);
                    const int n_pages = (n_ctx + ap.page_tokens - 1) >> ap.page_shift;
                    const size_t item0 = ((size_t)(seq * ap.Hkv + kvh) * ap.n_qtiles + qt) * n_splits;
                    if (counted) {      // all items of this (sequence, kv head, query tile) have stored their partials
                        const unsigned* cntp = p.attn_cnt + (seq * ap.Hkv + kvh) * ap.n_qtiles + qt;
                        const unsigned target = (unsigned)n_splits * ((unsigned)l + 1u);
                        bool ready = false;
                        for (uint32_t it = 0; !ready && it < SPIN_LIMIT; ++it) {
                            ready = ld_acquire(cntp) >= target;
                            if (!ready && (it & 63u) == 63u && (*abort_flag || *(volatile int*)p.status != 0)) break;
                        }
                        if (!ready) {
                            atomicCAS(p.status, 0, 11);
                            *abort_flag = 1;
                            ok = false;
                            break;
                        }
                        if (first_pair) mark(tb + 4);
                        first_pair = false;
                    }
                    // Lanes take the splits for maxima and weights, and 4 output columns each (the
                    // first HD/4 lanes) for the sums.  Whether a split was written follows from the
                    // page count alone, so the loads of the partial outputs do not wait for the weights.
                    constexpr int CCH = 12;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    float lsum = 0.f;
                    for (int s0 = 0; s0 < n_splits; s0 += 32) {
                        const int s = s0 + lane;
                        const bool used = s < n_splits && (s == ap.n_cache_splits || s * ap.pages_per_split < n_pages);
                        float2 ml = make_float2(-INFINITY, 0.f);
                        if (used) ml = __ldcg(reinterpret_cast<const float2*>(ap.part_ml + (item0 + s) * att::QT * 2 + qi * 2));
                        // the first partial outputs are requested together with the maxima, before any weight is known
                        const int cnt = min(32, n_splits - s0);
                        float4 v[CCH];
                        auto load_chunk = [&](int k0) {
#pragma unroll
                            for (int k = 0; k < CCH; ++k) {
                                const int z = s0 + k0 + k;
                                const bool uz = k0 + k < cnt && (z == ap.n_cache_splits || z * ap.pages_per_split < n_pages);
                                v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
                                if (uz && lane < HD / 4) v[k] = __ldcg(reinterpret_cast<const float4*>(ap.part_o + ((item0 + z) * att::QT + qi) * HD) + lane);
                            }
                        };
                        load_chunk(0);
                        // the maximum over all splits is needed before any weight: second sweep when n_splits > 32
                        float mx = warp_max(ml.x);
                        for (int z0 = 0; z0 < n_splits; z0 += 32) {
                            if (z0 == s0) continue;
                            const int z = z0 + lane;
                            const bool uz = z < n_splits && (z == ap.n_cache_splits || z * ap.pages_per_split < n_pages);
                            mx = fmaxf(mx, warp_max(uz ? __ldcg(ap.part_ml + (item0 + z) * att::QT * 2 + qi * 2) : -INFINITY));
                        }
                        const float w_l = ml.x == -INFINITY ? 0.f : exp2f(ml.x - mx);
                        lsum += warp_sum(w_l * ml.y);
                        for (int k0 = 0; k0 < cnt; k0 += CCH) {
                            if (k0 > 0) load_chunk(k0);
#pragma unroll
                            for (int k = 0; k < CCH; ++k) {
                                const float w = __shfl_sync(0xffffffffu, w_l, (k0 + k) & 31);
                                if (k0 + k < cnt && w != 0.f) {
                                    acc.x += w * v[k].x;
                                    acc.y += w * v[k].y;
                                    acc.z += w * v[k].z;
                                    acc.w += w * v[k].w;
                                }
                            }
                        }
                    }
                    if (lane < HD / 4) {
                        const size_t o = ((size_t)r * p.Hq + hq) * HD + 4 * lane;
                        store_hi_lo_x4(p.attn + o, p.attn_lo + o, acc.x / lsum, acc.y / lsum, acc.z / lsum, acc.w / lsum);
                    }
                    publish_x(p.x_cnt[1] + hq * HD / tc::BLOCK_N);
                }
                if (counted && first_pair) mark(tb + 4);
                if (!ok) break;
            }
            // The O GEMM fetches the combined rows as their columns are counted, so dense layers need no
            // barrier here; from this point to the next layer's q/k/v the GEMMs of a dense layer follow each
            // other without one: every hand-over is a counted GEMM input or a counted partial, and every
            // buffer is next written only behind the grid barrier that follows the next layer's q/k/v,
            // which every CTA reaches after it has drained (hence read the inputs of) all of this layer's GEMMs.
            if (p.moe) {
                grid_sync(true, tb + 6, true);
                if (!ok) break;
            } else {
                mark(tb + 5);
            }
            // SwiGLU of a dense or shared-expert gate/up GEMM -> act (hi/lo), counted per tile
            // over the tiles [t_a, t_b) of the SwiGLU output
            auto swiglu_phase = [&](int gu_kind, int t_a, int t_b) {
                const int f_tiles = p.f / tc::BLOCK_N, n_pairs = (t_b - t_a) * M;
                // three (tile, row) pairs per step so that all their loads overlap
                constexpr int NP = 3;
                for (int pair = gw; pair < n_pairs; pair += NP * GW) {
                    int tt[NP], mm[NP], tabs[2 * NP], rows[2 * NP];
                    const unsigned* pubs[2 * NP];
                    SsqLane sq_l[NP];
                    bool on[NP];
#pragma unroll
                    for (int q = 0; q < NP; ++q) {
                        const int pr = pair + q * GW;
                        on[q] = pr < n_pairs;
                        by_M.divmod(on[q] ? pr : 0, tt[q], mm[q]);
                        tt[q] += t_a;
                        tabs[2 * q] = on[q] ? tile_row_tab(p, gu_kind, tt[q], lane) : 0;
                        tabs[2 * q + 1] = on[q] ? tile_row_tab(p, gu_kind, tt[q] + f_tiles, lane) : 0;
                        rows[2 * q] = rows[2 * q + 1] = mm[q];
                        pubs[2 * q] = p.tile_cnt[gu_kind] + tt[q];
                        pubs[2 * q + 1] = p.tile_cnt[gu_kind] + tt[q] + f_tiles;
                    }
                    float4 sums[2 * NP];
                    const unsigned* const pubs_c[2 * NP] = {pubs[0], pubs[1], pubs[2], pubs[3], pubs[4], pubs[5]};
                    tile_row_sums<2 * NP, 4>(p, p.ws + p.ws_off[gu_kind], tabs, rows, pubs_c, (unsigned)l + 1u, lane, abort_flag, sums, [&](unsigned dep) {
#pragma unroll
                        for (int q = 0; q < NP; ++q) sq_l[q] = row_ssq_lane(p.ssq_b, d_tiles, mm[q], lane, dep);
                    });
                    float inv_q[NP];
#pragma unroll
                    for (int q = 0; q < NP; ++q) inv_q[q] = inv_rms_from(sq_l[q], d, p.eps);
#pragma unroll
                    for (int q = 0; q < NP; ++q) {
                        const float inv = inv_q[q];
                        if (!on[q]) continue;
                        const float4 g4 = sums[2 * q], u4 = sums[2 * q + 1];
                        const float gv[4] = {inv * g4.x, inv * g4.y, inv * g4.z, inv * g4.w};
                        const float uv[4] = {inv * u4.x, inv * u4.y, inv * u4.z, inv * u4.w};
                        float a[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) a[e] = __fdividef(gv[e], 1.f + __expf(-gv[e])) * uv[e];   // fast exp and divide: 2^-21, far below what the later stages add
                        const size_t o = (size_t)mm[q] * p.f + tt[q] * tc::BLOCK_N + 4 * lane;
                        store_hi_lo_x4(p.act + o, p.act_lo + o, a[0], a[1], a[2], a[3]);
                    }
                    // the writers' proxy fence, one release for the step's stores, then one count per finished pair
                    asm volatile("fence.proxy.async.global;" ::: "memory");
                    __syncwarp();
                    if (lane == 0) {
                        asm volatile("fence.acq_rel.gpu;" ::: "memory");
#pragma unroll
                        for (int q = 0; q < NP; ++q)
                            if (on[q]) asm volatile("red.relaxed.gpu.global.add.u32 [%0], 1;" ::"l"(p.x_cnt[2] + tt[q]) : "memory");
                    }
                }
            };
            const float* next_gain = l + 1 < p.n_layers ? p.gains[l + 1].attn_norm : p.final_norm;
            if (!p.moe) {
                // ---- O GEMM, residual; gate/up GEMM, SwiGLU; down GEMM, residual (prepares the next layer's or the
                // head's input).  Each runs sub-GEMM by sub-GEMM: once a sub-GEMM that completes a group of output
                // tiles is drained, the element-wise phase over that group follows, while the tensor pipe is already
                // on the next sub-GEMM (the accumulator ring holds what it finishes meanwhile).
                for (int sub = 0; sub < p.n_subs[K_O] && ok; ++sub) {
                    drain_sub(l, K_O, sub);
                    if (sub + 1 == p.n_subs[K_O]) mark(tb + 6);
                    const SubDesc& sd = p.subs[K_O][sub];
                    if (ok && sd.ew_t1 > sd.ew_t0) residual_phase(K_O, (unsigned)l + 1u, lg.ffn_norm, p.ssq_b, true, sd.ew_t0, sd.ew_t1);
                }
                mark(tb + 7);
                for (int sub = 0; sub < p.n_subs[K_GU] && ok; ++sub) {
                    drain_sub(l, K_GU, sub);
                    if (sub + 1 == p.n_subs[K_GU]) mark(tb + 8);
                    const SubDesc& sd = p.subs[K_GU][sub];
                    if (ok && sd.ew_t1 > sd.ew_t0) swiglu_phase(K_GU, sd.ew_t0, sd.ew_t1);
                }
                mark(tb + 9);
                for (int sub = 0; sub < p.n_subs[K_DOWN] && ok; ++sub) {
                    drain_sub(l, K_DOWN, sub);
                    if (sub + 1 == p.n_subs[K_DOWN]) mark(tb + 10);
                    const SubDesc& sd = p.subs[K_DOWN][sub];
                    if (ok && sd.ew_t1 > sd.ew_t0) residual_phase(K_DOWN, (unsigned)l + 1u, next_gain, p.ssq_a, false, sd.ew_t0, sd.ew_t1);
                }
                mark(tb + 11);
                if (*abort_flag) ok = false;
                continue;
            }
            // ---- O GEMM, residual ----
            drain(l, K_O);
            if (!ok) break;
            residual_phase(K_O, (unsigned)l + 1u, lg.ffn_norm, p.ssq_b, true, 0, d_tiles);
            grid_sync(true, tb + 9, true);
            if (!ok) break;
            // ================= mixture of experts =================
            // ---- router GEMM; per row: softmax over the experts, top-k (ties -> lowest id), gates renormalised ----
            drain(l, K_ROUTER);
            if (!ok) break;
            {
                const int e_tiles = p.n_experts / tc::BLOCK_N;     // 1 or 2
                for (int m = gw; m < M; m += GW) {
                    int tabs[2], rows[2] = {m, m};
                    const unsigned* pubs[2];
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        tabs[t] = t < e_tiles ? tile_row_tab(p, K_ROUTER, t, lane) : 0;
                        pubs[t] = p.tile_cnt[K_ROUTER] + t;
                    }
                    const SsqLane sq_l = row_ssq_lane(p.ssq_b, d_tiles, m, lane);
                    float4 sums[2];
                    const unsigned* const pubs_c[2] = {pubs[0], pubs[1]};
                    tile_row_sums<2, 8>(p, p.ws + p.ws_off[K_ROUTER], tabs, rows, pubs_c, (unsigned)l + 1u, lane, abort_flag, sums);
                    const float inv = inv_rms_from(sq_l, d, p.eps);
                    // lane holds logits of experts 4*lane .. +3 (tile 0) and 128 + 4*lane .. +3 (tile 1)
                    float x[8] = {inv * sums[0].x, inv * sums[0].y, inv * sums[0].z, inv * sums[0].w,
                                  inv * sums[1].x, inv * sums[1].y, inv * sums[1].z, inv * sums[1].w};
                    const int n_mine = 4 * e_tiles;
                    float mx = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (i < n_mine) mx = fmaxf(mx, x[i]);
                    mx = warp_max(mx);
                    float sum = 0.f;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (i < n_mine) sum += expf(x[i] - mx);
                    sum = warp_sum(sum);
                    float last_v = INFINITY, kept = 0.f, my_gate = 0.f;
                    int last_i = -1, my_id = 0;
                    for (int k = 0; k < p.top_k; ++k) {
                        // candidates strictly after (last_v, last_i) in the order (value desc, id asc)
                        float bv = -INFINITY;
                        int bi = 0x7fffffff;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            if (i >= n_mine) continue;
                            const int e = (i >> 2) * tc::BLOCK_N + 4 * lane + (i & 3);
                            const float v = x[i];
                            const bool after = (v < last_v) || (v == last_v && e > last_i);
                            if (after && (v > bv || (v == bv && e < bi))) {
                                bv = v;
                                bi = e;
                            }
                        }
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) {
                            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                            if (ov > bv || (ov == bv && oi < bi)) {
                                bv = ov;
                                bi = oi;
                            }
                        }
                        last_v = bv;
                        last_i = bi;
                        const float pk = expf(bv - mx) / sum;
                        kept += pk;
                        if (lane == k) {
                            my_gate = pk;
                            my_id = bi;
                        }
                    }
                    if (lane < p.top_k) {
                        p.moe_ids[(size_t)m * p.top_k + lane] = my_id;
                        p.moe_gates[(size_t)m * p.top_k + lane] = my_gate / kept;
                        p.moe_ids_trace[(size_t)l * p.trace_stride + (size_t)m * p.top_k + lane] = my_id;
                    }
                }
            }
            grid_sync(false, tb + 12, true);
            if (!ok) break;
            // ---- the touched experts of this layer, ascending; every CTA builds the same list ----
            {
                if (tid < MAX_EXPERTS / 32) routing->mask[tid] = 0;
                att::group_sync(BAR_COMPUTE, CTHREADS);
                for (int i = tid; i < M * p.top_k; i += CTHREADS) {
                    const int e = __ldcg(p.moe_ids + i);
                    atomicOr(&routing->mask[e >> 5], 1 << (e & 31));
                }
                att::group_sync(BAR_COMPUTE, CTHREADS);
                int before = 0;
                for (int w = 0; w < MAX_EXPERTS / 32; ++w) {
                    const unsigned mword = (unsigned)routing->mask[w];
                    for (int e = tid; e < 32; e += CTHREADS)   // tid < 32: one word per round
                        if (mword >> e & 1u) {
                            const int pos = before + __popc(mword & ((1u << e) - 1u));
                            routing->list[pos] = (short)(w * 32 + e);
                            routing->slot_of[w * 32 + e] = (short)pos;
                        }
                    before += __popc(mword);
                }
                att::group_sync(BAR_COMPUTE, CTHREADS);
                if (tid == 0) {
                    routing->n_touched = before;
                    __threadfence_block();
                    routing->layer_ready = l + 1;
                    if (cta == 0) p.n_touched_out[l] = before;
                }
                att::group_sync(BAR_COMPUTE, CTHREADS);
            }
            const int n_touched = routing->n_touched;
            // ---- shared expert gate/up, SwiGLU (its weights do not depend on the routing) ----
            drain(l, K_SGU);
            if (!ok) break;
            swiglu_phase(K_SGU, 0, p.f / tc::BLOCK_N);
            // ---- routed experts gate/up over all rows; SwiGLU only for the (row, expert) pairs that were routed ----
            drain(l, K_EGU);
            if (!ok) break;
            grid_sync(true, tb + 15, true);
            if (!ok) break;
            {
                const GemmShape g = gemm_shape(p, l, K_EGU, 0, n_touched);
                const int fe_tiles = p.fe / tc::BLOCK_N;
                const int n_items = M * p.top_k * fe_tiles;
                const float* wsb = p.ws + p.ws_off[K_EGU];
                for (int item = gw; item < n_items; item += GW) {
                    const int j = item % fe_tiles, rs = item / fe_tiles, m = rs / p.top_k;
                    const int slot = routing->slot_of[__ldcg(p.moe_ids + rs)];
                    const SsqLane sq_l = row_ssq_lane(p.ssq_b, d_tiles, m, lane);
                    const int tg = slot * g.tpe + j, tu = tg + fe_tiles;
                    const int tabs[2] = {dyn_tab(g, tg, G, p.max_segs[K_EGU], lane), dyn_tab(g, tu, G, p.max_segs[K_EGU], lane)};
                    const int rows[2] = {m, m};
                    const unsigned* const pubs[2] = {nullptr, nullptr};
                    float4 sums[2];
                    tile_row_sums<2, 8>(p, wsb, tabs, rows, pubs, 0u, lane, abort_flag, sums);
                    const float inv = inv_rms_from(sq_l, d, p.eps);
                    const float gv[4] = {inv * sums[0].x, inv * sums[0].y, inv * sums[0].z, inv * sums[0].w};
                    const float uv[4] = {inv * sums[1].x, inv * sums[1].y, inv * sums[1].z, inv * sums[1].w};
                    float a[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) a[e] = __fdividef(gv[e], 1.f + __expf(-gv[e])) * uv[e];
                    const size_t o = ((size_t)slot * T + m) * p.fe + j * tc::BLOCK_N + 4 * lane;
                    store_hi_lo_x4(p.act_e + o, p.act_e_lo + o, a[0], a[1], a[2], a[3]);
                }
            }
            grid_sync(true, tb + 18, true);
            if (!ok) break;
            // ---- shared and routed down GEMMs; h += shared + sum_k gate_k * expert_k; next layer's input ----
            drain(l, K_SDOWN);
            if (!ok) break;
            drain(l, K_EDOWN);
            if (!ok) break;
            grid_sync(false, tb + 21, true);
            if (!ok) break;
            {
                const GemmShape g = gemm_shape(p, l, K_EDOWN, 0, n_touched);
                const float* wsb = p.ws + p.ws_off[K_EDOWN];
                h_phase(next_gain, p.ssq_a, p.xn, p.xn_lo, p.x_cnt[0], 0, d_tiles, [&](int t, int m, int col) {
                    const float4 hv = __ldcg(reinterpret_cast<const float4*>(p.h + (size_t)m * d + col));
                    float4 x;
                    {   // shared expert
                        const int tabs[1] = {tile_row_tab(p, K_SDOWN, t, lane)}, rows[1] = {m};
                        const unsigned* const pubs[1] = {nullptr};
                        float4 sums[1];
                        tile_row_sums<1, 8>(p, p.ws + p.ws_off[K_SDOWN], tabs, rows, pubs, 0u, lane, abort_flag, sums);
                        x = sums[0];
                    }
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int k0 = 0; k0 < p.top_k; k0 += 4) {     // routed experts in slot order, four at a time
                        int tabs[4], rows[4] = {m, m, m, m};
                        float gk[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const bool on = k0 + q < p.top_k;
                            const int e = on ? __ldcg(p.moe_ids + (size_t)m * p.top_k + k0 + q) : 0;
                            gk[q] = on ? __ldcg(p.moe_gates + (size_t)m * p.top_k + k0 + q) : 0.f;
                            tabs[q] = on ? dyn_tab(g, routing->slot_of[e] * g.tpe + t, G, p.max_segs[K_EDOWN], lane) : 0;
                        }
                        const unsigned* const pubs[4] = {nullptr, nullptr, nullptr, nullptr};
                        float4 sums[4];
                        tile_row_sums<4, 4>(p, wsb, tabs, rows, pubs, 0u, lane, abort_flag, sums);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            acc.x += gk[q] * sums[q].x;
                            acc.y += gk[q] * sums[q].y;
                            acc.z += gk[q] * sums[q].z;
                            acc.w += gk[q] * sums[q].w;
                        }
                    }
                    x.x = hv.x + (acc.x + x.x);
                    x.y = hv.y + (acc.y + x.y);
                    x.z = hv.z + (acc.z + x.z);
                    x.w = hv.w + (acc.w + x.w);
                    return x;
                });
            }
            grid_sync(true, tb + 24, true);
        }
        if (ok && p.n_logit > 0) {
            // ---- LM head on the rows that need logits ----
            t_drained = 0;
            drain(p.n_layers, K_LM);
            if (ok) {
                const int n_tiles = (p.V + tc::BLOCK_N - 1) / tc::BLOCK_N;
                const bool vec = (p.V & 3) == 0;
                // one item = a 128-column tile and up to four logit rows: the tile's part list and
                // counter are fetched once and the partials of all four rows are in flight together
                constexpr int NR = 4;
                const int groups = (p.n_logit + NR - 1) / NR;
                const FastDiv by_groups(groups);
                for (int item = gw; item < n_tiles * groups; item += GW) {
                    int t, lr0;
                    by_groups.divmod(item, t, lr0);
                    lr0 *= NR;
                    const int tab = tile_row_tab(p, 4, t, lane);
                    int tabs[NR], rows[NR];
                    const unsigned* pubs[NR];
                    SsqLane sq_l[NR];
#pragma unroll
                    for (int q = 0; q < NR; ++q) {
                        const bool on = lr0 + q < p.n_logit;
                        rows[q] = on ? __ldg(p.pv.logit_rows + lr0 + q) : 0;
                        tabs[q] = on ? tab : 0;
                        pubs[q] = p.tile_cnt[4] + t;
                    }
                    const unsigned* const pubs_c[NR] = {pubs[0], pubs[1], pubs[2], pubs[3]};
                    float4 sums[NR];
                    tile_row_sums<NR, 2>(p, p.ws + p.ws_off[K_LM], tabs, rows, pubs_c, 1u, lane, abort_flag, sums, [&](unsigned dep) {
#pragma unroll
                        for (int q = 0; q < NR; ++q) sq_l[q] = row_ssq_lane(p.ssq_a, d_tiles, rows[q], lane, dep);
                    });
                    float sc_q[NR];
#pragma unroll
                    for (int q = 0; q < NR; ++q) sc_q[q] = p.logit_scale * inv_rms_from(sq_l[q], d, p.eps);
                    const int col = t * tc::BLOCK_N + 4 * lane;
#pragma unroll
                    for (int q = 0; q < NR; ++q) {
                        const float sc = sc_q[q];
                        if (lr0 + q >= p.n_logit) continue;        // warp-uniform
                        const float4 s4 = sums[q];
                        float* dst = p.logits + (size_t)(lr0 + q) * p.V + col;
                        if (vec && col + 3 < p.V) {
                            *reinterpret_cast<float4*>(dst) = make_float4(sc * s4.x, sc * s4.y, sc * s4.z, sc * s4.w);
                        } else {
                            const float o[4] = {sc * s4.x, sc * s4.y, sc * s4.z, sc * s4.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e)
                                if (col + e < p.V) dst[e] = o[e];
                        }
                    }
                }
            }
        }
        // the LM-head phase ends without a barrier: its two marks are the time this CTA had drained its
        // LM-head accumulators and the time it finished its logits
        if (p.trace && tid == 0) {
            const int k = 3 + (p.moe ? 27 : 12) * p.n_layers;
            if (k + 1 < p.trace_cap - 1) {
                p.trace[(size_t)cta * p.trace_cap + k] = t_drained;
                mark(k + 1);
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
    if (warp == 2) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

}  // namespace pp
}  // namespace s2d2
