// Vocabulary-wide kernels of the decode step: SampleFromLogits statistics of the
// draft rows, and the fused acceptance kernel (ScoreFromLogits, ratio test against
// Philox uniforms, first rejection, residual resampling).
//
// Precision: sums of exponentials, the acceptance ratio and the residual
// distribution are evaluated in fp64 from the fp32 logits.  The residual
// (pi_v - pi_d)_+ is a difference of nearly equal numbers when drafter and
// verifier agree; an fp32 normaliser would move its inverse CDF by far more than
// one token's mass on a 150k-wide vocabulary.
#pragma once
#include "common.cuh"

namespace s2d2 {


struct Top2 {
    float v1;   // best value
    int i1;     // its index (lowest id among equals)
    float v2;   // second best value (== v1 when the maximum is attained twice)
};
__device__ __forceinline__ Top2 top2_merge(Top2 a, Top2 b) {
    bool a_first = (a.v1 > b.v1) || (a.v1 == b.v1 && a.i1 < b.i1);
    Top2 w = a_first ? a : b, l = a_first ? b : a;
    w.v2 = fmaxf(w.v2, l.v1);
    return w;
}
__device__ __forceinline__ Top2 top2_push(Top2 t, float v, int i) {
    if (v > t.v1) {           // ids are visited in ascending order inside a thread: strict > keeps the lowest id
        t.v2 = t.v1;
        t.v1 = v;
        t.i1 = i;
    } else if (v > t.v2) {
        t.v2 = v;
    }
    return t;
}
__device__ __forceinline__ Top2 block_top2(Top2 t, Top2* sh) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 other;
        other.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        other.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        other.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, other);
    }
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sh[w] = t;
    __syncthreads();
    if (w == 0) {
        int nw = blockDim.x >> 5;
        Top2 x = lane < nw ? sh[lane] : Top2{-INFINITY, 0x7fffffff, -INFINITY};
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            Top2 other;
            other.v1 = __shfl_xor_sync(0xffffffffu, x.v1, o);
            other.i1 = __shfl_xor_sync(0xffffffffu, x.i1, o);
            other.v2 = __shfl_xor_sync(0xffffffffu, x.v2, o);
            x = top2_merge(x, other);
        }
        if (lane == 0) sh[0] = x;
    }
    __syncthreads();
    return sh[0];
}
__device__ __forceinline__ double block_sum_d(double v, double* sh) {
    v = warp_sum(v);
    int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) sh[w] = v;
    __syncthreads();
    if (w == 0) {
        int nw = blockDim.x >> 5;
        double x = lane < nw ? sh[lane] : 0.0;
        x = warp_sum(x);
        if (lane == 0) sh[0] = x;
    }
    __syncthreads();
    return sh[0];
}

struct DraftStatsOut {
    int* xhat;
    float* conf;      // pi_d(xhat)
    float* margin;    // top-1 minus top-2 probability
    float* entropy;
    double* lse;      // log-sum-exp of the row, fp64
};

// ---------------------------------------------------------------------------------------------
// Stage 1, shared by the draft statistics and the acceptance step: the vocabulary of every logit
// row is cut into chunks of VCHUNK entries, one CTA per (chunk, row), so that a handful of rows
// still fills the GPU.  Per chunk: its top-2, and sum exp(x - max_chunk), sum x exp(x - max_chunk)
// in fp64.  Stage 2 kernels merge the chunks of a row in chunk order.
// ---------------------------------------------------------------------------------------------
constexpr int VCHUNK = 4096;
constexpr int VCHUNK_THREADS = 256;
constexpr int VPER = VCHUNK / VCHUNK_THREADS;   // 16 entries per thread

struct ChunkStats {
    float mx;      // largest logit of the chunk
    int arg;       // its index (lowest id among equals)
    float mx2;     // second largest (== mx when attained twice)
    int pad;
    double s;      // sum exp(x - mx)
    double sx;     // sum x * exp(x - mx)
};
__host__ __device__ inline int vocab_chunks(int V) { return (V + VCHUNK - 1) / VCHUNK; }

// Loads the VPER entries of thread t of a chunk: entries (k * 256 + t) * 4 .. + 3 for k = 0..3
// (ids ascending inside a thread); entries past V read as -inf.
__device__ __forceinline__ void load_chunk_strided(const float* row, int V, int base, int t, float (&x)[VPER]) {
    const bool vec = (V & 3) == 0;
#pragma unroll
    for (int k = 0; k < VPER / 4; ++k) {
        const int i0 = base + (k * VCHUNK_THREADS + t) * 4;
        if (vec && i0 + 3 < V) {
            const float4 v = *reinterpret_cast<const float4*>(row + i0);
            x[4 * k] = v.x;
            x[4 * k + 1] = v.y;
            x[4 * k + 2] = v.z;
            x[4 * k + 3] = v.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) x[4 * k + e] = i0 + e < V ? row[i0 + e] : -INFINITY;
        }
    }
}

// One (chunk, row) by the whole CTA of VCHUNK_THREADS threads; thread 0 writes *out.
__device__ __forceinline__ void chunk_stats_block(const float* __restrict__ row, int V, int chunk, ChunkStats* __restrict__ out,
                                                  Top2* sh_t, double* sh_d) {
    const int base = chunk * VCHUNK;
    float x[VPER];
    load_chunk_strided(row, V, base, threadIdx.x, x);
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
#pragma unroll
    for (int k = 0; k < VPER; ++k) t = top2_push(t, x[k], base + ((k >> 2) * VCHUNK_THREADS + threadIdx.x) * 4 + (k & 3));
    t = block_top2(t, sh_t);
    const double mx = (double)t.v1;
    double s = 0.0, sx = 0.0;
#pragma unroll
    for (int k = 0; k < VPER; ++k) {
        if (x[k] != -INFINITY) {
            const double xi = (double)x[k], e = exp(xi - mx);
            s += e;
            sx += e * xi;
        }
    }
    s = block_sum_d(s, sh_d);
    sx = block_sum_d(sx, sh_d);
    if (threadIdx.x == 0) {
        ChunkStats o;
        o.mx = t.v1;
        o.arg = t.i1;
        o.mx2 = t.v2;
        o.pad = 0;
        o.s = s;
        o.sx = sx;
        *out = o;
    }
}
static __global__ void __launch_bounds__(VCHUNK_THREADS) vocab_chunk_stats_kernel(const float* __restrict__ logits, int V,
                                                                                  ChunkStats* __restrict__ out) {
    __shared__ Top2 sh_t[32];
    __shared__ double sh_d[32];
    const int chunk = blockIdx.x, r = blockIdx.y, n_chunks = gridDim.x;
    chunk_stats_block(logits + (size_t)r * V, V, chunk, out + (size_t)r * n_chunks + chunk, sh_t, sh_d);
}

// Merge of a row's chunks by one warp: top-2 in chunk order, then the sums rescaled to the row
// maximum.  Every lane returns the same values.
struct RowStats {
    Top2 t;
    double s, sx;
};
__device__ __forceinline__ RowStats warp_row_stats(const ChunkStats* cs, int n_chunks, int lane) {
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int c = lane; c < n_chunks; c += 32) {
        Top2 o{cs[c].mx, cs[c].arg, cs[c].mx2};
        t = top2_merge(t, o);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        Top2 other;
        other.v1 = __shfl_xor_sync(0xffffffffu, t.v1, o);
        other.i1 = __shfl_xor_sync(0xffffffffu, t.i1, o);
        other.v2 = __shfl_xor_sync(0xffffffffu, t.v2, o);
        t = top2_merge(t, other);
    }
    const double mx = (double)t.v1;
    double s = 0.0, sx = 0.0;
    for (int c = lane; c < n_chunks; c += 32) {
        const double w = exp((double)cs[c].mx - mx);
        s += cs[c].s * w;
        sx += cs[c].sx * w;
    }
    RowStats r;
    r.t = t;
    r.s = warp_sum(s);
    r.sx = warp_sum(sx);
    return r;
}

// SampleFromLogits, greedy, stage 2: one warp per logit row.
static __global__ void draft_finish_kernel(const ChunkStats* __restrict__ cs, int n_chunks, int n_rows, DraftStatsOut o) {
    const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (r >= n_rows) return;
    const RowStats st = warp_row_stats(cs + (size_t)r * n_chunks, n_chunks, lane);
    if (lane == 0) {
        const double mx = (double)st.t.v1, lse = mx + log(st.s);
        o.xhat[r] = st.t.i1;
        o.conf[r] = (float)(1.0 / st.s);
        o.margin[r] = (float)((1.0 - exp((double)st.t.v2 - mx)) / st.s);
        o.entropy[r] = (float)(lse - st.sx / st.s);
        o.lse[r] = lse;
    }
}

struct AcceptIn {
    const float* draft_logits;
    const float* verify_logits;
    int V;
    const int* seq_draft_row0;    // first draft-logit row of the span, per sequence
    const int* seq_verify_row0;   // first verifier-logit row of the span
    const int* seq_len;           // L
    const int* seq_pos0;          // absolute position of the span's first token
    const unsigned* seq_stream;   // Philox sequence stream
    const int* seq_step;          // Philox step word
    const int* xhat;              // per draft-logit row
    const double* draft_lse;      // per draft-logit row (may be null: taken from draft_chunks)
    const int* seq_mode;          // 1: acceptance scan; 0: confidence branch (may be null: all 1)
    const float* conf;            // per draft-logit row, for the confidence branch
    const ChunkStats* verify_chunks;   // stage-1 output over the verifier-logit rows
    const ChunkStats* draft_chunks;    // stage-1 output over the draft-logit rows (when draft_lse is null)
    float tau_conf;
    unsigned seed;
    float gamma;
    float accept_override;        // > 0: a_i is this constant instead of min(1, (v_i/d_i)^gamma)
    int resample;
    int l_cap;                    // stride of the per-position outputs
};
struct AcceptOut {
    int* n_accepted;
    int* first_reject;
    int* resampled;
    int* n_near;
    unsigned* commit_bits;   // confidence branch: bit k = k-th masked position is committed
    float* u;   // [n_seqs, l_cap]
    float* a;
    float* v;
};
// What the residual kernels need to know about a sequence's rejected position.
struct RejectInfo {
    int draft_row, verify_row;   // logit rows; draft_row < 0: nothing to resample
    unsigned pos;
    int pad;
    double lse_d, lse_v;
};

// Acceptance scan, one CTA of 128 threads per sequence (Algorithm "SampleBlock for S2D2", the
// left-to-right loop; the else-branch for sequences that were not verified).  Warps merge the
// verifier chunks of the span's rows, thread i evaluates position i (v_i, d_i, a_i, u_i), thread 0
// scans left to right up to the first rejection.
struct ScanShared {
    double lse_v[32], lse_d[32], a[32], u[32], v[32];
};
// Sequence s by the whole CTA (any number of warps).
__device__ __forceinline__ void accept_scan_block(const AcceptIn& in, const AcceptOut& out, RejectInfo* rej, int s, ScanShared& sh) {
    double *sh_lse_v = sh.lse_v, *sh_lse_d = sh.lse_d, *sh_a = sh.a, *sh_u = sh.u, *sh_v = sh.v;
    const int L = in.seq_len[s];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_chunks = vocab_chunks(in.V);
    if (threadIdx.x == 0) rej[s].draft_row = -1;
    if (in.seq_mode && in.seq_mode[s] == 0) {
        // Not verified: S = {i in M_t : d_i > tau} U {argmax d_i} (ties -> leftmost); L = |M_t| here.
        if (threadIdx.x == 0) {
            unsigned bits = 0;
            int best = 0;
            const float* c = in.conf + in.seq_draft_row0[s];
            for (int k = 0; k < L; ++k) {
                if (c[k] > in.tau_conf) bits |= 1u << k;
                if (c[k] > c[best]) best = k;
            }
            out.commit_bits[s] = bits | (1u << best);
            out.n_accepted[s] = 0;
            out.first_reject[s] = -1;
            out.resampled[s] = -1;
            out.n_near[s] = 0;
        }
        return;
    }
    const int dr0 = in.seq_draft_row0[s], vr0 = in.seq_verify_row0[s];
    for (int i = warp; i < L; i += (int)(blockDim.x >> 5)) {
        const RowStats sv = warp_row_stats(in.verify_chunks + (size_t)(vr0 + i) * n_chunks, n_chunks, lane);
        if (lane == 0) sh_lse_v[i] = (double)sv.t.v1 + log(sv.s);
        if (in.draft_lse) {
            if (lane == 0) sh_lse_d[i] = in.draft_lse[dr0 + i];
        } else {
            const RowStats sd = warp_row_stats(in.draft_chunks + (size_t)(dr0 + i) * n_chunks, n_chunks, lane);
            if (lane == 0) sh_lse_d[i] = (double)sd.t.v1 + log(sd.s);
        }
    }
    __syncthreads();
    if ((int)threadIdx.x < L) {
        const int i = threadIdx.x, tok = in.xhat[dr0 + i];
        const double xv = (double)in.verify_logits[(size_t)(vr0 + i) * in.V + tok];
        const double xd = (double)in.draft_logits[(size_t)(dr0 + i) * in.V + tok];
        const double v = exp(xv - sh_lse_v[i]), d = exp(xd - sh_lse_d[i]);
        double ratio = v / d;
        if (in.gamma != 1.f) ratio = pow(ratio, (double)in.gamma);
        sh_v[i] = v;
        sh_a[i] = in.accept_override > 0.f ? (double)in.accept_override : fmin(1.0, ratio);
        sh_u[i] = philox_uniform(in.seed, (unsigned)(in.seq_pos0[s] + i), in.seq_stream[s], (unsigned)in.seq_step[s], STREAM_ACCEPT);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int n_acc = 0, first_rej = -1, near = 0;
        for (int i = 0; i < L; ++i) {
            const double u = sh_u[i], a = sh_a[i];
            out.u[(size_t)s * in.l_cap + i] = (float)u;
            out.a[(size_t)s * in.l_cap + i] = (float)a;
            out.v[(size_t)s * in.l_cap + i] = (float)sh_v[i];
            if (fabs(u - a) < 1e-4) ++near;
            if (u < a) {
                ++n_acc;
                continue;
            }
            first_rej = i;
            break;
        }
        out.n_accepted[s] = n_acc;
        out.first_reject[s] = first_rej;
        out.resampled[s] = -1;
        out.n_near[s] = near;
        if (first_rej >= 0 && in.resample) {
            RejectInfo r;
            r.draft_row = dr0 + first_rej;
            r.verify_row = vr0 + first_rej;
            r.pos = (unsigned)(in.seq_pos0[s] + first_rej);
            r.pad = 0;
            r.lse_d = sh_lse_d[first_rej];
            r.lse_v = sh_lse_v[first_rej];
            rej[s] = r;
        }
    }
}

// Residual (pi_v - pi_d)_+ of the rejected position, stage 1: per (chunk, sequence) the chunk's
// residual mass and its pi_v mass in fp64.  Thread t owns the 16 consecutive entries
// [base + 16 t, base + 16 t + 16) so that prefixes over threads follow the vocabulary order.
__device__ __forceinline__ void load_chunk_contiguous(const float* row, int V, int base, int t, float (&x)[VPER]) {
    const bool vec = (V & 3) == 0;
#pragma unroll
    for (int k = 0; k < VPER / 4; ++k) {
        const int i0 = base + t * VPER + 4 * k;
        if (vec && i0 + 3 < V) {
            const float4 v = *reinterpret_cast<const float4*>(row + i0);
            x[4 * k] = v.x;
            x[4 * k + 1] = v.y;
            x[4 * k + 2] = v.z;
            x[4 * k + 3] = v.w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) x[4 * k + e] = i0 + e < V ? row[i0 + e] : -INFINITY;
        }
    }
}
// SampleFromLogits, sampling mode: xhat ~ pi_d by inverse CDF in vocabulary order with one uniform of the
// draft-sampling Philox stream; conf = pi_d(xhat).  One CTA per logit row, after stage 1 and the greedy stage 2
// (which leave margin, entropy and the log-sum-exp of the row; this kernel replaces xhat and conf).  Thread 0 walks
// the chunk masses s_c * exp(mx_c - mx) to the chunk that holds u * sum, the CTA then walks that chunk (prefix over
// threads in vocabulary order, then the owning thread over its 16 entries), all in fp64.
struct DraftSampleIn {
    const float* logits;
    int V;
    const ChunkStats* chunks;
    const int* row_pos;          // absolute position of the row's token
    const unsigned* row_stream;  // Philox sequence stream
    const int* row_step;         // Philox step word
    unsigned seed;
};
static __global__ void __launch_bounds__(VCHUNK_THREADS) draft_sample_kernel(DraftSampleIn in, int n_chunks, DraftStatsOut o) {
    __shared__ double sh_warp[VCHUNK_THREADS / 32];
    __shared__ double sh_target, sh_mx;
    __shared__ int sh_chunk, sh_pick;
    const int r = blockIdx.x;
    const ChunkStats* cs = in.chunks + (size_t)r * n_chunks;
    const float* row = in.logits + (size_t)r * in.V;
    if (threadIdx.x == 0) {
        float mxf = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) mxf = fmaxf(mxf, cs[c].mx);
        const double mx = (double)mxf;
        double total = 0.0;
        for (int c = 0; c < n_chunks; ++c) total += cs[c].s * exp((double)cs[c].mx - mx);
        const double u = philox_uniform(in.seed, (unsigned)in.row_pos[r], in.row_stream[r], (unsigned)in.row_step[r], STREAM_DRAFT);
        const double target = u * total;
        double before = 0.0;
        int pick_chunk = -1;
        for (int c = 0; c < n_chunks; ++c) {
            const double m = cs[c].s * exp((double)cs[c].mx - mx);
            if (before + m > target) {
                pick_chunk = c;
                break;
            }
            before += m;
        }
        sh_chunk = pick_chunk;
        sh_target = target - before;
        sh_mx = mx;
        sh_pick = in.V - 1;
    }
    __syncthreads();
    const int chunk = sh_chunk;
    if (chunk >= 0) {
        const double target = sh_target, mx = sh_mx;
        float x[VPER];
        load_chunk_contiguous(row, in.V, chunk * VCHUNK, threadIdx.x, x);
        double w[VPER], mine = 0.0;
#pragma unroll
        for (int k = 0; k < VPER; ++k) {
            w[k] = x[k] == -INFINITY ? 0.0 : exp((double)x[k] - mx);
            mine += w[k];
        }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        double incl = mine;
#pragma unroll
        for (int k = 1; k < 32; k <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, k);
            if (lane >= k) incl += up;
        }
        if (lane == 31) sh_warp[warp] = incl;
        __syncthreads();
        double before = incl - mine;
        for (int k = 0; k < warp; ++k) before += sh_warp[k];
        if (before <= target && before + mine > target) {
            int pick = VPER - 1;
#pragma unroll
            for (int k = VPER - 1; k >= 0; --k) {
                double upto = before;
#pragma unroll
                for (int j = 0; j < VPER; ++j)
                    if (j <= k) upto += w[j];
                if (upto > target) pick = k;
            }
            atomicMin(&sh_pick, min(in.V - 1, chunk * VCHUNK + (int)threadIdx.x * VPER + pick));
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const int tok = sh_pick;
        o.xhat[r] = tok;
        o.conf[r] = (float)exp((double)row[tok] - o.lse[r]);
    }
}

// One chunk of the rejected position's residual by the whole CTA: thread 0 writes the chunk's residual mass and pi_v mass.
__device__ __forceinline__ void residual_chunk_block(const AcceptIn& in, const RejectInfo& r, int chunk, double* rs_out, double* vs_out,
                                                     double* sh_d) {
    float xv[VPER], xd[VPER];
    load_chunk_contiguous(in.verify_logits + (size_t)r.verify_row * in.V, in.V, chunk * VCHUNK, threadIdx.x, xv);
    load_chunk_contiguous(in.draft_logits + (size_t)r.draft_row * in.V, in.V, chunk * VCHUNK, threadIdx.x, xd);
    double rs = 0.0, vs = 0.0;
#pragma unroll
    for (int k = 0; k < VPER; ++k) {
        if (xv[k] == -INFINITY && xd[k] == -INFINITY) continue;      // past the vocabulary
        const double pv = exp((double)xv[k] - r.lse_v), pd = exp((double)xd[k] - r.lse_d);
        rs += fmax(0.0, pv - pd);
        vs += pv;
    }
    rs = block_sum_d(rs, sh_d);
    vs = block_sum_d(vs, sh_d);
    if (threadIdx.x == 0) {
        *rs_out = rs;
        *vs_out = vs;
    }
}

// Stage 2: inverse CDF in vocabulary order with one uniform.  Thread 0 walks the chunk masses to
// the chunk that holds u * Z, the CTA then walks that chunk (prefix over threads, then the
// owning thread over its 16 entries).  If the residual mass is zero (cannot follow a true
// rejection in exact arithmetic) the draw is from pi_v.
struct PickShared {
    double warp[VCHUNK_THREADS / 32];
    double target;
    int chunk, use_res, pick;
};
__device__ __forceinline__ void residual_pick_block(const AcceptIn& in, const RejectInfo& r, int s, const double* __restrict__ rsum,
                                                    const double* __restrict__ vsum, int n_chunks, int* __restrict__ resampled,
                                                    PickShared& sh) {
    double* sh_warp = sh.warp;
    double& sh_target = sh.target;
    int &sh_chunk = sh.chunk, &sh_use_res = sh.use_res, &sh_pick = sh.pick;
    if (threadIdx.x == 0) {
        double Z = 0.0;
        for (int c = 0; c < n_chunks; ++c) Z += rsum[(size_t)s * n_chunks + c];
        const bool use_res = Z > 0.0;
        const double* mass = (use_res ? rsum : vsum) + (size_t)s * n_chunks;
        double total = 0.0;
        for (int c = 0; c < n_chunks; ++c) total += mass[c];
        const double u2 = philox_uniform(in.seed, r.pos, in.seq_stream[s], (unsigned)in.seq_step[s], STREAM_RESAMPLE);
        const double target = u2 * total;
        double before = 0.0;
        int pick_chunk = -1;
        for (int c = 0; c < n_chunks; ++c) {
            if (before + mass[c] > target) {
                pick_chunk = c;
                break;
            }
            before += mass[c];
        }
        sh_chunk = pick_chunk;
        sh_use_res = use_res;
        sh_target = target - before;
        sh_pick = in.V - 1;
    }
    __syncthreads();
    const int chunk = sh_chunk;
    if (chunk >= 0) {
        const bool use_res = sh_use_res != 0;
        const double target = sh_target;
        float xv[VPER], xd[VPER];
        load_chunk_contiguous(in.verify_logits + (size_t)r.verify_row * in.V, in.V, chunk * VCHUNK, threadIdx.x, xv);
        load_chunk_contiguous(in.draft_logits + (size_t)r.draft_row * in.V, in.V, chunk * VCHUNK, threadIdx.x, xd);
        double w[VPER], mine = 0.0;
#pragma unroll
        for (int k = 0; k < VPER; ++k) {
            w[k] = 0.0;
            if (!(xv[k] == -INFINITY && xd[k] == -INFINITY)) {
                const double pv = exp((double)xv[k] - r.lse_v), pd = exp((double)xd[k] - r.lse_d);
                w[k] = use_res ? fmax(0.0, pv - pd) : pv;
            }
            mine += w[k];
        }
        // exclusive prefix over threads in thread order
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        double incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) sh_warp[warp] = incl;
        __syncthreads();
        double before = incl - mine;
        for (int k = 0; k < warp; ++k) before += sh_warp[k];
        if (before <= target && before + mine > target) {
            double c = before;
            int pick = VPER - 1;
#pragma unroll
            for (int k = VPER - 1; k >= 0; --k) {
                // prefix(k) in the same left-to-right order for every k; keep the smallest k that passes
                double upto = before;
#pragma unroll
                for (int j = 0; j < VPER; ++j)
                    if (j <= k) upto += w[j];
                if (upto > target) pick = k;
            }
            (void)c;
            atomicMin(&sh_pick, min(in.V - 1, chunk * VCHUNK + (int)threadIdx.x * VPER + pick));
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) resampled[s] = sh_pick;
}

// ---------------------------------------------------------------------------------------------
// The acceptance step in two launches that wait for nothing: verifier probabilities, ratio test against the Philox
// uniforms and first rejection here, the residual draw in residual_fused_kernel (Algorithm "SampleBlock for S2D2", the
// left-to-right loop and its resampling line).
// Grid (vocabulary chunks, verifier logit rows + sequences).  CTA (chunk, row) computes the chunk statistics of its row
// and takes a ticket of the row's sequence; the CTA that takes the sequence's last ticket (all chunks of all its rows
// are then written) runs the scan for that sequence.  CTAs (0, n_verify_rows + s) serve the sequences that were not
// verified (confidence branch).  row_seq[r] is the sequence of verifier logit row r (-1: none of this call's); tickets
// are zero before and after the launch.  (The residual sums by that one CTA as well made a single launch, and a slow
// one: 300 000 fp64 exponentials on one SM.)
// ---------------------------------------------------------------------------------------------
static __global__ void __launch_bounds__(VCHUNK_THREADS) accept_fused_kernel(AcceptIn in, AcceptOut out, RejectInfo* rej,
                                                                             ChunkStats* __restrict__ chunk_v,
                                                                             const int* __restrict__ row_seq, unsigned* tickets,
                                                                             int n_verify_rows) {
    __shared__ Top2 sh_t[32];
    __shared__ double sh_d[32];
    __shared__ ScanShared sh_scan;
    __shared__ int sh_last;
    const int chunk = blockIdx.x, n_chunks = gridDim.x;
    if ((int)blockIdx.y >= n_verify_rows) {
        const int s = blockIdx.y - n_verify_rows;
        if (chunk == 0 && in.seq_mode && in.seq_mode[s] == 0) accept_scan_block(in, out, rej, s, sh_scan);
        return;
    }
    const int r = blockIdx.y;
    chunk_stats_block(in.verify_logits + (size_t)r * in.V, in.V, chunk, chunk_v + (size_t)r * n_chunks + chunk, sh_t, sh_d);
    const int s = row_seq[r];
    if (s < 0) return;
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned t = atomicAdd(&tickets[s], 1u);
        sh_last = t == (unsigned)(in.seq_len[s] * n_chunks) - 1u;
    }
    __syncthreads();
    if (!sh_last) return;
    if (threadIdx.x == 0) tickets[s] = 0;
    __threadfence();
    accept_scan_block(in, out, rej, s, sh_scan);
}
// The residual draw of the rejected positions as one launch, grid (vocabulary chunks, sequences): every CTA sums its chunk
// of (pi_v - pi_d)_+ in fp64 (the sums are what is expensive, so they stay spread over the GPU), and the CTA that takes
// the sequence's last ticket walks the inverse CDF.
static __global__ void __launch_bounds__(VCHUNK_THREADS) residual_fused_kernel(AcceptIn in, const RejectInfo* __restrict__ rej,
                                                                               double* rsum, double* vsum, unsigned* tickets,
                                                                               int* __restrict__ resampled) {
    __shared__ double sh_d[32];
    __shared__ PickShared sh_pick;
    __shared__ int sh_last;
    const int chunk = blockIdx.x, s = blockIdx.y, n_chunks = gridDim.x;
    const RejectInfo rj = rej[s];
    if (rj.draft_row < 0) return;
    residual_chunk_block(in, rj, chunk, rsum + (size_t)s * n_chunks + chunk, vsum + (size_t)s * n_chunks + chunk, sh_d);
    if (threadIdx.x == 0) {
        __threadfence();
        sh_last = atomicAdd(&tickets[s], 1u) == (unsigned)n_chunks - 1u;
    }
    __syncthreads();
    if (!sh_last) return;
    if (threadIdx.x == 0) tickets[s] = 0;
    __threadfence();
    residual_pick_block(in, rj, s, rsum, vsum, n_chunks, resampled, sh_pick);
}

}  // namespace s2d2
