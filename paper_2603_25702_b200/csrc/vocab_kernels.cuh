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

constexpr int VOCAB_THREADS = 1024;

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

// SampleFromLogits, greedy: one block per logit row.
__global__ void draft_stats_kernel(const float* __restrict__ logits, int V, DraftStatsOut o) {
    __shared__ Top2 sh_t[32];
    __shared__ double sh_d[32];
    int r = blockIdx.x;
    const float* x = logits + (size_t)r * V;
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int i = threadIdx.x; i < V; i += blockDim.x) t = top2_push(t, x[i], i);
    t = block_top2(t, sh_t);
    double mx = (double)t.v1, s = 0.0, sx = 0.0;
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
        double xi = (double)x[i];
        double e = exp(xi - mx);
        s += e;
        sx += e * xi;
    }
    s = block_sum_d(s, sh_d);
    sx = block_sum_d(sx, sh_d);
    if (threadIdx.x == 0) {
        double lse = mx + log(s);
        o.xhat[r] = t.i1;
        o.conf[r] = (float)(1.0 / s);
        o.margin[r] = (float)((1.0 - exp((double)t.v2 - mx)) / s);
        o.entropy[r] = (float)(lse - sx / s);
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
    const double* draft_lse;      // per draft-logit row (may be null: recomputed)
    const int* seq_mode;          // 1: acceptance scan; 0: confidence branch (may be null: all 1)
    const float* conf;            // per draft-logit row, for the confidence branch
    float tau_conf;
    unsigned seed;
    float gamma;
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

__device__ __forceinline__ double row_lse_block(const float* x, int V, double* sh_d, Top2* sh_t) {
    Top2 t{-INFINITY, 0x7fffffff, -INFINITY};
    for (int i = threadIdx.x; i < V; i += blockDim.x) t = top2_push(t, x[i], i);
    t = block_top2(t, sh_t);
    double mx = (double)t.v1, s = 0.0;
    for (int i = threadIdx.x; i < V; i += blockDim.x) s += exp((double)x[i] - mx);
    s = block_sum_d(s, sh_d);
    return mx + log(s);
}

// Reference form of the acceptance step: one block per sequence, rows scanned
// left to right, stopping at the first rejection.
__global__ void accept_block_kernel(AcceptIn in, AcceptOut out) {
    __shared__ Top2 sh_t[32];
    __shared__ double sh_d[32];
    __shared__ double sh_pref[VOCAB_THREADS];
    __shared__ int sh_pick;
    int s = blockIdx.x;
    int L = in.seq_len[s];
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
    int n_acc = 0, first_rej = -1, resampled = -1, near = 0;
    for (int i = 0; i < L; ++i) {
        int dr = in.seq_draft_row0[s] + i;
        const float* xd = in.draft_logits + (size_t)dr * in.V;
        const float* xv = in.verify_logits + (size_t)(in.seq_verify_row0[s] + i) * in.V;
        double lse_v = row_lse_block(xv, in.V, sh_d, sh_t);
        double lse_d = in.draft_lse ? in.draft_lse[dr] : row_lse_block(xd, in.V, sh_d, sh_t);
        int tok = in.xhat[dr];
        double v = exp((double)xv[tok] - lse_v), d = exp((double)xd[tok] - lse_d);
        double ratio = v / d;
        if (in.gamma != 1.f) ratio = pow(ratio, (double)in.gamma);
        double a = fmin(1.0, ratio);
        unsigned pos = (unsigned)(in.seq_pos0[s] + i);
        double u = philox_uniform(in.seed, pos, in.seq_stream[s], (unsigned)in.seq_step[s], STREAM_ACCEPT);
        if (threadIdx.x == 0) {
            out.u[(size_t)s * in.l_cap + i] = (float)u;
            out.a[(size_t)s * in.l_cap + i] = (float)a;
            out.v[(size_t)s * in.l_cap + i] = (float)v;
        }
        if (fabs(u - a) < 1e-4) ++near;
        if (u < a) {
            ++n_acc;
            continue;
        }
        first_rej = i;
        if (in.resample) {
            // residual (pi_v - pi_d)_+ : each thread owns a contiguous slice so that the
            // block prefix over threads is the vocabulary-order CDF
            int per = (in.V + blockDim.x - 1) / blockDim.x;
            int lo = min(in.V, (int)threadIdx.x * per), hi = min(in.V, lo + per);
            double mine = 0.0;
            for (int w = lo; w < hi; ++w) mine += fmax(0.0, exp((double)xv[w] - lse_v) - exp((double)xd[w] - lse_d));
            double Z = block_sum_d(mine, sh_d);
            bool use_residual = Z > 0.0;
            if (!use_residual) {   // unreachable after a true rejection in exact arithmetic
                mine = 0.0;
                for (int w = lo; w < hi; ++w) mine += exp((double)xv[w] - lse_v);
            }
            sh_pref[threadIdx.x] = mine;
            __syncthreads();
            if (threadIdx.x == 0) {
                double run = 0.0;
                for (int t = 0; t < (int)blockDim.x; ++t) {
                    double x = sh_pref[t];
                    sh_pref[t] = run;          // exclusive prefix
                    run += x;
                }
                sh_d[0] = run;
                sh_pick = in.V - 1;
            }
            __syncthreads();
            double total = sh_d[0];
            double u2 = philox_uniform(in.seed, pos, in.seq_stream[s], (unsigned)in.seq_step[s], STREAM_RESAMPLE);
            double target = u2 * total;
            double before = sh_pref[threadIdx.x];
            __syncthreads();
            if (before <= target && before + mine > target) {
                double c = before;
                int pick = hi - 1;
                for (int w = lo; w < hi; ++w) {
                    double wgt = use_residual ? fmax(0.0, exp((double)xv[w] - lse_v) - exp((double)xd[w] - lse_d))
                                              : exp((double)xv[w] - lse_v);
                    c += wgt;
                    if (c > target) {
                        pick = w;
                        break;
                    }
                }
                atomicMin(&sh_pick, pick);
            }
            __syncthreads();
            resampled = sh_pick;
        }
        break;
    }
    if (threadIdx.x == 0) {
        out.n_accepted[s] = n_acc;
        out.first_reject[s] = first_rej;
        out.resampled[s] = resampled;
        out.n_near[s] = near;
    }
}

}  // namespace s2d2
