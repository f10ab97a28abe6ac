// GEMM dispatch of the forward pass: bf16 models go to the tcgen05 weight-streaming
// kernel (gemm_tc.cuh); the fp32 model, shapes the tensor-core kernel does not take
// (K not a multiple of 64) and contexts created with use_tensor_cores = 0 go to the
// SIMT kernel.
#include "gemm.h"

#include <cuda.h>

#include <atomic>
#include <map>
#include <mutex>
#include <tuple>

#include "context.h"
#include "gemm_tc.cuh"
#include "gemm_wide.cuh"
#include "kernels_simt.cuh"

using namespace s2d2;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct GemmState {
    EncodeTiledFn encode = nullptr;
    bool tc_ok = false;
    int n_sms = 148;
    float* ws = nullptr;
    size_t ws_floats = 0;
    unsigned* tickets = nullptr;
    size_t n_tickets = 0;
    int max_smem = 0;
    std::map<std::tuple<const void*, int, int, int>, CUtensorMap> maps;   // (ptr, rows, K, box_rows)
};

GemmState* state(s2d2_ctx* c) { return (GemmState*)c->gemm_state; }

// Tensor map of a row-major bf16 matrix [rows, K]: boxes of box_rows x 64 elements, 128-byte swizzle,
// zero fill outside the matrix.
const CUtensorMap* get_map(s2d2_ctx* c, const void* ptr, int rows, int K, int box_rows) {
    GemmState* g = state(c);
    auto key = std::make_tuple(ptr, rows, K, box_rows);
    auto it = g->maps.find(key);
    if (it != g->maps.end()) return &it->second;
    CUtensorMap m;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)tc::BLOCK_K, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        c->err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
        return nullptr;
    }
    return &(g->maps[key] = m);
}

template <typename TW, typename TX>
void gemm_simt(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale,
               int accumulate) {
    constexpr int ROWS = 8;
    dim3 grid((N + 3) / 4, (M + ROWS - 1) / ROWS);
    gemm_simt_kernel<TW, TX, ROWS><<<grid, 128, 0, c->stream>>>((const TX*)X, (const TW*)W, Y, M, N, K, ldy, scale, accumulate);
    c->cnt.n_kernel_launches++;
}

// Wide passes (more than 64 token rows): gemm_wide_kernel.  One CTA per SM (its stage ring and its epilogue
// buffers take most of the shared memory); the host picks weight sub-tiles per CTA and K splits so that the
// CTAs cover the SMs: a GEMM with few weight tiles (QKV, O, down) would otherwise run on a third of the machine.
// Cost model in microseconds: a k-block takes the slowest of the fill of one SM's shared memory (80 KB/us), the fill of
// all streaming SMs together (10.5 MB/us) and its MMAs; a CTA adds WIDE_CTA_US of set-up and epilogue; a split adds the
// round trip of its partial sub-tiles through the workspace.
constexpr double WIDE_CTA_US = 7.0, WIDE_SPLIT_US = 3.0;
int gemm_wide(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale,
              int accumulate, const void* X_lo) {
    GemmState* g = state(c);
    tc::GemmParams p;
    p.Y = Y;
    p.M = M;
    p.N = N;
    p.K = K;
    p.ldy = ldy;
    p.scale = scale;
    p.accumulate = accumulate;
    p.kb_total = K / tc::BLOCK_K;
    p.hilo = X_lo != nullptr;
    const int t_max = 128;                        // an epilogue buffer is [T][128] fp32; three of them fit beside nothing else
    p.m_tiles = (M + t_max - 1) / t_max;
    const int per = (M + p.m_tiles - 1) / p.m_tiles;
    p.T = std::min(t_max, (per + 15) / 16 * 16);
    p.m_tiles = (M + p.T - 1) / p.T;
    const int TN = p.hilo ? 2 * p.T : p.T;
    const size_t smem_max = 225 * 1024;
    int best = 0, best_wt = 0, best_stages = 0;
    double best_cost = 1e30;
    for (int wt = 1; wt <= 2; ++wt) {
        if (wt == 2 && (2 * TN > 512 || N < 2 * tc::BLOCK_N)) break;
        const size_t sb = tc::stage_bytes(TN, wt);
        const int tiles = (N + wt * tc::BLOCK_N - 1) / (wt * tc::BLOCK_N) * p.m_tiles;
        const double kb_kb = sb / 1024.0, mma_us = wt * TN * (0.276 / 256.0);
        for (int s = 1; s <= 16 && (s == 1 || s <= p.kb_total / 4); ++s) {
            int stages = (int)std::min<size_t>(8, (200 * 1024) / sb);
            stages = std::min(stages, (p.kb_total + s - 1) / s);
            if (stages < 2 && p.kb_total > 1) break;
            stages = std::max(stages, 1);
            if (tc::wide_smem_bytes(p.T, TN, stages, wt, s) > smem_max) continue;
            if (s > 1 && ((size_t)tiles * s * wt * p.T * tc::BLOCK_N > g->ws_floats || (size_t)tiles > g->n_tickets)) break;
            const int ctas = tiles * s, waves = (ctas + g->n_sms - 1) / g->n_sms, streaming = std::min(ctas, g->n_sms);
            const double kb_us = std::max(std::max(kb_kb / 80.0, kb_kb * streaming / 10500.0), mma_us);
            const double sub_kb = p.T * 0.5;
            const double cost = waves * ((double)((p.kb_total + s - 1) / s) * kb_us + WIDE_CTA_US + wt * sub_kb / 80.0) +
                                (s > 1 ? WIDE_SPLIT_US + wt * (s + 1) * sub_kb / 80.0 : 0.0);
            if (cost < best_cost - 1e-9) {
                best_cost = cost;
                best = s;
                best_wt = wt;
                best_stages = stages;
            }
        }
    }
    if (!best) return -1;
    p.splits = best;
    p.wtiles = best_wt;
    p.stages = best_stages;
    p.n_tiles = (N + best_wt * tc::BLOCK_N - 1) / (best_wt * tc::BLOCK_N);
    p.ws = g->ws;
    p.tickets = g->tickets;
    p.status = c->d_status;
    p.evict_first = 0;
    const CUtensorMap* mw = get_map(c, W, N, K, tc::BLOCK_N);
    const CUtensorMap* mx = get_map(c, X, M, K, p.T);
    const CUtensorMap* mx_lo = p.hilo ? get_map(c, X_lo, M, K, p.T) : mx;
    if (!mw || !mx || !mx_lo) return S2D2_ERR_CUDA;
    const int grid = p.n_tiles * p.m_tiles * p.splits;
    tc::gemm_wide_kernel<<<grid, tc::THREADS, tc::wide_smem_bytes(p.T, TN, p.stages, p.wtiles, p.splits), c->stream>>>(*mw, *mx, *mx_lo, p);
    c->cnt.n_kernel_launches++;
    return S2D2_OK;
}

// gate/up GEMM of a wide pass with SwiGLU in its epilogue (see GemmParams::swiglu): two sub-tiles per CTA, no K split
// (a layer's gate/up has weight tiles enough for every SM).
int gemm_wide_swiglu(s2d2_ctx* c, const void* X, const void* X_lo, const void* W, int M, int f, int K, void* act, void* act_lo) {
    tc::GemmParams p;
    p.Y = nullptr;
    p.M = M;
    p.N = 2 * f;
    p.K = K;
    p.ldy = 0;
    p.scale = 1.f;
    p.accumulate = 0;
    p.kb_total = K / tc::BLOCK_K;
    p.hilo = X_lo != nullptr;
    p.m_tiles = (M + 127) / 128;
    const int per = (M + p.m_tiles - 1) / p.m_tiles;
    p.T = std::min(128, (per + 15) / 16 * 16);
    p.m_tiles = (M + p.T - 1) / p.T;
    const int TN = p.hilo ? 2 * p.T : p.T;
    p.wtiles = 2;
    p.splits = 1;
    p.stages = (int)std::min<size_t>(8, (200 * 1024) / tc::stage_bytes(TN, 2));
    p.stages = std::max(1, std::min(p.stages, p.kb_total));
    p.n_tiles = f / tc::BLOCK_N;
    p.ws = nullptr;
    p.tickets = nullptr;
    p.status = c->d_status;
    p.evict_first = 0;
    p.swiglu = 1;
    p.f = f;
    p.act = (bf16*)act;
    p.act_lo = (bf16*)act_lo;
    const CUtensorMap* mw = get_map(c, W, 2 * f, K, tc::BLOCK_N);
    const CUtensorMap* mx = get_map(c, X, M, K, p.T);
    const CUtensorMap* mx_lo = p.hilo ? get_map(c, X_lo, M, K, p.T) : mx;
    if (!mw || !mx || !mx_lo) return S2D2_ERR_CUDA;
    tc::gemm_wide_kernel<<<p.n_tiles * p.m_tiles, tc::THREADS, tc::wide_smem_bytes(p.T, TN, p.stages, 2, 1), c->stream>>>(*mw, *mx, *mx_lo, p);
    c->cnt.n_kernel_launches++;
    return S2D2_OK;
}

int gemm_tc(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale,
            int accumulate, const void* X_lo) {
    GemmState* g = state(c);
    // bulk copies want 16-byte rows: Y, its leading dimension and the width of the matrix in whole float4
    if (M > 64 && ldy % 4 == 0 && N % 4 == 0 && ((uintptr_t)Y & 15) == 0) {
        int rc = gemm_wide(c, X, W, Y, M, N, K, ldy, scale, accumulate, X_lo);
        if (rc >= 0) return rc;
    }
    tc::GemmParams p;
    p.Y = Y;
    p.M = M;
    p.N = N;
    p.K = K;
    p.ldy = ldy;
    p.scale = scale;
    p.accumulate = accumulate;
    p.kb_total = K / tc::BLOCK_K;
    p.hilo = X_lo != nullptr;
    const int t_max = p.hilo ? 128 : 256;       // the MMA takes up to 256 token rows, the low halves count
    p.m_tiles = (M + t_max - 1) / t_max;
    int per = (M + p.m_tiles - 1) / p.m_tiles;
    p.T = std::min(t_max, (per + 15) / 16 * 16);
    p.m_tiles = (M + p.T - 1) / p.T;
    const int TN = p.hilo ? 2 * p.T : p.T;
    // Weight sub-tiles per CTA (1 or 2) and K splits, by a time model fitted to measurements on the 8B-class
    // shapes (microseconds, KB).  A k-block (weight sub-tiles + token block) takes the slowest of: what one SM
    // takes into shared memory (80 KB/us, shared by the CTAs resident on it), the same for all busy SMs together
    // (10.5 MB/us), the weights' part from HBM (50 KB/us per SM, 6.5 MB/us in all).  A wave of CTAs adds about
    // 10 us of set-up and epilogue (5 us where two CTAs per SM overlap them); a K split adds the partial tile's
    // round trip through the workspace (0.22 us per token row and sub-tile).
    int best = 1, best_wt = 1;
    double best_cost = 1e30;
    for (int wt = 1; wt <= 2; ++wt) {
        if (wt == 2 && (2 * TN > 512 || N < 2 * tc::BLOCK_N)) break;       // two accumulators of TN columns in tensor memory
        const bool two = TN <= 64 && wt == 1;                               // two CTAs per SM while the stage is small
        const size_t budget = two ? 100 * 1024 : 200 * 1024;
        if ((budget - 1280) / tc::stage_bytes(TN, wt) < 2) break;
        const int slots = g->n_sms * (two ? 2 : 1);
        const int tiles = (N + wt * tc::BLOCK_N - 1) / (wt * tc::BLOCK_N) * p.m_tiles;
        const double w_kb = wt * 16.0, kb_bytes = w_kb + TN * 0.125;       // KB per k-block
        for (int s = 1; s <= 16 && s <= p.kb_total / 2 + (p.kb_total < 2 ? 1 : 0); ++s) {
            if ((size_t)tiles * s * p.T * tc::BLOCK_N * wt > g->ws_floats && s > 1) break;
            if ((size_t)tiles > g->n_tickets && s > 1) break;
            const int ctas = tiles * s;
            const int waves = (ctas + slots - 1) / slots;
            const int streaming = std::min(ctas, slots);                    // CTAs streaming at once
            const int share = (two && ctas > g->n_sms) ? 2 : 1;           // of them on one SM
            const double kb_us = std::max(std::max(kb_bytes * share / 80.0, kb_bytes * streaming / 10500.0),
                                          std::max(w_kb * share / 50.0, w_kb * streaming / 6500.0));
            const double cost = waves * ((double)((p.kb_total + s - 1) / s) * kb_us + (two ? 5.0 : 10.0)) +
                                (s > 1 ? 2.0 + 0.22 * p.T * wt : 0.0);
            if (cost < best_cost - 1e-9) {
                best_cost = cost;
                best = s;
                best_wt = wt;
            }
        }
    }
    p.splits = best;
    p.wtiles = best_wt;
    p.n_tiles = (N + best_wt * tc::BLOCK_N - 1) / (best_wt * tc::BLOCK_N);
    const int tiles = p.n_tiles * p.m_tiles;
    {
        const bool two = TN <= 64 && best_wt == 1;
        const size_t budget = two ? 100 * 1024 : 200 * 1024;
        p.stages = (int)std::min<size_t>(8, (budget - 1280) / tc::stage_bytes(TN, best_wt));
        p.stages = std::max(2, std::min(p.stages, p.kb_total));
    }
    p.ws = g->ws;
    p.tickets = g->tickets;
    p.status = c->d_status;
    p.evict_first = (M <= 64);
    const CUtensorMap* mw = get_map(c, W, N, K, tc::BLOCK_N);
    const CUtensorMap* mx = get_map(c, X, M, K, p.T);
    const CUtensorMap* mx_lo = p.hilo ? get_map(c, X_lo, M, K, p.T) : mx;
    if (!mw || !mx || !mx_lo) return S2D2_ERR_CUDA;
    size_t smem = tc::smem_bytes(TN, p.stages, p.wtiles);
    int grid = tiles * p.splits;
    tc::gemm_tc_kernel<<<grid, tc::THREADS, smem, c->stream>>>(*mw, *mx, *mx_lo, p);
    c->cnt.n_kernel_launches++;
    return S2D2_OK;
}

}  // namespace

int gemm_init(s2d2_ctx* c) {
    GemmState* g = new GemmState();
    c->gemm_state = g;
    if (c->m.dtype != S2D2_DTYPE_BF16 || !c->dc.use_tensor_cores) return S2D2_OK;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, c->device) != cudaSuccess) return S2D2_ERR_CUDA;
    g->n_sms = prop.multiProcessorCount;
    if (prop.major != 10) {
        c->err = "the tensor-core kernels are built for sm_100a only";
        return S2D2_ERR_UNSUPPORTED;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) {
        c->err = "cuTensorMapEncodeTiled not available";
        return S2D2_ERR_CUDA;
    }
    g->encode = (EncodeTiledFn)fn;
    g->ws_floats = (size_t)16 << 20;          // 64 MiB of split-K partial tiles
    g->n_tickets = 1 << 16;
    if (cudaMalloc((void**)&g->ws, g->ws_floats * 4) != cudaSuccess) return S2D2_ERR_CUDA;
    if (cudaMalloc((void**)&g->tickets, g->n_tickets * 4) != cudaSuccess) return S2D2_ERR_CUDA;
    if (cudaMemset(g->tickets, 0, g->n_tickets * 4) != cudaSuccess) return S2D2_ERR_CUDA;
    if (cudaFuncSetAttribute(tc::gemm_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess ||
        cudaFuncSetAttribute(tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess) {
        c->err = "cannot raise the dynamic shared memory limit";
        return S2D2_ERR_CUDA;
    }
    g->tc_ok = true;
    return S2D2_OK;
}

void gemm_destroy(s2d2_ctx* c) {
    for (cudaEvent_t e : c->prof_events) cudaEventDestroy(e);
    c->prof_events.clear();
    GemmState* g = state(c);
    if (!g) return;
    if (g->ws) cudaFree(g->ws);
    if (g->tickets) cudaFree(g->tickets);
    delete g;
    c->gemm_state = nullptr;
}

bool gemm_tc_available(s2d2_ctx* c) { return state(c) && state(c)->tc_ok; }

int gemm_encode_map(s2d2_ctx* c, void* out, const void* ptr, unsigned long long rows, int cols, int box_rows) {
    GemmState* g = state(c);
    if (!g || !g->encode) return -1;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g->encode((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : (int)r;
}

int gemm_encode_map3(s2d2_ctx* c, void* out, const void* ptr, int cols, int mid, unsigned long long rows, int box_mid, int box_rows) {
    GemmState* g = state(c);
    if (!g || !g->encode) return -1;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)mid, (cuuint64_t)rows};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * (cuuint64_t)mid};
    cuuint32_t box[3] = {64u, (cuuint32_t)box_mid, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g->encode((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : (int)r;
}

void gemm_forget(s2d2_ctx* c, const void* ptr) {
    GemmState* g = state(c);
    if (!g) return;
    for (auto it = g->maps.begin(); it != g->maps.end();)
        it = (std::get<0>(it->first) == ptr) ? g->maps.erase(it) : std::next(it);
}

void gemm_prof_begin(s2d2_ctx* c) {
    if (!c->profiling) return;
    if (c->prof_used + 2 > c->prof_events.size()) {
        for (int i = 0; i < 512; ++i) {
            cudaEvent_t e;
            cudaEventCreate(&e);
            c->prof_events.push_back(e);
        }
    }
    cudaEventRecord(c->prof_events[c->prof_used], c->stream);
}
void gemm_prof_end(s2d2_ctx* c, double bytes) {
    if (!c->profiling) return;
    cudaEventRecord(c->prof_events[c->prof_used + 1], c->stream);
    c->prof_used += 2;
    c->prof_bytes += bytes;
    c->prof_launches++;
}
int gemm_prof_collect(s2d2_ctx* c) {
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return S2D2_ERR_CUDA;
    for (size_t i = 0; i + 1 < c->prof_used; i += 2) {
        float ms = 0;
        cudaEventElapsedTime(&ms, c->prof_events[i], c->prof_events[i + 1]);
        c->prof_ms_done += ms;
    }
    c->prof_used = 0;
    return S2D2_OK;
}

int gemm(s2d2_ctx* c, const void* X, const void* W, float* Y, int M, int N, int K, int ldy, float scale, int accumulate,
         const void* X_lo) {
    size_t es = c->m.dtype == S2D2_DTYPE_F32 ? 4 : 2;
    gemm_prof_begin(c);
    struct End {
        s2d2_ctx* c;
        double b;
        ~End() { gemm_prof_end(c, b); }
    } end{c, (double)N * K * es + (double)M * K * es * (X_lo ? 2 : 1) + (double)M * N * 4 * (accumulate ? 2 : 1)};
    if (c->m.dtype == S2D2_DTYPE_F32) {
        gemm_simt<float, float>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
        return S2D2_OK;
    }
    if (state(c)->tc_ok && K % tc::BLOCK_K == 0) return gemm_tc(c, X, W, Y, M, N, K, ldy, scale, accumulate, X_lo);
    gemm_simt<bf16, bf16>(c, X, W, Y, M, N, K, ldy, scale, accumulate);
    if (X_lo) gemm_simt<bf16, bf16>(c, X_lo, W, Y, M, N, K, ldy, scale, 1);
    return S2D2_OK;
}

int gemm_swiglu(s2d2_ctx* c, const void* X, const void* X_lo, const void* W, int M, int f, int K, void* act, void* act_lo) {
    if (c->m.dtype != S2D2_DTYPE_BF16 || !state(c)->tc_ok || M <= 64 || K % tc::BLOCK_K || f % tc::BLOCK_N || !act_lo) return -1;
    gemm_prof_begin(c);
    int rc = gemm_wide_swiglu(c, X, X_lo, W, M, f, K, act, act_lo);
    gemm_prof_end(c, 2.0 * f * K * 2 + (double)M * K * 2 * (X_lo ? 2 : 1) + (double)M * f * 4);
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Allocation-free GEMM entry (see s2d2_gemm_bf16_noalloc in the header).
//
// The scratch of the split-K kernel lives in file-scope device arrays.  In host code the
// array names below are only handles: the device addresses come from cudaGetSymbolAddress,
// looked up once per device with that device current, and are what the kernel receives.
// ---------------------------------------------------------------------------------------------
namespace {
constexpr size_t NOALLOC_WS_FLOATS = S2D2_NOALLOC_WS_BYTES / 4;
constexpr int NOALLOC_TICKETS = 4096;
constexpr int NOALLOC_MAX_DEVICES = 64;
static __device__ __align__(256) float g_noalloc_ws[NOALLOC_WS_FLOATS];
static __device__ __align__(256) unsigned g_noalloc_tickets[NOALLOC_TICKETS];
static __device__ __align__(256) int g_noalloc_status[4];

struct NoallocDevice {
    std::atomic<bool> ready{false};
    float* ws = nullptr;
    unsigned* tickets = nullptr;
    int* status = nullptr;
    int n_sms = 0;
};
NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
EncodeTiledFn g_noalloc_encode = nullptr;
std::mutex g_noalloc_setup;      // first calls from several host threads take their turn in the one-time set-up
thread_local char g_noalloc_err[256] = "";

int noalloc_fail(int code, const char* msg, cudaError_t e = cudaSuccess) {
    if (e != cudaSuccess) snprintf(g_noalloc_err, sizeof(g_noalloc_err), "%s: %s", msg, cudaGetErrorString(e));
    else snprintf(g_noalloc_err, sizeof(g_noalloc_err), "%s", msg);
    return code;
}

int noalloc_map(CUtensorMap* m, const void* ptr, int rows, int K, int box_rows) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    cuuint32_t box[2] = {(cuuint32_t)tc::BLOCK_K, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = g_noalloc_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : (int)r;
}
}  // namespace

void gemm_reset_tickets(s2d2_ctx* c) {
    GemmState* g = (GemmState*)c->gemm_state;
    if (g && g->tickets) cudaMemsetAsync(g->tickets, 0, g->n_tickets * 4, c->stream);
}

extern "C" const char* s2d2_noalloc_last_error(void) { return g_noalloc_err; }

extern "C" int s2d2_gemm_bf16_noalloc(const void* d_x, const void* d_w, float* d_y, int32_t M, int32_t N, int32_t K,
                                      void* cuda_stream) {
    g_noalloc_err[0] = 0;
    if (!d_x || !d_w || !d_y) return noalloc_fail(S2D2_ERR_INVALID, "null pointer");
    if (M < 1 || M > 256) return noalloc_fail(S2D2_ERR_INVALID, "M must be in 1..256");
    if (N < 1 || N > (1 << 20)) return noalloc_fail(S2D2_ERR_INVALID, "N must be in 1..1048576");
    if (K < 64 || K > 65536 || K % 64) return noalloc_fail(S2D2_ERR_INVALID, "K must be a multiple of 64 in 64..65536");
    if (((uintptr_t)d_x | (uintptr_t)d_w | (uintptr_t)d_y) & 15) return noalloc_fail(S2D2_ERR_INVALID, "pointers must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return noalloc_fail(S2D2_ERR_CUDA, "cudaGetDevice", e);
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return noalloc_fail(S2D2_ERR_UNSUPPORTED, "device index too large");
    NoallocDevice& nd = g_noalloc_dev[dev];
    if (!nd.ready.load(std::memory_order_acquire)) {
        // one-time set-up for this device (do this before any stream capture); host threads are serialised here
        std::lock_guard<std::mutex> lock(g_noalloc_setup);
        if (!nd.ready.load(std::memory_order_relaxed)) {
        int major = 0;
        if ((e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaDeviceGetAttribute", e);
        if (major != 10) return noalloc_fail(S2D2_ERR_UNSUPPORTED, "built for sm_100a only");
        if ((e = cudaDeviceGetAttribute(&nd.n_sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaDeviceGetAttribute", e);
        if (!g_noalloc_encode) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult q;
            if ((e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q)) != cudaSuccess || !fn)
                return noalloc_fail(S2D2_ERR_CUDA, "cuTensorMapEncodeTiled not available", e);
            g_noalloc_encode = (EncodeTiledFn)fn;
        }
        if ((e = cudaGetSymbolAddress((void**)&nd.ws, g_noalloc_ws)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaGetSymbolAddress(ws)", e);
        if ((e = cudaGetSymbolAddress((void**)&nd.tickets, g_noalloc_tickets)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaGetSymbolAddress(tickets)", e);
        if ((e = cudaGetSymbolAddress((void**)&nd.status, g_noalloc_status)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaGetSymbolAddress(status)", e);
        if ((e = cudaFuncSetAttribute(tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024)) != cudaSuccess)
            return noalloc_fail(S2D2_ERR_CUDA, "cudaFuncSetAttribute", e);
        nd.ready.store(true, std::memory_order_release);
        }
    }
    tc::GemmParams p;
    p.Y = d_y;
    p.M = M;
    p.N = N;
    p.K = K;
    p.ldy = N;
    p.scale = 1.f;
    p.accumulate = 0;
    p.kb_total = K / tc::BLOCK_K;
    p.n_tiles = (N + tc::BLOCK_N - 1) / tc::BLOCK_N;
    p.T = (M + 15) / 16 * 16;
    p.m_tiles = 1;
    bool two = p.T <= 64;
    size_t budget = two ? 100 * 1024 : 200 * 1024;
    p.stages = (int)std::min<size_t>(8, (budget - 1280) / tc::stage_bytes(p.T));
    p.stages = std::max(2, std::min(p.stages, p.kb_total));
    int slots = nd.n_sms * (two ? 2 : 1);
    int best = 1;
    double best_cost = 1e30;
    for (int s = 1; s <= 16 && s <= std::max(1, p.kb_total / 2); ++s) {
        // the partial tiles and the ticket counters must fit the fixed scratch
        if (s > 1 && ((size_t)p.n_tiles * s * p.T * tc::BLOCK_N > NOALLOC_WS_FLOATS || p.n_tiles > NOALLOC_TICKETS)) break;
        int waves = (p.n_tiles * s + slots - 1) / slots;
        double cost = waves * ((double)(p.kb_total + s - 1) / s + 6.0) + (s > 1 ? 2.0 : 0.0);
        if (cost < best_cost - 1e-9) {
            best_cost = cost;
            best = s;
        }
    }
    p.splits = best;
    p.ws = nd.ws;
    p.tickets = nd.tickets;
    p.status = nd.status;
    p.evict_first = 0;
    p.hilo = 0;
    p.wtiles = 1;
    CUtensorMap mw, mx;
    if (noalloc_map(&mw, d_w, N, K, tc::BLOCK_N) || noalloc_map(&mx, d_x, M, K, p.T))
        return noalloc_fail(S2D2_ERR_CUDA, "cuTensorMapEncodeTiled failed");
    // the scratch keeps whatever the previous call left: counters and status start from zero
    if ((e = cudaMemsetAsync(nd.tickets, 0, NOALLOC_TICKETS * sizeof(unsigned), st)) != cudaSuccess)
        return noalloc_fail(S2D2_ERR_CUDA, "cudaMemsetAsync", e);
    if ((e = cudaMemsetAsync(nd.status, 0, sizeof(int), st)) != cudaSuccess)
        return noalloc_fail(S2D2_ERR_CUDA, "cudaMemsetAsync", e);
    tc::gemm_tc_kernel<<<p.n_tiles * p.splits, tc::THREADS, tc::smem_bytes(p.T, p.stages), st>>>(mw, mx, mx, p);
    if ((e = cudaGetLastError()) != cudaSuccess) return noalloc_fail(S2D2_ERR_CUDA, "kernel launch", e);
    int status = 0;
    if ((e = cudaMemcpyAsync(&status, nd.status, sizeof(int), cudaMemcpyDeviceToHost, st)) != cudaSuccess)
        return noalloc_fail(S2D2_ERR_CUDA, "cudaMemcpyAsync", e);
    if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return noalloc_fail(S2D2_ERR_CUDA, "cudaStreamSynchronize", e);
    if (status != 0) return noalloc_fail(S2D2_ERR_TIMEOUT, "a bounded wait inside the kernel ran out");
    return S2D2_OK;
}
