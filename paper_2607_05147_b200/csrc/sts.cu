// dspark_sts_*: Sequential Temperature Scaling of the confidence head (Section 3.2.1, "Post-hoc
// Calibration").  From left to right, position k receives the temperature of a caller-given 1-D grid that
// minimises the Expected Calibration Error of the cumulative product
//     a_{n,k} = prod_{i<=k} sigmoid(logit(c_{n,i}) / T_i)
// over N held-out blocks, with the temperatures of the earlier positions already fixed.  The label of
// (n, k) is 1 when the draft prefix through k was accepted (accepted_len[n] > k); a block counts at
// position k only if that position was verified (k < verified_len[n]).
//     ECE = (1/N_k) sum_b | sum_{n in b} y_n - sum_{n in b} a_n |,   b = min(n_bins-1, floor(a n_bins)).
//
// All grid points of a position are evaluated in one launch (one CTA column per grid point, the samples
// split over blockIdx.y); per-bin sums of a are kept as exact integers (a * 2^32, truncated), so the
// result does not depend on the order in which threads add.  A small kernel picks the first minimum and
// one more folds the chosen temperature into the running products.  Nothing here is bound by
// bandwidth or arithmetic (N * G sigmoids per position): the point is that calibration runs on the
// device, asynchronously, next to the scheduler that consumes its output.
#include <math.h>

#include "common.cuh"

namespace dspark {

constexpr int kStsThreads = 256;
constexpr int kStsMaxBins = 64;

struct StsAcc {                 // one bin of one (position, grid point)
    unsigned long long sum_a;   // sum of trunc(a * 2^32)
    unsigned int sum_y;         // accepted prefixes
    unsigned int count;         // samples
};

// sigmoid(logit(c) / T); confidences outside (0,1) are clamped to [0,1] (NaN -> 0) and not rescaled
__device__ __forceinline__ float sts_scaled(float c, float inv_T)
{
    if (!(c > 0.f)) return 0.f;
    if (c >= 1.f) return 1.f;
    const float z = logf(c) - log1pf(-c);
    return 1.f / (1.f + expf(-z * inv_T));
}

// grid point g < G: calibrated chain times the candidate scaling; g == G: the raw chain (T = 1 throughout)
__global__ void __launch_bounds__(kStsThreads)
sts_eval_kernel(const float* __restrict__ conf, int N, int gamma, int k, const int32_t* __restrict__ accepted_len,
                const int32_t* __restrict__ verified_len, const float* __restrict__ grid, int G, int n_bins,
                const float* __restrict__ a_cal, const float* __restrict__ a_raw, StsAcc* acc)
{
    __shared__ StsAcc bins[kStsThreads / 32][kStsMaxBins];
    pdl_wait();
    const int g = blockIdx.x, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < (kStsThreads / 32) * kStsMaxBins; i += kStsThreads) {
        StsAcc z = {0ull, 0u, 0u};
        (&bins[0][0])[i] = z;
    }
    __syncthreads();
    const bool raw = g == G;
    const float inv_T = raw ? 1.f : 1.f / grid[g];
    const float* prev = raw ? a_raw : a_cal;
    const int per = (N + gridDim.y - 1) / gridDim.y;
    const int lo = blockIdx.y * per, hi = min(N, lo + per);
    for (int n = lo + threadIdx.x; n < hi; n += kStsThreads) {
        if (verified_len && k >= verified_len[n]) continue;
        const float a = prev[n] * sts_scaled(conf[(size_t)n * gamma + k], inv_T);
        int b = (int)floorf(a * (float)n_bins);
        b = min(max(b, 0), n_bins - 1);
        atomicAdd(&bins[warp][b].sum_a, (unsigned long long)(a * 4294967296.f));
        atomicAdd(&bins[warp][b].count, 1u);
        if (accepted_len[n] > k) atomicAdd(&bins[warp][b].sum_y, 1u);
    }
    __syncthreads();
    StsAcc* out = acc + ((size_t)k * (G + 1) + g) * n_bins;
    for (int b = threadIdx.x; b < n_bins; b += kStsThreads) {
        StsAcc t = {0ull, 0u, 0u};
        for (int w = 0; w < kStsThreads / 32; ++w) {
            t.sum_a += bins[w][b].sum_a; t.sum_y += bins[w][b].sum_y; t.count += bins[w][b].count;
        }
        if (t.count) {
            atomicAdd(&out[b].sum_a, t.sum_a);
            atomicAdd(&out[b].sum_y, t.sum_y);
            atomicAdd(&out[b].count, t.count);
        }
    }
}

// ECE of every grid point, first minimum -> T_k
__global__ void __launch_bounds__(kStsThreads)
sts_pick_kernel(const StsAcc* acc, int k, const float* __restrict__ grid, int G, int n_bins,
                float* out_T, double* ece_before, double* ece_after, double* ece_grid)
{
    __shared__ double s_e[kStsThreads];
    __shared__ int s_g[kStsThreads];
    pdl_wait();
    double best = INFINITY;
    int bg = 0x7fffffff;
    for (int g = threadIdx.x; g <= G; g += kStsThreads) {
        const StsAcc* a = acc + ((size_t)k * (G + 1) + g) * n_bins;
        double e = 0.0;
        unsigned long long cnt = 0;
        for (int b = 0; b < n_bins; ++b) {
            e += fabs((double)a[b].sum_y - (double)a[b].sum_a * (1.0 / 4294967296.0));
            cnt += a[b].count;
        }
        e = cnt ? e / (double)cnt : 0.0;
        if (g == G) { if (ece_before) ece_before[k] = e; continue; }
        // a grid point that is not a positive finite temperature is never chosen (its scaled confidences are
        // meaningless); its entry of the ECE table says so
        const float Tg = grid[g];
        const bool usable = Tg > 0.f && Tg < INFINITY;
        if (ece_grid) ece_grid[(size_t)k * G + g] = usable ? e : NAN;
        if (usable && cnt && e < best) { best = e; bg = g; }          // g ascends within a thread: first minimum
    }
    s_e[threadIdx.x] = best; s_g[threadIdx.x] = bg;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int t = 1; t < kStsThreads; ++t)
            if (s_g[t] != 0x7fffffff && (s_e[t] < best || (s_e[t] == best && s_g[t] < bg))) { best = s_e[t]; bg = s_g[t]; }
        const bool any = bg != 0x7fffffff;                  // nobody verified this position: T = 1
        out_T[k] = any ? grid[bg] : 1.f;
        if (ece_after) ece_after[k] = any ? best : 0.0;
    }
}

// a_cal *= sigmoid(logit(c_k) / T_k), a_raw *= clamp(c_k)
__global__ void __launch_bounds__(kStsThreads)
sts_update_kernel(const float* __restrict__ conf, int N, int gamma, int k, const float* __restrict__ T, float* a_cal, float* a_raw)
{
    pdl_wait();
    const int n = blockIdx.x * kStsThreads + threadIdx.x;
    if (n >= N) return;
    const float c = conf[(size_t)n * gamma + k];
    a_cal[n] *= sts_scaled(c, 1.f / T[k]);
    a_raw[n] *= sts_scaled(c, 1.f);
}

__global__ void __launch_bounds__(kStsThreads) sts_init_kernel(int N, float* a_cal, float* a_raw, StsAcc* acc, size_t n_acc)
{
    pdl_wait();
    const size_t i = (size_t)blockIdx.x * kStsThreads + threadIdx.x;
    if (i < (size_t)N) { a_cal[i] = 1.f; a_raw[i] = 1.f; }
    if (i < n_acc) { StsAcc z = {0ull, 0u, 0u}; acc[i] = z; }
}

__global__ void __launch_bounds__(kStsThreads)
sts_apply_kernel(const float* __restrict__ conf, long long total, int gamma, const float* __restrict__ T, float* out)
{
    pdl_wait();
    const long long i = (long long)blockIdx.x * kStsThreads + threadIdx.x;
    if (i < total) out[i] = sts_scaled(conf[i], 1.f / T[i % gamma]);
}

struct StsWs { size_t a_cal, a_raw, acc, n_acc, total; };
static StsWs sts_layout(int N, int gamma, int G, int n_bins)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    StsWs w;
    size_t o = 0;
    w.a_cal = o; o += up((size_t)N * 4);
    w.a_raw = o; o += up((size_t)N * 4);
    w.n_acc = (size_t)gamma * (G + 1) * n_bins;
    w.acc = o;   o += up(w.n_acc * sizeof(StsAcc));
    w.total = o;
    return w;
}

}  // namespace dspark

using namespace dspark;

extern "C" {

size_t dspark_sts_workspace_bytes(int N, int gamma, int G, int n_bins)
{
    if (N < 1 || gamma < 1 || G < 1 || n_bins < 1 || n_bins > kStsMaxBins) return 0;
    return sts_layout(N, gamma, G, n_bins).total;
}

int dspark_sts_calibrate(const float* conf, int N, int gamma, const int32_t* accepted_len, const int32_t* verified_len,
                         const float* grid, int G, int n_bins, float* out_T, double* out_ece_before,
                         double* out_ece_after, double* out_ece_grid, void* workspace, size_t workspace_bytes, void* stream)
{
    if (!conf || !accepted_len || !grid || !out_T) return DSPARK_ERR_INVALID_ARG;
    if (N < 1 || gamma < 1 || G < 1 || n_bins < 1) return DSPARK_ERR_INVALID_ARG;
    if (n_bins > kStsMaxBins) return DSPARK_ERR_SHAPE;
    const StsWs w = sts_layout(N, gamma, G, n_bins);
    if (!workspace || workspace_bytes < w.total) return DSPARK_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return DSPARK_ERR_ALIGNMENT;
    unsigned char* ws = (unsigned char*)workspace;
    float* a_cal = (float*)(ws + w.a_cal);
    float* a_raw = (float*)(ws + w.a_raw);
    StsAcc* acc = (StsAcc*)(ws + w.acc);
    cudaStream_t s = (cudaStream_t)stream;
    const size_t n_init = (size_t)N > w.n_acc ? (size_t)N : w.n_acc;
    launch_pdl(sts_init_kernel, dim3((unsigned)((n_init + kStsThreads - 1) / kStsThreads)), dim3(kStsThreads), 0, s, N, a_cal,
               a_raw, acc, w.n_acc);
    int slices = (N + 16 * kStsThreads - 1) / (16 * kStsThreads);      // about 16 samples per thread
    if (slices > 64) slices = 64;
    for (int k = 0; k < gamma; ++k) {
        launch_pdl(sts_eval_kernel, dim3(G + 1, slices), dim3(kStsThreads), 0, s, conf, N, gamma, k, accepted_len,
                   verified_len, grid, G, n_bins, (const float*)a_cal, (const float*)a_raw, acc);
        launch_pdl(sts_pick_kernel, dim3(1), dim3(kStsThreads), 0, s, (const StsAcc*)acc, k, grid, G, n_bins, out_T,
                   out_ece_before, out_ece_after, out_ece_grid);
        launch_pdl(sts_update_kernel, dim3((N + kStsThreads - 1) / kStsThreads), dim3(kStsThreads), 0, s, conf, N, gamma, k,
                   (const float*)out_T, a_cal, a_raw);
    }
    return launch_status();
}

int dspark_sts_apply(const float* conf, int N, int gamma, const float* T, float* out, void* stream)
{
    if (!conf || !T || !out || N < 1 || gamma < 1) return DSPARK_ERR_INVALID_ARG;
    const long long total = (long long)N * gamma;
    launch_pdl(sts_apply_kernel, dim3((unsigned)((total + kStsThreads - 1) / kStsThreads)), dim3(kStsThreads), 0,
               (cudaStream_t)stream, conf, total, gamma, T, out);
    return launch_status();
}

}  // extern "C"
