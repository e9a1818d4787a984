// Host-side objects of the C ABI: the engine throughput profile, the per-kernel
// event timer, status strings.
#include <cstdio>
#include <cstdlib>
#include <new>
#include <vector>

#include "common.cuh"

struct dspark_profile {
    double* d_table;
    int max_tokens;
    int device;
};

struct dspark_ktimer {
    int capacity;
    int used;
    std::vector<cudaEvent_t> start, stop;
    std::vector<int> kernel_id;
};

namespace dspark {

static dspark_ktimer* g_timer = nullptr;

KernelTimerScope::KernelTimerScope(int kernel_id, cudaStream_t s) : slot(-1), stream(s)
{
    dspark_ktimer* t = g_timer;
    if (t && t->used < t->capacity) {
        slot = t->used++;
        t->kernel_id[slot] = kernel_id;
        cudaEventRecord(t->start[slot], stream);
    }
}
KernelTimerScope::~KernelTimerScope()
{
    if (slot >= 0 && g_timer) cudaEventRecord(g_timer->stop[slot], stream);
}

int launch_status()
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        fprintf(stderr, "dspark: CUDA launch failed: %s\n", cudaGetErrorString(e));
        return DSPARK_ERR_CUDA;
    }
    return DSPARK_OK;
}

}  // namespace dspark

extern "C" {

// SPS table: piecewise linear between breakpoints, constant outside (Section 3.2.2, cost table).
int dspark_profile_create(const int32_t* bp_tokens, const double* bp_sps, int n_bp, int max_tokens,
                          dspark_profile_t** out)
{
    if (!bp_tokens || !bp_sps || !out || n_bp < 1 || max_tokens < 1) return DSPARK_ERR_INVALID_ARG;
    for (int k = 1; k < n_bp; ++k)
        if (bp_tokens[k] <= bp_tokens[k - 1]) return DSPARK_ERR_INVALID_ARG;
    std::vector<double> tab((size_t)max_tokens + 1);
    int seg = 0;
    for (int B = 0; B <= max_tokens; ++B) {
        if (B <= bp_tokens[0]) { tab[B] = bp_sps[0]; continue; }
        if (B >= bp_tokens[n_bp - 1]) { tab[B] = bp_sps[n_bp - 1]; continue; }
        while (B >= bp_tokens[seg + 1]) ++seg;
        volatile double frac = (double)(B - bp_tokens[seg]) / (double)(bp_tokens[seg + 1] - bp_tokens[seg]);
        volatile double rise = (bp_sps[seg + 1] - bp_sps[seg]) * frac;   // rounded product, then rounded sum
        tab[B] = bp_sps[seg] + rise;
    }
    dspark_profile* p = new (std::nothrow) dspark_profile;
    if (!p) return DSPARK_ERR_CUDA;
    p->max_tokens = max_tokens;
    p->d_table = nullptr;
    if (cudaGetDevice(&p->device) != cudaSuccess ||
        cudaMalloc(&p->d_table, tab.size() * sizeof(double)) != cudaSuccess ||
        cudaMemcpy(p->d_table, tab.data(), tab.size() * sizeof(double), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        if (p->d_table) cudaFree(p->d_table);
        delete p;
        return DSPARK_ERR_CUDA;
    }
    *out = p;
    return DSPARK_OK;
}

int dspark_profile_destroy(dspark_profile_t* p)
{
    if (!p) return DSPARK_ERR_INVALID_ARG;
    cudaFree(p->d_table);
    delete p;
    return DSPARK_OK;
}

const double* dspark_profile_table(const dspark_profile_t* p, int* max_tokens)
{
    if (!p) return nullptr;
    if (max_tokens) *max_tokens = p->max_tokens;
    return p->d_table;
}

void dspark_uniforms(uint64_t seed, uint32_t request, uint32_t position, float* u_accept, float* u_resample)
{
    float a, b;
    dspark::philox_uniforms(seed, request, position, a, b);
    if (u_accept) *u_accept = a;
    if (u_resample) *u_resample = b;
}

int dspark_ktimer_create(int capacity, dspark_ktimer_t** out)
{
    if (!out || capacity < 1) return DSPARK_ERR_INVALID_ARG;
    dspark_ktimer* t = new (std::nothrow) dspark_ktimer;
    if (!t) return DSPARK_ERR_CUDA;
    t->capacity = capacity;
    t->used = 0;
    t->start.resize(capacity);
    t->stop.resize(capacity);
    t->kernel_id.assign(capacity, -1);
    for (int i = 0; i < capacity; ++i) {
        if (cudaEventCreate(&t->start[i]) != cudaSuccess || cudaEventCreate(&t->stop[i]) != cudaSuccess) {
            cudaGetLastError();
            return DSPARK_ERR_CUDA;
        }
    }
    *out = t;
    return DSPARK_OK;
}

int dspark_ktimer_destroy(dspark_ktimer_t* t)
{
    if (!t) return DSPARK_ERR_INVALID_ARG;
    if (dspark::g_timer == t) dspark::g_timer = nullptr;
    for (int i = 0; i < t->capacity; ++i) { cudaEventDestroy(t->start[i]); cudaEventDestroy(t->stop[i]); }
    delete t;
    return DSPARK_OK;
}

int dspark_ktimer_attach(dspark_ktimer_t* t)
{
    dspark::g_timer = t;
    return DSPARK_OK;
}

int dspark_ktimer_reset(dspark_ktimer_t* t)
{
    if (!t) return DSPARK_ERR_INVALID_ARG;
    t->used = 0;
    return DSPARK_OK;
}

int dspark_ktimer_read(dspark_ktimer_t* t, int kernel_id, float* total_ms, int* launches)
{
    if (!t || !total_ms || !launches) return DSPARK_ERR_INVALID_ARG;
    float sum = 0.f;
    int n = 0;
    for (int i = 0; i < t->used; ++i) {
        if (t->kernel_id[i] != kernel_id) continue;
        if (cudaEventSynchronize(t->stop[i]) != cudaSuccess) { cudaGetLastError(); return DSPARK_ERR_CUDA; }
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t->start[i], t->stop[i]) != cudaSuccess) { cudaGetLastError(); return DSPARK_ERR_CUDA; }
        sum += ms;
        ++n;
    }
    *total_ms = sum;
    *launches = n;
    return DSPARK_OK;
}

const char* dspark_status_string(int s)
{
    switch (s) {
        case DSPARK_OK: return "ok";
        case DSPARK_ERR_INVALID_ARG: return "invalid argument";
        case DSPARK_ERR_SHAPE: return "unsupported shape";
        case DSPARK_ERR_ALIGNMENT: return "misaligned buffer";
        case DSPARK_ERR_WORKSPACE: return "workspace too small";
        case DSPARK_ERR_CUDA: return "CUDA error";
        case DSPARK_ERR_STATIC_LIMIT: return "batch exceeds the built-in scratch array";
        default: return "unknown status";
    }
}

const char* dspark_kernel_name(int id)
{
    static const char* names[DSPARK_K_COUNT] = {
        "schedule", "build_offsets", "stream_stats", "decide", "residual_stream", "finalize",
        "greedy_stream", "greedy_decide", "row_scale", "markov_gemm", "markov_draw", "truncate"};
    return (id >= 0 && id < DSPARK_K_COUNT) ? names[id] : "?";
}

int dspark_version(void) { return 100; }

}  // extern "C"
