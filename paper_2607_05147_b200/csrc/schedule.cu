// dspark_schedule: the hardware-aware prefix scheduler (Algorithm 1; Sections 3.2.2, 4.2)
// as one single-CTA kernel: survival products -> 64-bit key sort in shared memory ->
// exact integer prefix sums of the expected-accept mass -> Theta path and stop rule ->
// per-request lengths, row offsets, expected lengths.  The problem is a few thousand
// keys: latency-bound, so everything stays inside one CTA with no host round trip.
#include "common.cuh"

namespace dspark {

constexpr int kSchedThreads = 1024;
constexpr int kSmemKeyCap = 16384;          // 128 KB of 64-bit keys in shared memory
constexpr unsigned long long kPadKey = ~0ull;

struct SchedParams {
    const float* conf;
    const int32_t* draft_len;
    int R, gamma, budget, mode, topk;
    const double* table;
    int max_tokens;
    int32_t* out_len;
    int32_t* out_offsets;
    float* out_surv;
    float* out_exp;
    dspark_sched_info_t* info;
    unsigned long long* keys_global;
    int n_pad;
};

__device__ __forceinline__ float sanitize_conf(float c, int& clamped)
{
    if (!(c >= 0.0f)) { clamped = 1; return 0.0f; }
    if (c > 1.0f) { clamped = 1; return 1.0f; }
    return c;
}
__device__ __forceinline__ unsigned long long fix40(float a)
{
    return __double2ull_rz(__dmul_rn((double)a, 1099511627776.0));
}
__device__ __forceinline__ float key_survival(unsigned long long key)
{
    return __uint_as_float(~(uint32_t)(key >> 32));
}

// Inclusive scan of one 64-bit value per thread over the CTA (1024 threads).
__device__ __forceinline__ unsigned long long block_scan_u64(unsigned long long v, unsigned long long* warp_tot)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
    }
    if (lane == 31) warp_tot[warp] = v;
    __syncthreads();
    if (warp == 0) {
        unsigned long long t = warp_tot[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long n = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t += n;
        }
        warp_tot[lane] = t;
    }
    __syncthreads();
    if (warp > 0) v += warp_tot[warp - 1];
    __syncthreads();
    return v;
}

template <bool kSmemKeys>
__global__ void __launch_bounds__(kSchedThreads, 1) schedule_kernel(SchedParams P)
{
    extern __shared__ __align__(16) unsigned long long smem_keys[];
    unsigned long long* keys = kSmemKeys ? smem_keys : P.keys_global;
    __shared__ unsigned long long s_warp_tot[32];
    __shared__ unsigned long long s_carry, s_T_best;
    __shared__ double s_theta_best;
    __shared__ int s_first_bad, s_istar, s_nE, s_status, s_done;
    __shared__ double s_red_theta[32];
    __shared__ int s_red_i[32];
    __shared__ unsigned long long s_red_T[32];

    const int tid = threadIdx.x;
    const int R = P.R, gamma = P.gamma;
    const int n = R * gamma;

    if (tid == 0) { s_nE = 0; s_status = 0; s_first_bad = 0x7fffffff; s_done = 0; }
    __syncthreads();

    // ---- S1: survival products a_{r,j} (fp32, left to right) and sort keys --------------
    {
        int my_cand = 0, clamped = 0;
        for (int r = tid; r < R; r += kSchedThreads) {
            int lim = gamma;
            if (P.draft_len) { lim = P.draft_len[r]; lim = lim < 0 ? 0 : (lim > gamma ? gamma : lim); }
            float a = 1.0f;
            bool dead = false;
            for (int j = 0; j < gamma; ++j) {
                if (j >= lim) dead = true;
                if (!dead) {
                    a = __fmul_rn(a, sanitize_conf(P.conf[(size_t)r * gamma + j], clamped));
                    if (!(a > 0.0f)) dead = true;
                }
                float s = dead ? 0.0f : a;
                if (P.out_surv) P.out_surv[(size_t)r * gamma + j] = s;
                unsigned long long key = kPadKey;
                if (!dead) {
                    // ascending key order == (a descending, position ascending, request ascending)
                    key = ((unsigned long long)(~__float_as_uint(s)) << 32) | ((unsigned)j << 20) | (unsigned)r;
                    ++my_cand;
                }
                keys[(size_t)r * gamma + j] = key;
            }
        }
        for (int i = n + tid; i < P.n_pad; i += kSchedThreads) keys[i] = kPadKey;
        if (my_cand) atomicAdd(&s_nE, my_cand);
        if (clamped) atomicOr(&s_status, DSPARK_DEV_CONF_CLAMPED);
    }
    __syncthreads();

    // ---- S2: bitonic sort, ascending ----------------------------------------------------
    const int np = P.n_pad;
    for (int k = 2; k <= np; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < (np >> 1); i += kSchedThreads) {
                int lo = ((i & ~(j - 1)) << 1) | (i & (j - 1));
                int hi = lo + j;
                unsigned long long x = keys[lo], y = keys[hi];
                bool up = (lo & k) == 0;
                if ((x > y) == up) { keys[lo] = y; keys[hi] = x; }
            }
            __syncthreads();
        }
    }

    // ---- S3 + S4: admission path, Theta_i = tau_i * SPS(R + i), stop rule -----------------
    const int nE = s_nE;
    long long cap = (long long)P.budget - (long long)R;
    if (cap < 0) { cap = 0; if (tid == 0) s_status |= DSPARK_DEV_BUDGET_LT_R; }
    const int N = (int)(nE < cap ? nE : cap);
    const unsigned long long T0 = (unsigned long long)R << 40;
    const int mt = P.max_tokens;
    if (tid == 0) {
        s_carry = T0;
        s_T_best = T0;
        s_theta_best = __dmul_rn(__ull2double_rn(T0), P.table[R < mt ? R : mt]);
        s_istar = 0;
    }
    __syncthreads();

    for (int base = 0; base < N; base += kSchedThreads) {
        const int i = base + tid + 1;                 // 1-based admitted count
        const bool valid = i <= N;
        unsigned long long v = valid ? fix40(key_survival(keys[i - 1])) : 0ull;
        unsigned long long Ti = block_scan_u64(v, s_warp_tot) + s_carry;
        double theta_i = 0.0;
        if (valid) {
            int B = R + i;
            theta_i = __dmul_rn(__ull2double_rn(Ti), P.table[B < mt ? B : mt]);
        }
        if (P.mode == DSPARK_SCHED_EARLY_STOP) {
            if (valid) {
                int Bp = R + i - 1;
                double theta_prev = __dmul_rn(__ull2double_rn(Ti - v), P.table[Bp < mt ? Bp : mt]);
                if (!(theta_i > theta_prev)) atomicMin(&s_first_bad, i);
            }
            __syncthreads();
            const int fb = s_first_bad;
            const int istar = (fb != 0x7fffffff) ? fb - 1 : (base + kSchedThreads < N ? base + kSchedThreads : N);
            if (valid && i == istar) { s_T_best = Ti; s_theta_best = theta_i; s_istar = i; }
            if (fb != 0x7fffffff && tid == 0) s_done = 1;
        } else if (P.mode == DSPARK_SCHED_GLOBAL) {
            // CTA-wide argmax of Theta with the smallest i on ties; NaN never wins
            double bt = (valid && theta_i == theta_i) ? theta_i : -INFINITY;
            int bi = valid ? i : 0x7fffffff;
            unsigned long long bT = Ti;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                double ot = __shfl_xor_sync(0xffffffffu, bt, o);
                int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                unsigned long long oT = __shfl_xor_sync(0xffffffffu, bT, o);
                if (ot > bt || (ot == bt && oi < bi)) { bt = ot; bi = oi; bT = oT; }
            }
            if ((tid & 31) == 0) { s_red_theta[tid >> 5] = bt; s_red_i[tid >> 5] = bi; s_red_T[tid >> 5] = bT; }
            __syncthreads();
            if (tid < 32) {
                bt = s_red_theta[tid]; bi = s_red_i[tid]; bT = s_red_T[tid];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    double ot = __shfl_xor_sync(0xffffffffu, bt, o);
                    int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                    unsigned long long oT = __shfl_xor_sync(0xffffffffu, bT, o);
                    if (ot > bt || (ot == bt && oi < bi)) { bt = ot; bi = oi; bT = oT; }
                }
                if (tid == 0 && bi != 0x7fffffff && bt > s_theta_best) {
                    s_theta_best = bt; s_istar = bi; s_T_best = bT;
                }
            }
        } else {  // DSPARK_SCHED_TOPK
            const int K = P.topk < 0 ? 0 : P.topk;
            const int istar = N < K ? N : K;
            if (valid && i == istar) { s_T_best = Ti; s_theta_best = theta_i; s_istar = i; }
        }
        if (tid == kSchedThreads - 1) s_carry = Ti;
        __syncthreads();
        if (s_done) break;
    }
    __syncthreads();
    const int istar = s_istar;

    // ---- lengths l*_r = admitted candidates of request r ---------------------------------
    for (int r = tid; r < R; r += kSchedThreads) P.out_len[r] = 0;
    __syncthreads();
    for (int k = tid; k < istar; k += kSchedThreads) atomicAdd(&P.out_len[(int)(keys[k] & 0xFFFFFu)], 1);
    __syncthreads();

    // ---- row offsets: exclusive scan of (l*_r + 1) ---------------------------------------
    if (P.out_offsets) {
        if (tid == 0) s_carry = 0ull;
        __syncthreads();
        for (int base = 0; base < R; base += kSchedThreads) {
            const int r = base + tid;
            unsigned long long v = r < R ? (unsigned long long)(__ldcg(&P.out_len[r]) + 1) : 0ull;
            unsigned long long incl = block_scan_u64(v, s_warp_tot) + s_carry;
            if (r < R) P.out_offsets[r] = (int32_t)(incl - v);
            if (r == R - 1) P.out_offsets[R] = (int32_t)incl;
            __syncthreads();
            if (tid == kSchedThreads - 1) s_carry = incl;
            __syncthreads();
        }
    }

    // ---- expected accepted length 1 + sum_{j < l*_r} a_{r,j} -----------------------------
    if (P.out_exp) {
        for (int r = tid; r < R; r += kSchedThreads) {
            const int len = __ldcg(&P.out_len[r]);
            float a = 1.0f;
            double e = 1.0;
            int dummy = 0;
            for (int j = 0; j < len; ++j) {
                a = __fmul_rn(a, sanitize_conf(P.conf[(size_t)r * gamma + j], dummy));
                e = __dadd_rn(e, (double)a);
            }
            P.out_exp[r] = (float)e;
        }
    }
    if (P.info && tid == 0) {
        dspark_sched_info_t o;
        o.B = R + istar;
        o.n_admitted = istar;
        o.status = s_status;
        o.n_candidates = nE;
        o.tau = __ull2double_rn(s_T_best) * (1.0 / 1099511627776.0);
        o.theta = s_theta_best * (1.0 / 1099511627776.0);
        *P.info = o;
    }
}

__global__ void __launch_bounds__(kSchedThreads, 1)
build_offsets_kernel(const int32_t* __restrict__ lengths, int R, int32_t* __restrict__ offsets)
{
    __shared__ unsigned long long s_warp_tot[32];
    __shared__ unsigned long long s_carry;
    const int tid = threadIdx.x;
    if (tid == 0) s_carry = 0ull;
    __syncthreads();
    for (int base = 0; base < R; base += kSchedThreads) {
        const int r = base + tid;
        int len = r < R ? lengths[r] : -1;
        if (len < 0 && r < R) len = 0;
        unsigned long long v = r < R ? (unsigned long long)(len + 1) : 0ull;
        unsigned long long incl = block_scan_u64(v, s_warp_tot) + s_carry;
        if (r < R) offsets[r] = (int32_t)(incl - v);
        if (r == R - 1) offsets[R] = (int32_t)incl;
        __syncthreads();
        if (tid == kSchedThreads - 1) s_carry = incl;
        __syncthreads();
    }
}

static int next_pow2(int x)
{
    int p = 2;
    while (p < x) p <<= 1;
    return p;
}

}  // namespace dspark

using namespace dspark;

extern "C" {

size_t dspark_schedule_workspace_bytes(int R, int gamma)
{
    if (R < 1 || gamma < 0) return 0;
    long long n = (long long)R * gamma;
    if (n > (1 << 20)) return 0;
    return (size_t)next_pow2((int)(n > 2 ? n : 2)) * sizeof(unsigned long long);
}

int dspark_schedule(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                    int R, int gamma, int budget_tokens, int mode, int topk_K,
                    int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                    float* out_expected_len, dspark_sched_info_t* out_info,
                    void* workspace, size_t workspace_bytes, void* stream)
{
    if (!prof || !out_len || (!conf && gamma > 0)) return DSPARK_ERR_INVALID_ARG;
    if (mode != DSPARK_SCHED_EARLY_STOP && mode != DSPARK_SCHED_GLOBAL && mode != DSPARK_SCHED_TOPK)
        return DSPARK_ERR_INVALID_ARG;
    if (R < 1 || gamma < 0) return DSPARK_ERR_INVALID_ARG;
    if (R > (1 << 20) || gamma > 4096 || (long long)R * gamma > (1 << 20)) return DSPARK_ERR_SHAPE;
    const size_t need = dspark_schedule_workspace_bytes(R, gamma);
    if (!workspace || workspace_bytes < need) return DSPARK_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 15u) != 0) return DSPARK_ERR_ALIGNMENT;

    int max_tokens = 0;
    const double* table = dspark_profile_table(prof, &max_tokens);
    SchedParams P;
    P.conf = conf; P.draft_len = draft_len;
    P.R = R; P.gamma = gamma; P.budget = budget_tokens; P.mode = mode; P.topk = topk_K;
    P.table = table; P.max_tokens = max_tokens;
    P.out_len = out_len; P.out_offsets = out_row_offsets; P.out_surv = out_survival;
    P.out_exp = out_expected_len; P.info = out_info;
    P.keys_global = (unsigned long long*)workspace;
    P.n_pad = next_pow2(R * gamma > 2 ? R * gamma : 2);

    cudaStream_t s = (cudaStream_t)stream;
    KernelTimerScope timer(DSPARK_K_SCHEDULE, s);
    if (P.n_pad <= kSmemKeyCap) {
        const size_t smem = (size_t)P.n_pad * sizeof(unsigned long long);
        static bool attr_set = false;
        if (!attr_set) {
            if (cudaFuncSetAttribute(schedule_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     kSmemKeyCap * (int)sizeof(unsigned long long)) != cudaSuccess)
                return launch_status();
            attr_set = true;
        }
        schedule_kernel<true><<<1, kSchedThreads, smem, s>>>(P);
    } else {
        schedule_kernel<false><<<1, kSchedThreads, 0, s>>>(P);
    }
    return launch_status();
}

int dspark_build_offsets(const int32_t* lengths, int R, int32_t* row_offsets, void* stream)
{
    if (!lengths || !row_offsets || R < 1) return DSPARK_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    KernelTimerScope timer(DSPARK_K_OFFSETS, s);
    build_offsets_kernel<<<1, kSchedThreads, 0, s>>>(lengths, R, row_offsets);
    return launch_status();
}

}  // extern "C"
