// top-k / top-p truncation of fp32 target rows (per-request sampling parameters, Section 4.1): the same value cut as
// truncate.cu computes for bf16 rows,
//   S = { v : x_v >= tau },  tau = max(tau_k, tau_p),
//   tau_k = k-th largest logit,  tau_p = first value, walking the distinct values downwards inside the top-k set,
//           at which the cumulative mass reaches top_p * Z_k,
// found exactly on the 32-bit patterns.  A bf16 logit is a 16-bit key and a window of a histogram resolves it; an fp32
// logit needs a descent.  One CTA per row (the row is read from L2 after the first pass):
//   pass 0      row maximum m, NaN / +inf detection;
//   level A     histogram over 2048 bins linear in (m - x) (bin width 8 T / 2047; monotone in x, so a lower bin holds
//               strictly larger values): count and mass per bin, everything further than 8 T below the maximum summed
//               as one last bin in registers (no shared-memory atomics for the bulk of a peaked row); a threshold in
//               that last bin (flat rows) moves the window 8 T further down, one more pass per window;
//   descent     inside the bin that holds the threshold: one more pass moves its elements (usually a few hundred) to
//               shared memory and finds their key range; then histograms of 11 bits of (largest key - key) at a time
//               over that list until the bins are single keys.  A bin too large for the list is re-read from the row.
// Masses are exponentials relative to the maximum in units of 2^-40, summed as integers: the sums do not depend on
// the order of the atomics, so the result is the same from run to run.  Counts are exact, so the top-k part is exact;
// the top-p decision compares integer sums of fp32 exponentials with top_p * Z and can differ from an fp64 reference
// only when the two sides agree to ~1e-6 of Z.
#include <math.h>

#include <atomic>

#include "common.cuh"

namespace dspark {

constexpr int kF32Threads = 1024;
constexpr int kF32Bins = 2048;
constexpr int kF32PerThread = kF32Bins / kF32Threads;
constexpr int kF32Unroll = 4;
constexpr int kF32ListCap = 16384;                 // 64 KB: a bin with more elements is re-read from the row instead

struct TruncF32Params {
    float* target; long long stride; int V;                // stride in elements
    const int32_t* row_offsets; int R, n_rows;
    const int32_t* top_k; const float* top_p; const float* temperatures; float temperature;
    float* out_tau; int32_t* out_kept;
    // virtual mode (inside the verifier): the row is not modified; its statistics blocks receive the sums
    // restricted to the kept set instead
    float2* stats; int nblk, epb;
};

// order-preserving key of an fp32 value (-0 and +0 share a key) and back
__device__ __forceinline__ uint32_t f32_key(float x)
{
    uint32_t b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float f32_key_value(uint32_t k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// fn(i, x) for every element of the row: 16-byte loads over the aligned middle of the row, kF32Unroll of them in
// flight per thread, element loads for the few elements before and after it.
template <typename F>
__device__ __forceinline__ void for_each_elem(const float* row, int V, F fn)
{
    int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) >> 2);
    if (head > V) head = V;
    const int nvec = (V - head) >> 2;
    const float4* p = reinterpret_cast<const float4*>(row + head);
    for (int c0 = threadIdx.x; c0 < nvec; c0 += kF32Unroll * kF32Threads) {
        float4 v[kF32Unroll];
#pragma unroll
        for (int u = 0; u < kF32Unroll; ++u) {
            const int c = c0 + u * kF32Threads;
            v[u] = c < nvec ? __ldcg(&p[c]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kF32Unroll; ++u) {
            const int c = c0 + u * kF32Threads;
            if (c < nvec) {
                const int i = head + 4 * c;
                fn(i, v[u].x); fn(i + 1, v[u].y); fn(i + 2, v[u].z); fn(i + 3, v[u].w);
            }
        }
    }
    const int tail0 = head + 4 * nvec;
    for (int i = threadIdx.x; i < head + (V - tail0); i += kF32Threads) {
        const int e = i < head ? i : tail0 + (i - head);
        fn(e, __ldcg(&row[e]));
    }
}

// The same walk with the aligned middle of the row handed over four elements at a time: vec(v) for every 16-byte
// vector, elem(x) for the few elements before and after.  The passes below decide about a whole vector with a handful
// of instructions (almost every vector of a row lies entirely below the window) and fall back to the element form
// only for the vectors that do not.
template <typename FV, typename FE>
__device__ __forceinline__ void for_each_vec(const float* row, int V, FV vec, FE elem)
{
    int head = (int)(((16u - (unsigned)((uintptr_t)row & 15u)) & 15u) >> 2);
    if (head > V) head = V;
    const int nvec = (V - head) >> 2;
    const float4* p = reinterpret_cast<const float4*>(row + head);
    for (int c0 = threadIdx.x; c0 < nvec; c0 += kF32Unroll * kF32Threads) {
        float4 v[kF32Unroll];
#pragma unroll
        for (int u = 0; u < kF32Unroll; ++u) {
            const int c = c0 + u * kF32Threads;
            v[u] = c < nvec ? __ldcg(&p[c]) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < kF32Unroll; ++u)
            if (c0 + u * kF32Threads < nvec) vec(v[u]);
    }
    const int tail0 = head + 4 * nvec;
    for (int i = threadIdx.x; i < head + (V - tail0); i += kF32Threads) elem(__ldcg(&row[i < head ? i : tail0 + (i - head)]));
}
__device__ __forceinline__ float max_nan(float a, float b)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

struct F32Shared {
    unsigned int cnt[kF32Bins];
    unsigned long long mass[kF32Bins];
    unsigned long long warp_c[kF32Threads / 32], warp_m[kF32Threads / 32];
    unsigned long long red_c, red_m;                        // block reductions / results of a scan
    unsigned long long before_c, before_m, bin_c, bin_m;
    unsigned int kmin, kmax;
    int req, flag, hit, n_list;
    float m;
    float list[kF32ListCap];                               // the elements of the level A bin under descent
};

// Sum of one (count, mass) pair per thread over the CTA; result in S.red_c / S.red_m, valid after the call.
__device__ __forceinline__ void block_sum_pair(F32Shared& S, unsigned long long c, unsigned long long m)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        c += __shfl_xor_sync(0xffffffffu, c, o);
        m += __shfl_xor_sync(0xffffffffu, m, o);
    }
    __syncthreads();
    if (lane == 0) { S.warp_c[warp] = c; S.warp_m[warp] = m; }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long tc = 0ull, tm = 0ull;
        for (int w = 0; w < kF32Threads / 32; ++w) { tc += S.warp_c[w]; tm += S.warp_m[w]; }
        S.red_c = tc; S.red_m = tm;
    }
    __syncthreads();
}

// Walks the histogram in S.cnt / S.mass (bin 0 first) and finds the first non-empty bin at which
// pred(count through the bin, mass through the bin) holds, counts and masses starting from (c0, m0).
// Returns the bin or -1; S.before_* then hold the sums of the bins before it, S.bin_* its own.
template <typename Pred>
__device__ int scan_histogram(F32Shared& S, unsigned long long c0, unsigned long long m0, Pred pred)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned int c[kF32PerThread];
    unsigned long long m[kF32PerThread];
    unsigned long long lc = 0ull, lm = 0ull;
#pragma unroll
    for (int j = 0; j < kF32PerThread; ++j) {
        c[j] = S.cnt[tid * kF32PerThread + j];
        m[j] = S.mass[tid * kF32PerThread + j];
        lc += c[j]; lm += m[j];
    }
    unsigned long long ic = lc, im = lm;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long nc = __shfl_up_sync(0xffffffffu, ic, o);
        const unsigned long long nm = __shfl_up_sync(0xffffffffu, im, o);
        if (lane >= o) { ic += nc; im += nm; }
    }
    if (tid == 0) S.hit = 0x7fffffff;
    __syncthreads();
    if (lane == 31) { S.warp_c[warp] = ic; S.warp_m[warp] = im; }
    __syncthreads();
    unsigned long long bc = c0, bm = m0;
    for (int w = 0; w < warp; ++w) { bc += S.warp_c[w]; bm += S.warp_m[w]; }
    unsigned long long rc = bc + (ic - lc), rm = bm + (im - lm);      // before my first bin
    int mine = 0x7fffffff;
    unsigned long long mine_c = 0ull, mine_m = 0ull;
#pragma unroll
    for (int j = 0; j < kF32PerThread; ++j) {
        if (mine == 0x7fffffff && c[j] && pred(rc + c[j], rm + m[j])) { mine = tid * kF32PerThread + j; mine_c = rc; mine_m = rm; }
        rc += c[j]; rm += m[j];
    }
    if (mine != 0x7fffffff) atomicMin(&S.hit, mine);
    __syncthreads();
    const int h = S.hit;
    if (h != 0x7fffffff && h == mine) {
        S.before_c = mine_c; S.before_m = mine_m;
        S.bin_c = S.cnt[h]; S.bin_m = S.mass[h];
    }
    __syncthreads();
    return h == 0x7fffffff ? -1 : h;
}

__device__ void truncate_row_f32(const TruncF32Params& P, const int row, F32Shared& S)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        int lo = 0, hi = P.R;                               // largest r with row_offsets[r] <= row
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (P.row_offsets[mid] <= row) lo = mid; else hi = mid;
        }
        const int n = P.row_offsets[P.R];
        S.req = (row < n && row < P.n_rows && row >= P.row_offsets[0]) ? lo : -1;
        S.flag = 0;
    }
    __syncthreads();
    const int r = S.req;
    if (r < 0) return;
    const int V = P.V;
    const int k = P.top_k ? P.top_k[r] : 0;
    const float pf = P.top_p ? P.top_p[r] : 1.f;
    const float T = P.temperatures ? P.temperatures[r] : P.temperature;
    const bool use_k = k > 0 && k < V, use_p = pf < 1.f;
    if (tid == 0) {
        if (P.out_tau) P.out_tau[row] = -INFINITY;
        if (P.out_kept) P.out_kept[row] = V;
    }
    if ((!use_k && !use_p) || !(T > 0.f) || isinf(T)) return;
    float* rowp = P.target + (long long)row * P.stride;

    // ---- pass 0: maximum, NaN / +inf ------------------------------------------------------------------------
    {
        float mx = -INFINITY;                                // a NaN anywhere survives this maximum
        for_each_vec(rowp, V, [&](float4 v) { mx = max_nan(mx, max_nan(max_nan(v.x, v.y), max_nan(v.z, v.w))); },
                     [&](float x) { mx = max_nan(mx, x); });
        const bool bad = mx != mx;
        mx = warp_max_f32(bad ? -INFINITY : mx);
        if (bad) S.flag = 1;
        __syncthreads();
        if (lane == 0) S.warp_c[warp] = (unsigned long long)f32_key(mx);
        __syncthreads();
        if (tid == 0) {
            unsigned long long best = 0ull;
            for (int w = 0; w < kF32Threads / 32; ++w) best = S.warp_c[w] > best ? S.warp_c[w] : best;
            S.m = f32_key_value((uint32_t)best);
        }
        __syncthreads();
    }
    const float m = S.m;
    if (S.flag || m == INFINITY || m == -INFINITY) return;    // left as it is: the verifier reports such rows
    const float scale2 = (float)(1.4426950408889634 / (double)T);
    const float nm2 = -m * scale2;
    // mass of an element relative to the maximum, in units of 2^-40
    // (only top-p looks at masses: a top-k cut alone is pure counting)
    auto mass_of = [&](float x) -> unsigned long long {
        return use_p ? __float2ull_rz(ex2_approx(__fmaf_rn(x, scale2, nm2)) * 1099511627776.0f) : 0ull;
    };
    // Linear index of an element: its distance to the maximum in units of 8 T / 2047.  Window w of the histogram
    // holds the indices [2047 w, 2047 (w + 1)) in its first 2047 bins and everything further down in its last bin;
    // what lies above the window is not counted (the caller carries its sums).  Window 0 reaches 8 T below the
    // maximum -- a token further down carries less than e^-8 of the maximum's mass, so the thresholds of a peaked
    // row lie inside it; a flat row moves on to the next windows.
    const float bin_scale = (float)(kF32Bins - 1) / (8.0f * T);
    // (one multiply-add per element, non-increasing in x; the bulk of a row leaves after one comparison)
    const float mb = m * bin_scale;
    auto win_bin = [&](float x, int w) -> int {
        const float d = fmaxf(__fmaf_rn(x, -bin_scale, mb), 0.0f);
        const float lo = (float)(w * (kF32Bins - 1));
        if (!(d < lo + (float)(kF32Bins - 1))) return kF32Bins - 1;      // far below, -inf included
        return d < lo ? -1 : (int)d - w * (kF32Bins - 1);
    };
    int cur_w = -1;                                                      // window whose histogram is in shared memory
    auto build_window = [&](int w) {
        __syncthreads();
        for (int i = tid; i < kF32Bins; i += kF32Threads) { S.cnt[i] = 0u; S.mass[i] = 0ull; }
        __syncthreads();
        unsigned long long far_c = 0ull, far_m = 0ull;
        auto one = [&](float x) {
            const int b = win_bin(x, w);
            if (b < 0) return;
            const unsigned long long fx = mass_of(x);
            if (b == kF32Bins - 1) { ++far_c; far_m += fx; }
            else { atomicAdd(&S.cnt[b], 1u); atomicAdd(&S.mass[b], fx); }
        };
        // a vector entirely below the window: counted, and (top-p) its masses summed in fp32 per vector lane -- every
        // thread adds its own elements in a fixed order, so these sums are the same from run to run as well
        const float far_from = (float)((w + 1) * (kF32Bins - 1));
        unsigned int far_v = 0u;
        float4 fa = make_float4(0.f, 0.f, 0.f, 0.f);
        for_each_vec(rowp, V, [&](float4 v) {
            const float d0 = __fmaf_rn(v.x, -bin_scale, mb), d1 = __fmaf_rn(v.y, -bin_scale, mb);
            const float d2 = __fmaf_rn(v.z, -bin_scale, mb), d3 = __fmaf_rn(v.w, -bin_scale, mb);
            if (fminf(fminf(d0, d1), fminf(d2, d3)) >= far_from) {
                ++far_v;
                if (use_p) {
                    fa.x += ex2_approx(__fmaf_rn(v.x, scale2, nm2)); fa.y += ex2_approx(__fmaf_rn(v.y, scale2, nm2));
                    fa.z += ex2_approx(__fmaf_rn(v.z, scale2, nm2)); fa.w += ex2_approx(__fmaf_rn(v.w, scale2, nm2));
                }
            } else {
                one(v.x); one(v.y); one(v.z); one(v.w);
            }
        }, one);
        far_c += 4ull * far_v;
        far_m += __double2ull_rz((((double)fa.x + (double)fa.y) + ((double)fa.z + (double)fa.w)) * 1099511627776.0);
        block_sum_pair(S, far_c, far_m);
        if (tid == 0) { S.cnt[kF32Bins - 1] = (unsigned int)S.red_c; S.mass[kF32Bins - 1] = S.red_m; }
        __syncthreads();
        cur_w = w;
    };

    // ---- window 0: one histogram serves both thresholds ----------------------------------------------------
    build_window(0);
    // total mass of the row (top-p without top-k normalises by it)
    unsigned long long z_all;
    {
        unsigned long long lc = 0ull, lm = 0ull;
        for (int j = 0; j < kF32PerThread; ++j) { lc += S.cnt[tid * kF32PerThread + j]; lm += S.mass[tid * kF32PerThread + j]; }
        block_sum_pair(S, lc, lm);
        z_all = S.red_m;
    }
    // it is needed twice (top-k, then top-p): keep a copy in registers
    unsigned int a_cnt[kF32PerThread];
    unsigned long long a_mass[kF32PerThread];
#pragma unroll
    for (int j = 0; j < kF32PerThread; ++j) { a_cnt[j] = S.cnt[tid * kF32PerThread + j]; a_mass[j] = S.mass[tid * kF32PerThread + j]; }
    constexpr int kMaxWindows = 8;                                       // 64 T below the maximum; beyond: by keys alone

    // Descent: the key at which pred first holds walking the values downwards; count and mass of everything at or
    // above that key.
    auto descend = [&](auto pred, uint32_t& key_out, unsigned long long& cnt_out, unsigned long long& mass_out) -> bool {
        int w = 0, bA;
        unsigned long long c0 = 0ull, m0 = 0ull;
        for (;;) {
            if (w == 0 && cur_w != 0) {
                __syncthreads();
#pragma unroll
                for (int j = 0; j < kF32PerThread; ++j) { S.cnt[tid * kF32PerThread + j] = a_cnt[j]; S.mass[tid * kF32PerThread + j] = a_mass[j]; }
                __syncthreads();
                cur_w = 0;
            } else if (w != cur_w) {
                build_window(w);
            }
            bA = scan_histogram(S, c0, m0, pred);
            if (bA < 0) return false;
            if (bA != kF32Bins - 1 || w == kMaxWindows - 1) break;
            c0 = S.before_c; m0 = S.before_m;                            // the threshold lies further down: next window
            ++w;
        }
        cur_w = -1;                                                      // the levels below reuse the histogram
        auto lin_bin = [&](float x) -> int { return win_bin(x, w); };
        unsigned long long c_before = S.before_c, m_before = S.before_m;
        // The elements of that bin (usually a few hundred) move to shared memory in one more pass over the row,
        // which also gives their key range; the levels below then never touch the row again.  A bin too large for
        // the list (the far bin of a flat row) is re-read from the row at every level instead.
        const bool listed = S.bin_c <= (unsigned long long)kF32ListCap;
        if (tid == 0) { S.kmin = 0xFFFFFFFFu; S.kmax = 0u; S.n_list = 0; }
        __syncthreads();
        {
            uint32_t lo = 0xFFFFFFFFu, hi = 0u;
            // members of an inner bin have Bf <= d < Bf + 1: a vector with all four distances on one side of that has none
            const float Bf = (float)(bA + w * (kF32Bins - 1));
            const bool inner = bA != kF32Bins - 1;
            auto one = [&](float x) {
                if (lin_bin(x) == bA) {
                    const uint32_t kx = f32_key(x);
                    lo = min(lo, kx); hi = max(hi, kx);
                    if (listed) {
                        // one shared-memory atomic per group of lanes that found a member in the same step
                        const unsigned act = __activemask();
                        const int leader = __ffs(act) - 1;
                        int at = 0;
                        if (lane == leader) at = atomicAdd(&S.n_list, __popc(act));
                        at = __shfl_sync(act, at, leader);
                        S.list[at + __popc(act & ((1u << lane) - 1u))] = x;
                    }
                }
            };
            for_each_vec(rowp, V, [&](float4 v) {
                if (inner) {
                    const float d0 = __fmaf_rn(v.x, -bin_scale, mb), d1 = __fmaf_rn(v.y, -bin_scale, mb);
                    const float d2 = __fmaf_rn(v.z, -bin_scale, mb), d3 = __fmaf_rn(v.w, -bin_scale, mb);
                    if (fminf(fminf(d0, d1), fminf(d2, d3)) >= Bf + 1.0f) return;
                    if (Bf > 0.0f && fmaxf(fmaxf(d0, d1), fmaxf(d2, d3)) < Bf) return;
                }
                one(v.x); one(v.y); one(v.z); one(v.w);
            }, one);
            lo = __reduce_min_sync(0xffffffffu, lo);
            hi = __reduce_max_sync(0xffffffffu, hi);
            if (lane == 0) { atomicMin(&S.kmin, lo); atomicMax(&S.kmax, hi); }
        }
        __syncthreads();
        const int n_list = S.n_list;
        const uint32_t kref = S.kmax;
        uint32_t base = 0u;                                  // distances [base, base + 2^width) are still candidates
        int width = 32 - __clz(kref - S.kmin);               // bits of the largest distance (0: one key)
        for (;;) {
            const int shift = width > 11 ? width - 11 : 0;
            __syncthreads();
            for (int i = tid; i < kF32Bins; i += kF32Threads) { S.cnt[i] = 0u; S.mass[i] = 0ull; }
            __syncthreads();
            auto count = [&](float x) {
                const uint32_t d = kref - f32_key(x);
                if (d < base || (width < 32 && d - base >= (1u << width))) return;
                const uint32_t b = (d - base) >> shift;
                atomicAdd(&S.cnt[b], 1u);
                atomicAdd(&S.mass[b], mass_of(x));
            };
            if (listed) {
                for (int i = tid; i < n_list; i += kF32Threads) count(S.list[i]);
            } else {
                for_each_elem(rowp, V, [&](int, float x) { if (lin_bin(x) == bA) count(x); });
            }
            __syncthreads();
            const int h = scan_histogram(S, c_before, m_before, pred);
            if (h < 0) return false;                          // cannot happen: the bin of level A satisfied pred
            c_before = S.before_c; m_before = S.before_m;
            base += (uint32_t)h << shift;
            if (shift == 0) {
                key_out = kref - base;
                cnt_out = c_before + S.bin_c;
                mass_out = m_before + S.bin_m;
                return true;
            }
            width = shift;
        }
    };

    // ---- top-k, then top-p inside the top-k set ------------------------------------------------------------
    bool have = false;
    uint32_t tau_key = 0u;
    unsigned long long kept = (unsigned long long)V, zk = z_all;
    if (use_k) {
        const unsigned long long need = (unsigned long long)k;
        uint32_t key; unsigned long long c, q;
        if (descend([&](unsigned long long cc, unsigned long long) { return cc >= need; }, key, c, q)) {
            have = true; tau_key = key; kept = c; zk = q;
        }
    }
    if (use_p) {
        if (!(pf > 0.f)) {
            // only the maximum
            uint32_t key; unsigned long long c, q;
            if (descend([&](unsigned long long cc, unsigned long long) { return cc >= 1ull; }, key, c, q)) {
                have = true; tau_key = key; kept = c;
            }
        } else {
            const double thr = (double)pf * (double)zk;
            uint32_t key; unsigned long long c, q;
            if (descend([&](unsigned long long, unsigned long long qq) { return (double)qq >= thr; }, key, c, q)) {
                if (!have || key > tau_key) { tau_key = key; kept = c; }
                have = true;
            }
        }
    }
    if (!have) return;                                        // nothing to cut (rounding left the sum below the threshold)
    const float tau_f = f32_key_value(tau_key);

    if (P.stats) {
        // ---- virtual mode: block sums of the verifier's statistics, restricted to x >= tau -------------------
        // (c, s) of a block: c = max * scale, s = sum 2^(x * scale - c); the maximum of the row is always kept, so
        // only the sums change.  One warp per block; a block whose maximum lies below tau gets 0.
        const float ctau = __fmul_rn(tau_f, scale2);
        float2* st = P.stats + (long long)row * P.nblk;
        for (int b = warp; b < P.nblk; b += kF32Threads / 32) {
            const float2 e = st[b];
            float sum = 0.f;
            if (e.x >= ctau && e.x > -INFINITY) {
                const int e0 = b * P.epb;
                const int cnt = (V - e0) < P.epb ? (V - e0) : P.epb;
                for (int i = lane; i < cnt; i += 32) {
                    const float x = __ldcg(&rowp[e0 + i]);
                    if (x >= tau_f) sum += ex2_approx(__fmaf_rn(x, scale2, -e.x));
                }
                sum = warp_sum_f32(sum);
            }
            if (lane == 0) st[b].y = sum;
        }
        if (tid == 0) {
            if (P.out_tau) P.out_tau[row] = tau_f;
            if (P.out_kept) P.out_kept[row] = (int32_t)kept;
        }
        return;
    }
    // ---- mask ---------------------------------------------------------------------------------------------------
    {
        int head = (int)(((16u - (unsigned)((uintptr_t)rowp & 15u)) & 15u) >> 2);
        if (head > V) head = V;
        const int nvec = (V - head) >> 2;
        float4* p = reinterpret_cast<float4*>(rowp + head);
        for (int c = tid; c < nvec; c += kF32Threads) {
            float4 v = p[c];
            const bool cut = v.x < tau_f || v.y < tau_f || v.z < tau_f || v.w < tau_f;
            if (cut) {
                v.x = v.x < tau_f ? -INFINITY : v.x; v.y = v.y < tau_f ? -INFINITY : v.y;
                v.z = v.z < tau_f ? -INFINITY : v.z; v.w = v.w < tau_f ? -INFINITY : v.w;
                p[c] = v;
            }
        }
        const int tail0 = head + 4 * nvec;
        for (int i = tid; i < head + (V - tail0); i += kF32Threads) {
            const int e = i < head ? i : tail0 + (i - head);
            if (rowp[e] < tau_f) rowp[e] = -INFINITY;
        }
    }
    if (tid == 0) {
        if (P.out_tau) P.out_tau[row] = tau_f;
        if (P.out_kept) P.out_kept[row] = (int32_t)kept;
    }
}

__global__ void __launch_bounds__(kF32Threads) truncate_f32_kernel(TruncF32Params P)
{
    extern __shared__ __align__(16) unsigned char f32_smem[];
    pdl_wait();
    truncate_row_f32(P, blockIdx.x, *reinterpret_cast<F32Shared*>(f32_smem));
}

int truncate_f32_launch(const TruncF32Params& P, cudaStream_t stream)
{
    static std::atomic<int> attr[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return DSPARK_ERR_CUDA; }
    if (!attr[dev].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(truncate_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(F32Shared)) != cudaSuccess)
            return launch_status();
        attr[dev].store(1, std::memory_order_release);
    }
    launch_pdl(truncate_f32_kernel, dim3(P.n_rows), dim3(kF32Threads), sizeof(F32Shared), stream, P);
    return launch_status();
}

// Used by the sampling verifier after its statistics pass on fp32 rows (virtual truncation: rows stay as they are).
int truncate_f32_virtual_launch(const void* target, long long stride_elems, int V, const int32_t* row_offsets, int R, int n_rows,
                                const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                                float* tau_rows, float2* stats_t, int nblk, int epb, cudaStream_t stream)
{
    TruncF32Params P;
    P.target = (float*)const_cast<void*>(target); P.stride = stride_elems; P.V = V;
    P.row_offsets = row_offsets; P.R = R; P.n_rows = n_rows;
    P.top_k = top_k; P.top_p = top_p; P.temperatures = temperatures; P.temperature = temperature;
    P.out_tau = tau_rows; P.out_kept = nullptr;
    P.stats = stats_t; P.nblk = nblk; P.epb = epb;
    return truncate_f32_launch(P, stream);
}

// dspark_truncate_target on fp32 rows (in place)
int truncate_f32_in_place(void* target, long long stride_elems, int V, const int32_t* row_offsets, int R, int n_rows,
                          const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                          float* out_tau, int32_t* out_kept, cudaStream_t stream)
{
    TruncF32Params P;
    P.target = (float*)target; P.stride = stride_elems; P.V = V;
    P.row_offsets = row_offsets; P.R = R; P.n_rows = n_rows;
    P.top_k = top_k; P.top_p = top_p; P.temperatures = temperatures; P.temperature = temperature;
    P.out_tau = out_tau; P.out_kept = out_kept;
    P.stats = nullptr; P.nblk = 0; P.epb = 0;
    return truncate_f32_launch(P, stream);
}

}  // namespace dspark
