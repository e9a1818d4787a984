// dspark_truncate_target: top-k / top-p truncation of the target rows of a ragged verification batch
// (per-request sampling parameters; Section 4.1 evaluates with the models' recommended sampling
// parameters).  The logits of the excluded tokens are set to -inf in place, so that softmax renormalises
// over the kept set S and the lossless verifier runs unchanged on the masked rows.
//   S = { v : x_v >= tau }  (a value cut: every token tied with the threshold is kept)
//   top-k first: tau_k = k-th largest logit; then top-p on the distribution renormalised over the top-k
//   set: walking the distinct values downwards, tau_p is the first value at which the cumulative mass
//   reaches top_p * Z_k; tau = max(tau_k, tau_p).
//
// bf16 rows only: a bf16 logit is a 16-bit key, so the threshold is found exactly on a histogram of the
// keys.  One CTA per row:
//   pass 0 (HBM)  row maximum on packed bf16 pairs, NaN / +inf detection; the first 192 KB of the row stay in
//                 shared memory for the later passes;
//   pass 1 (L2)   counts of the keys at distance d = key(max) - key(x) < 4096 in shared memory (integer
//                 atomics, the bulk of the row lies beyond and is only counted), and sum of 2^((x-m) s)
//                 over the whole row when top-p needs the full normaliser;
//   scan          per-key masses = count * exp((value - m) / T), summed in fp64: block-wide prefix sums over the
//                 window; further windows of 4096 keys only if the threshold lies beyond (flat rows);
//   pass 2 (L2)   masked write.
// Counts are integers, so the top-k part is exact; the top-p decision compares fp64 sums against
// top_p * Z and can differ from an fp64 reference only when the two sides agree to ~1e-6 of Z.
#include <cuda_bf16.h>
#include <math.h>

#include "common.cuh"

namespace dspark {

constexpr int kTruncThreads = 1024;              // one CTA per SM
constexpr int kTruncBins = 4096;                 // keys per window
constexpr int kBinsPerThread = kTruncBins / kTruncThreads;
constexpr int kUnroll = 4;                       // row vectors in flight per thread

struct TruncParams {
    unsigned char* target; long long stride_bytes; int V;
    const int32_t* row_offsets; int R, n_rows;
    const int32_t* top_k; const float* top_p; const float* temperatures; float temperature;
    float* out_tau; int32_t* out_kept; int32_t* dev_status;
    // virtual mode (inside the verifier): the row is not modified; its statistics blocks receive the sums
    // restricted to the kept set instead
    float2* stats; int nblk, epb;
    const int32_t* only_flagged;              // virtual mode: rows whose flag is 0 are somebody else's (NULL: all rows);
                                              // [n_rows] work counter, [n_rows + 1] number of flagged rows
};

__device__ __forceinline__ uint32_t key_of(uint32_t b) { return bf16_key(b); }
__device__ __forceinline__ float value_of_key(uint32_t k) { return bf16_key_value(k); }

// eight consecutive elements starting at element 8c; elements past V read as -inf
struct RowAccess {
    unsigned char* row; int V; bool vec;
    __device__ __forceinline__ uint4 load(int c) const
    {
        if (vec && 8 * c + 8 <= V) return *reinterpret_cast<const uint4*>(row + (size_t)c * 16);
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = 8 * c + 2 * i;
            const uint32_t lo = e < V ? reinterpret_cast<const unsigned short*>(row)[e] : 0xFF80u;
            const uint32_t hi = e + 1 < V ? reinterpret_cast<const unsigned short*>(row)[e + 1] : 0xFF80u;
            w[i] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    __device__ __forceinline__ void store(int c, uint4 v) const
    {
        if (vec && 8 * c + 8 <= V) { *reinterpret_cast<uint4*>(row + (size_t)c * 16) = v; return; }
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = 8 * c + 2 * i;
            if (e < V) reinterpret_cast<unsigned short*>(row)[e] = (unsigned short)(w[i] & 0xFFFFu);
            if (e + 1 < V) reinterpret_cast<unsigned short*>(row)[e + 1] = (unsigned short)(w[i] >> 16);
        }
    }
};

// Calls fn(c, v) for every 8-element chunk c of the row.  For 16-byte aligned rows the whole chunks are read by
// plain vector loads, kUnroll of them in flight per thread (no branch between the loads); the ragged last
// chunk and unaligned rows go through RowAccess::load.  The first kCacheChunks chunks of an aligned row are
// kept in shared memory: kFill reads them from global memory and stores them there, later passes (kFill
// false) read them back from shared memory and only the rest of the row from L2 / HBM.
constexpr int kCacheChunks = 12288;              // 192 KB: 98 304 of the 129 280 logits of a full-vocabulary row
template <bool kFill, typename F>
__device__ __forceinline__ void for_each_chunk(const RowAccess& A, uint4* cache, F fn)
{
    const int n_chunks = (A.V + 7) >> 3;
    if (!A.vec) {
        for (int c = threadIdx.x; c < n_chunks; c += kTruncThreads) fn(c, A.load(c));
        return;
    }
    const int n_full = A.V >> 3;
    const int n_cached = n_full < kCacheChunks ? n_full : kCacheChunks;
    const uint4* p = reinterpret_cast<const uint4*>(A.row);
    const uint4 fill = make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u);
    if (!kFill)
        for (int c = threadIdx.x; c < n_cached; c += kTruncThreads) fn(c, cache[c]);
    for (int c0 = (kFill ? 0 : n_cached) + threadIdx.x; c0 < n_full; c0 += kUnroll * kTruncThreads) {
        uint4 vv[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int c = c0 + u * kTruncThreads;
            vv[u] = c < n_full ? p[c] : fill;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int c = c0 + u * kTruncThreads;
            if (c < n_full) {
                if (kFill && c < n_cached) cache[c] = vv[u];
                fn(c, vv[u]);
            }
        }
    }
    if (n_full < n_chunks && threadIdx.x == 0) fn(n_full, A.load(n_full));
}

__device__ __forceinline__ double block_sum_f64(double x, double* s_tmp)
{
    x = warp_sum_f64(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_tmp[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x < 32) {
        const double t = warp_sum_f64(threadIdx.x < kTruncThreads / 32 ? s_tmp[threadIdx.x] : 0.0);
        if (threadIdx.x == 0) s_tmp[0] = t;
    }
    __syncthreads();
    return s_tmp[0];
}

__device__ void truncate_row(const TruncParams& P, const int row, uint4* cache)
{
    __shared__ unsigned int bins[kTruncBins];
    __shared__ double s_tmp[kTruncThreads / 32];
    __shared__ double s_scan[kTruncThreads / 32];
    __shared__ unsigned long long s_scan_c[kTruncThreads / 32];
    __shared__ unsigned long long s_tot_c;
    __shared__ double s_tot_m;
    __shared__ int s_req, s_flag, s_hit;
    __shared__ unsigned int s_max;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        int lo = 0, hi = P.R;                               // largest r with row_offsets[r] <= row
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (P.row_offsets[mid] <= row) lo = mid; else hi = mid;
        }
        const int n = P.row_offsets[P.R];
        s_req = (row < n && row < P.n_rows && row >= P.row_offsets[0]) ? lo : -1;
        s_flag = 0; s_max = 0u; s_hit = 0x7fffffff;
    }
    __syncthreads();
    const int r = s_req;
    if (r < 0) return;
    if (P.only_flagged && !P.only_flagged[row]) return;
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

    RowAccess A;
    A.row = P.target + (long long)row * P.stride_bytes;
    A.V = V;
    A.vec = (((uintptr_t)A.row) & 15u) == 0;

    // ---- pass 0: maximum key, NaN / +inf ------------------------------------------------------------
    uint32_t kmax = 0u;
    bool bad = false;
    const uint32_t neg_inf2 = 0xFF80FF80u;
    __nv_bfloat162 mx2 = *reinterpret_cast<const __nv_bfloat162*>(&neg_inf2);
    for_each_chunk<true>(A, cache, [&](int, uint4 v) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)                         // one packed, NaN-propagating maximum per pair
            mx2 = __hmax2_nan(mx2, *reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    });
    {
        const uint32_t mb = *reinterpret_cast<const uint32_t*>(&mx2);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint32_t b = (mb >> (16 * h)) & 0xFFFFu;
            bad |= (b & 0x7FFFu) > 0x7F80u;                  // NaN
            kmax = max(kmax, key_of(b));
        }
    }
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    if (lane == 0) atomicMax(&s_max, kmax);
    if (bad) s_flag = 1;
    __syncthreads();
    kmax = s_max;
    const float m = value_of_key(kmax);
    if (s_flag || m == INFINITY || m == -INFINITY) return;   // left as it is: the verifier reports such rows

    const float inv_Tf = 1.f / T;
    const float scale2 = (float)(1.4426950408889634 / (double)T);

    // window w of the key space: distances [win_start(w), win_start(w) + win_size(w)) below the maximum.
    // Window 0 ends at the key of m - 8 T (at most 4096 keys): a token below that carries less than e^-8 of
    // the maximum's mass, so for a peaked row the threshold lies inside and only the few tokens of the tail
    // cost a shared-memory atomic; the later windows hold 4096 keys each.
    uint32_t first_size = kTruncBins;
    {
        const __nv_bfloat16 lo = __float2bfloat16_rd(m - 8.f * T);
        const uint32_t klo = key_of((uint32_t)__bfloat16_as_ushort(lo));
        if (klo <= kmax && kmax - klo + 1u < (uint32_t)kTruncBins) first_size = kmax - klo + 1u;
    }
    auto win_start = [&](int w) -> uint32_t { return w == 0 ? 0u : first_size + (uint32_t)(w - 1) * kTruncBins; };
    auto win_size = [&](int w) -> uint32_t { return w == 0 ? first_size : (uint32_t)kTruncBins; };
    auto win_of = [&](long long d) -> int { return d < (long long)first_size ? 0 : 1 + (int)((d - first_size) / kTruncBins); };
    int cur_window = -1;
    double z_all = 0.0;                                     // sum over the whole row (first build only)
    auto build_window = [&](int w, bool want_z) {
        if (w == cur_window) return;
        for (int i = tid; i < kTruncBins; i += kTruncThreads) bins[i] = 0u;
        __syncthreads();
        uint64_t za = pack2(0.f, 0.f), zb = pack2(0.f, 0.f);
        const uint64_t sc2 = pack2(scale2, scale2), no2 = pack2(-m * scale2, -m * scale2);
        const uint32_t base = win_start(w), size = win_size(w);
        // lowest value of the window as a packed operand: pairs entirely below it (almost all of the row)
        // cost one packed compare
        const uint32_t last = base + size - 1;
        const __nv_bfloat16 cut_b = __float2bfloat16(last >= kmax ? -INFINITY : value_of_key(kmax - last));
        const __nv_bfloat162 cut2 = __halves2bfloat162(cut_b, cut_b);
        for_each_chunk<false>(A, cache, [&](int c, uint4 v) {
            const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (__hge2_mask(*reinterpret_cast<const __nv_bfloat162*>(&wd[i]), cut2)) {
                    const uint32_t b0 = wd[i] & 0xFFFFu, b1 = wd[i] >> 16;
                    const uint32_t d0 = kmax - key_of(b0) - base, d1 = kmax - key_of(b1) - base;   // wraps above the window
                    const int e = 8 * c + 2 * i;            // padding past V is not a token
                    if (d0 < size && e < V) atomicAdd(&bins[d0], 1u);
                    if (d1 < size && e + 1 < V) atomicAdd(&bins[d1], 1u);
                }
                if (want_z) {
                    float t0, t1;
                    unpack2(fma2(pack2(bf16lo(wd[i]), bf16hi(wd[i])), sc2, no2), t0, t1);
                    if (i & 1) zb = add2(zb, pack2(ex2_approx(t0), ex2_approx(t1)));
                    else za = add2(za, pack2(ex2_approx(t0), ex2_approx(t1)));
                }
            }
        });
        if (want_z) {
            float s0, s1;
            unpack2(add2(za, zb), s0, s1);
            z_all = block_sum_f64((double)s0 + (double)s1, s_tmp);
        }
        __syncthreads();
        cur_window = w;
    };
    // prefix sums of counts and masses over the current window; thread t owns bins [8t, 8t + 8)
    unsigned int cnt[kBinsPerThread];
    double mass[kBinsPerThread];
    unsigned long long cnt_excl = 0ull;                     // tokens at smaller distance inside the window
    double mass_excl = 0.0;
    unsigned long long win_cnt = 0ull;
    double win_mass = 0.0;
    int scanned_window = -1;
    auto scan_window = [&](int w) {
        if (w == scanned_window) return;                    // the prefix sums of this window are still in the registers
        scanned_window = w;
        unsigned long long lc = 0ull;
        double lm = 0.0;
#pragma unroll
        for (int j = 0; j < kBinsPerThread; ++j) {
            const int d = tid * kBinsPerThread + j;
            cnt[j] = bins[d];
            const long long key = (long long)kmax - ((long long)win_start(w) + d);
            // fp32 exponential of an exact difference (fp64 exponentials are far too slow here); its ~1e-7
            // relative error is what the 1e-6 agreement quoted above allows for
            mass[j] = (cnt[j] && key >= 0) ? (double)cnt[j] * (double)expf((value_of_key((uint32_t)key) - m) * inv_Tf) : 0.0;
            lc += cnt[j];
            lm += mass[j];
        }
        unsigned long long ic = lc;
        double im = lm;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long nc = __shfl_up_sync(0xffffffffu, ic, o);
            const double nm = __shfl_up_sync(0xffffffffu, im, o);
            if (lane >= o) { ic += nc; im += nm; }
        }
        __syncthreads();
        if (lane == 31) { s_scan_c[warp] = ic; s_scan[warp] = im; }
        __syncthreads();
        if (warp == 0) {                                    // one warp turns the 32 warp totals into exclusive prefixes
            const unsigned long long wc = lane < kTruncThreads / 32 ? s_scan_c[lane] : 0ull;
            const double wm = lane < kTruncThreads / 32 ? s_scan[lane] : 0.0;
            unsigned long long pc = wc;
            double pm = wm;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long nc = __shfl_up_sync(0xffffffffu, pc, o);
                const double nm = __shfl_up_sync(0xffffffffu, pm, o);
                if (lane >= o) { pc += nc; pm += nm; }
            }
            if (lane < kTruncThreads / 32) { s_scan_c[lane] = pc - wc; s_scan[lane] = pm - wm; }
            if (lane == 31) { s_tot_c = pc; s_tot_m = pm; }
        }
        __syncthreads();
        cnt_excl = s_scan_c[warp] + (ic - lc);
        mass_excl = s_scan[warp] + (im - lm);
        win_cnt = s_tot_c;
        win_mass = s_tot_m;
        __syncthreads();                                    // s_scan is reused by through()
    };
    // first bin of the current window (scanned state) that satisfies pred(count_through, mass_through); the
    // smallest distance over the block, or -1
    auto first_hit = [&](auto pred, unsigned long long cnt_before, double mass_before) -> int {
        if (tid == 0) s_hit = 0x7fffffff;
        __syncthreads();
        unsigned long long c = cnt_before + cnt_excl;
        double q = mass_before + mass_excl;
        int mine = 0x7fffffff;
#pragma unroll
        for (int j = 0; j < kBinsPerThread; ++j) {
            c += cnt[j];
            q += mass[j];
            if (mine == 0x7fffffff && cnt[j] && pred(c, q)) mine = tid * kBinsPerThread + j;
        }
        mine = __reduce_min_sync(0xffffffffu, mine);
        if (lane == 0 && mine != 0x7fffffff) atomicMin(&s_hit, mine);
        __syncthreads();
        const int h = s_hit;
        __syncthreads();
        return h == 0x7fffffff ? -1 : h;
    };
    // count and mass of the window up to and including bin d (scanned state)
    auto through = [&](int d, unsigned long long& c_out, double& m_out) {
        __syncthreads();
        if (d / kBinsPerThread == tid) {
            unsigned long long c = cnt_excl;
            double q = mass_excl;
            for (int j = 0; j <= d % kBinsPerThread; ++j) { c += cnt[j]; q += mass[j]; }
            s_scan_c[0] = c; s_scan[0] = q;
        }
        __syncthreads();
        c_out = s_scan_c[0]; m_out = s_scan[0];
        __syncthreads();
    };
    const int n_windows = win_of((long long)kmax) + 1;      // keys 0 .. kmax

    // ---- top-k: distance of the k-th largest key, size and mass of the top-k set --------------------------
    long long dist_k = -1;                                  // -1: no top-k cut
    unsigned long long kept = (unsigned long long)V;
    double Zk = 0.0;
    build_window(0, use_p && !use_k);
    if (use_k) {
        unsigned long long c_before = 0ull;
        double m_before = 0.0;
        for (int w = 0; w < n_windows; ++w) {
            build_window(w, false);
            scan_window(w);
            const unsigned long long need = (unsigned long long)k;
            const int h = first_hit([&](unsigned long long c, double) { return c >= need; }, c_before, m_before);
            if (h >= 0) {
                unsigned long long c; double q;
                through(h, c, q);
                dist_k = (long long)win_start(w) + h;
                kept = c_before + c;
                Zk = m_before + q;
                break;
            }
            c_before += win_cnt;
            m_before += win_mass;
        }
    } else {
        Zk = z_all;
    }
    // ---- top-p inside the top-k set -------------------------------------------------------------------------
    long long dist = dist_k;
    if (use_p) {
        long long dist_p = -1;
        if (!(pf > 0.f)) {
            dist_p = 0;                                     // only the maximum
            build_window(0, false);
            scan_window(0);
            unsigned long long c; double q;
            through(0, c, q);
            kept = c;
        } else {
            const double thr = (double)pf * Zk;
            unsigned long long c_before = 0ull;
            double m_before = 0.0;
            const int last_w = dist_k >= 0 ? win_of(dist_k) : n_windows - 1;
            for (int w = 0; w <= last_w; ++w) {
                build_window(w, false);
                scan_window(w);
                const int h = first_hit([&](unsigned long long, double q) { return q >= thr; }, c_before, m_before);
                if (h >= 0) {
                    unsigned long long c; double q;
                    through(h, c, q);
                    dist_p = (long long)win_start(w) + h;
                    if (dist_k < 0 || dist_p < dist_k) kept = c_before + c;
                    break;
                }
                c_before += win_cnt;
                m_before += win_mass;
            }
        }
        if (dist_p >= 0 && (dist < 0 || dist_p < dist)) dist = dist_p;
    }
    if (dist < 0) return;                                   // nothing to cut (rounding left the sum below the threshold)
    const uint32_t tau_key = kmax - (uint32_t)dist;
    if (P.stats) {
        // ---- virtual mode: block sums of the verifier's statistics, restricted to x >= tau --------------------
        // (c, s) of a block: c = max * scale, s = sum 2^(x * scale - c); the maximum of the row is always
        // kept, so only the sums change.  One warp per block; a block whose maximum lies below tau gets 0.
        const float tau_f = value_of_key(tau_key);
        const float ctau = __fmul_rn(tau_f, scale2);
        float2* st = P.stats + (long long)row * P.nblk;
        const int chunks_per_block = P.epb >> 3;
        const int n_full = V >> 3, n_cached = (A.vec && n_full < kCacheChunks) ? n_full : (A.vec ? kCacheChunks : 0);
        for (int b = warp; b < P.nblk; b += kTruncThreads / 32) {
            const float2 e = st[b];
            float sum = 0.f;
            if (e.x >= ctau && e.x > -INFINITY) {
                const uint64_t sc2 = pack2(scale2, scale2), nc2 = pack2(-e.x, -e.x);
                uint64_t acc = pack2(0.f, 0.f);
                for (int i = lane; i < chunks_per_block; i += 32) {
                    const int c = b * chunks_per_block + i;
                    if (c * 8 >= V) break;
                    const uint4 v = c < n_cached ? cache[c] : A.load(c);
                    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float x0 = bf16lo(w[q]), x1 = bf16hi(w[q]);
                        x0 = x0 >= tau_f ? x0 : -INFINITY;
                        x1 = x1 >= tau_f ? x1 : -INFINITY;
                        float t0, t1;
                        unpack2(fma2(pack2(x0, x1), sc2, nc2), t0, t1);
                        acc = add2(acc, pack2(ex2_approx(t0), ex2_approx(t1)));
                    }
                }
                float a0, a1;
                unpack2(acc, a0, a1);
                sum = warp_sum_f32(a0 + a1);
            }
            if (lane == 0) st[b].y = sum;
        }
        if (tid == 0) {
            if (P.out_tau) P.out_tau[row] = tau_f;
            if (P.out_kept) P.out_kept[row] = (int32_t)kept;
        }
        return;
    }
    // ---- pass 2: mask ------------------------------------------------------------------------------------------
    const __nv_bfloat16 tau_b = __float2bfloat16(value_of_key(tau_key));
    const __nv_bfloat162 tau2 = __halves2bfloat162(tau_b, tau_b);
    for_each_chunk<false>(A, cache, [&](int c, uint4 v) {
        uint32_t w[4] = {v.x, v.y, v.z, v.w};
        bool changed = false;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // x < tau as a packed floating-point compare (-0 equals +0, as in the keys): all-ones half-words
            const uint32_t lt = __hlt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&w[i]), tau2);
            const uint32_t nw = (w[i] & ~lt) | (neg_inf2 & lt);
            changed |= nw != w[i];
            w[i] = nw;
        }
        if (changed) A.store(c, make_uint4(w[0], w[1], w[2], w[3]));
    });
    if (tid == 0) {
        if (P.out_tau) P.out_tau[row] = value_of_key(tau_key);
        if (P.out_kept) P.out_kept[row] = (int32_t)kept;
    }
}

// One CTA per row.  (A persistent CTA per SM walking its rows, with or without a bulk prefetch of the next row
// into L2, measured 25 % slower: rows take different times and the hardware's CTA scheduler balances them.)
__global__ void __launch_bounds__(kTruncThreads) truncate_kernel(TruncParams P)
{
    extern __shared__ uint4 cache[];                        // kCacheChunks vectors of the row
    pdl_wait();
    truncate_row(P, blockIdx.x, cache);
}

// The verifier's fallback: a few CTAs walk the rows and search only those that the streamed search flagged
// (usually none, and then this costs a glance at the flags).
__global__ void __launch_bounds__(kTruncThreads) truncate_flagged_kernel(TruncParams P)
{
    extern __shared__ uint4 cache[];
    __shared__ int s_row;
    pdl_wait();
    int* counter = const_cast<int*>(P.only_flagged) + P.n_rows;     // zeroed with the flags
    if (P.only_flagged[P.n_rows + 1] == 0) return;                  // nobody flagged a row: the usual case
    for (;;) {
        // rows are handed out one at a time (they take very different times); unflagged ones are skipped here
        if (threadIdx.x == 0) {
            int row;
            do { row = atomicAdd(counter, 1); } while (row < P.n_rows && !P.only_flagged[row]);
            s_row = row;
        }
        __syncthreads();
        const int row = s_row;
        if (row >= P.n_rows) return;
        truncate_row(P, row, cache);
        __syncthreads();                                    // the shared state (and s_row) is reused by the next row
    }
}

static int launch_truncate(const TruncParams& P, cudaStream_t stream)
{
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    const size_t smem = (size_t)kCacheChunks * sizeof(uint4);
    if (!attr_set[dev & 63]) {
        if (cudaFuncSetAttribute(truncate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
            cudaFuncSetAttribute(truncate_flagged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return launch_status();
        attr_set[dev & 63] = true;
    }
    if (P.only_flagged) {
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        launch_pdl(truncate_flagged_kernel, dim3(P.n_rows < sms ? P.n_rows : sms), dim3(kTruncThreads), smem, stream, P);
    } else {
        launch_pdl(truncate_kernel, dim3(P.n_rows), dim3(kTruncThreads), smem, stream, P);
    }
    return launch_status();
}

// Used by the sampling verifier after its statistics pass (virtual truncation: rows stay as they are).
int truncate_virtual_launch(const void* target, long long stride_bytes, int V, const int32_t* row_offsets, int R, int n_rows,
                            const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                            float* tau_rows, float2* stats_t, int nblk, int epb, const int32_t* only_flagged,
                            cudaStream_t stream)
{
    TruncParams P;
    P.target = (unsigned char*)const_cast<void*>(target); P.stride_bytes = stride_bytes; P.V = V;
    P.row_offsets = row_offsets; P.R = R; P.n_rows = n_rows;
    P.top_k = top_k; P.top_p = top_p; P.temperatures = temperatures; P.temperature = temperature;
    P.out_tau = tau_rows; P.out_kept = nullptr; P.dev_status = nullptr;
    P.stats = stats_t; P.nblk = nblk; P.epb = epb; P.only_flagged = only_flagged;
    return launch_truncate(P, stream);
}

}  // namespace dspark

using namespace dspark;

extern "C" {

int dspark_truncate_target(void* target_logits, int dtype, int64_t target_row_stride, int V,
                           const int32_t* row_offsets, int R, int n_rows,
                           const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                           float* out_tau, int32_t* out_kept, int32_t* dev_status, void* stream)
{
    if (!target_logits || !row_offsets || R < 1 || n_rows < 1 || V < 1 || target_row_stride < V) return DSPARK_ERR_INVALID_ARG;
    if (dtype != DSPARK_BF16 && dtype != DSPARK_F32) return DSPARK_ERR_INVALID_ARG;
    if (!top_k && !top_p) return DSPARK_OK;
    if (!temperatures && (!(temperature > 0.f) || isinf(temperature))) return DSPARK_ERR_INVALID_ARG;
    if (dtype == DSPARK_F32)                                 // 32-bit patterns: a descent instead of a key window
        return truncate_f32_in_place(target_logits, (long long)target_row_stride, V, row_offsets, R, n_rows, top_k, top_p,
                                     temperature, temperatures, out_tau, out_kept, (cudaStream_t)stream);
    TruncParams P;
    P.target = (unsigned char*)target_logits; P.stride_bytes = (long long)target_row_stride * 2; P.V = V;
    P.row_offsets = row_offsets; P.R = R; P.n_rows = n_rows;
    P.top_k = top_k; P.top_p = top_p; P.temperatures = temperatures; P.temperature = temperature;
    P.out_tau = out_tau; P.out_kept = out_kept; P.dev_status = dev_status;
    P.stats = nullptr; P.nblk = 0; P.epb = 0; P.only_flagged = nullptr;
    return launch_truncate(P, (cudaStream_t)stream);
}

}  // extern "C"
