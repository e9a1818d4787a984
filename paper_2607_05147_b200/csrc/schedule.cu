// dspark_schedule: the hardware-aware prefix scheduler (Algorithm 1; Sections 3.2.2 and 5.2).
//
// Algorithm 1 sorts all candidates (r, j) by survival probability and walks the sorted
// list.  Here nothing is sorted: every request's survival products are already in
// descending order (a_{r,j} is non-increasing in j), so the position of a candidate in the
// global order, and the exact expected-accept mass admitted up to it, are sums over all
// requests of one binary search each.  Three kernels on the caller's stream:
//   prep   one warp per request: a_{r,j} as a left-to-right fp32 product, per-tile inclusive
//          prefix sums of the fixed-point mass (units of 2^-40, exact integers);
//   select one CTA: histogram of the survival bit patterns, the threshold bin for the admission
//          cap (budget - R), compaction of the candidates that can possibly be admitted;
//   rank   one CTA per tile of 32 such candidates, 32 warps each searching a slice of all tiles
//          (tiles are loaded coalesced and searched with warp shuffles): candidate c gets
//          rank_c = #{keys <= key_c} and T_c = R*2^40 + mass of those keys, scattered to
//          by-rank arrays; the CTA that finishes last (a ticket counter, nobody waits) then
//          walks the path: Theta_i = T_i * SPS(R + i), stop rule, lengths, offsets.
// Integer sums are associative, so the result is bit-identical to the sequential walk.
#include "common.cuh"

namespace dspark {

constexpr int kSchedThreads = 1024;
constexpr int kPrepThreads = 128;
constexpr int kSmemLenCap = 4096;
constexpr int kModeAsync = 3;                 // internal: global search for the next K, top-K with the stored K

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
    // geometry: gpad = positions per request after padding (power of two <= 32, or a multiple of 32),
    // seg = min(gpad, 32) entries per sorted segment, n_tiles tiles of 32 entries
    int gpad, seg, n_tiles, R_pad;
    // workspace
    uint32_t* akey;                 // [n_tiles*32] fp32 bits of a_{r,j}, 0 where not a candidate
    unsigned long long* pfix;       // [n_tiles*32] inclusive prefix of fix40(a) inside the segment
    int32_t* cnt;                   // [R] candidates of request r (bit 30: a confidence was clamped)
    unsigned long long* t_by_rank;  // [N+1] T_i
    int32_t* owner_by_rank;         // [N+1] request of the i-th admitted candidate
    int32_t* async_state;           // asynchronous mode: {step, K slot 0, K slot 1} (caller-owned, device)
    int32_t* cand;                  // [n_tiles*32] entry indices of the candidates worth ranking
    int* ticket;                    // [0] finished rank CTAs, [1] number of entries in cand (select kernel)
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

// ---- S1: survival products (fp32, left to right), segment-local prefix sums ----------------
// One warp per 32/seg requests (seg = entries per segment): confidences are loaded coalesced,
// the product chain runs in request order through warp shuffles (every lane follows the same
// chain and keeps the value of its own position), the mass prefix is a segmented warp scan.
__global__ void __launch_bounds__(kPrepThreads) sched_prep_kernel(SchedParams P)
{
    pdl_wait();
    if (!P.cand && blockIdx.x == 0 && threadIdx.x == 0) P.ticket[0] = 0;   // else the select kernel does it
    const int lane = threadIdx.x & 31;
    const int wid = blockIdx.x * (kPrepThreads / 32) + (threadIdx.x >> 5);
    const int gamma = P.gamma, gpad = P.gpad, seg = P.seg;
    const int req_per_warp = 32 / seg;
    const int chunks = gpad / seg;                       // 32-entry tiles per request (1 when gpad <= 32)
    const int sub = lane / seg, k_in_seg = lane - sub * seg;
    const int r = wid * req_per_warp + sub;
    if (wid * req_per_warp >= P.R_pad) return;
    const bool real = r < P.R;
    int lim = 0;
    if (real) {
        lim = gamma;
        if (P.draft_len) { lim = P.draft_len[r]; lim = lim < 0 ? 0 : (lim > gamma ? gamma : lim); }
    }
    float a_run = 1.0f;
    bool dead = false;
    int clamped = 0, n = 0;
    for (int q = 0; q < chunks; ++q) {
        const int j = q * seg + k_in_seg;
        float c = 0.0f;
        if (real && j < lim) c = P.conf[(size_t)r * gamma + j];
        float mine = 0.0f;
        for (int k = 0; k < seg; ++k) {
            const float ck = __shfl_sync(0xffffffffu, c, sub * seg + k);
            if (q * seg + k >= lim) dead = true;
            if (!dead) {                                  // only confidences actually multiplied are judged
                a_run = __fmul_rn(a_run, sanitize_conf(ck, clamped));
                if (!(a_run > 0.0f)) dead = true;
            }
            if (k == k_in_seg) mine = dead ? 0.0f : a_run;
        }
        unsigned long long pre = mine > 0.0f ? fix40(mine) : 0ull;
        for (int o = 1; o < seg; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, pre, o, seg);
            if (k_in_seg >= o) pre += up;
        }
        const unsigned live = __ballot_sync(0xffffffffu, mine > 0.0f);
        const unsigned segmask = (seg == 32) ? 0xffffffffu : (((1u << seg) - 1u) << (sub * seg));
        n += __popc(live & segmask);
        const size_t e = (size_t)r * gpad + j;
        P.akey[e] = __float_as_uint(mine);
        P.pfix[e] = pre;
        if (real && j < gamma && P.out_surv) P.out_surv[(size_t)r * gamma + j] = mine;
    }
    if (real && k_in_seg == 0) P.cnt[r] = n | (clamped ? (1 << 30) : 0);
}

// ---- Candidates worth ranking ---------------------------------------------------------------
// At most cap = budget - R candidates can be admitted, so only the cap largest survival values
// need a rank.  One CTA histograms the fp32 bit patterns (32 bins per binade, larger a = lower
// bin), finds the first bin at which the running count reaches the cap, and compacts the entry
// indices of all candidates up to that bin (the top-M set, M >= min(cap, |E|)).
constexpr int kSelectBins = 4096;
__device__ __forceinline__ int select_bin(uint32_t a_bits) { return (int)((0x3F800000u - a_bits) >> 18); }

__global__ void __launch_bounds__(kSchedThreads, 1) sched_select_kernel(SchedParams P)
{
    __shared__ int s_hist[kSelectBins];
    __shared__ int s_warp_tot[32];
    __shared__ int s_bin_star, s_base;
    pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_entries = P.n_tiles * 32;
    long long cap = (long long)P.budget - (long long)P.R;
    if (cap < 0) cap = 0;
    for (int b = tid; b < kSelectBins; b += kSchedThreads) s_hist[b] = 0;
    if (tid == 0) { s_bin_star = kSelectBins - 1; s_base = 0; P.ticket[0] = 0; }
    __syncthreads();
    for (int e = tid; e < n_entries; e += kSchedThreads) {
        const uint32_t a = P.akey[e];
        if (a) atomicAdd(&s_hist[select_bin(a)], 1);
    }
    __syncthreads();
    // first bin whose inclusive prefix count reaches the cap (4 consecutive bins per thread)
    {
        int c[4], sum = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) { c[k] = s_hist[tid * 4 + k]; sum += c[k]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        if (lane == 31) s_warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int t = s_warp_tot[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const int u = __shfl_up_sync(0xffffffffu, t, o); if (lane >= o) t += u; }
            s_warp_tot[lane] = t;
        }
        __syncthreads();
        long long run = (long long)(incl - sum) + (warp > 0 ? s_warp_tot[warp - 1] : 0);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const long long before = run;
            run += c[k];
            if (before < cap && run >= cap) s_bin_star = tid * 4 + k;      // exactly one bin crosses the cap
        }
    }
    __syncthreads();
    const int bin_star = s_bin_star;
    // compaction: each warp reserves room with one shared-memory atomic (the order of cand does not
    // matter: every candidate is ranked independently of the others)
    for (int base = 0; base < n_entries; base += kSchedThreads) {
        const int e = base + tid;
        const uint32_t a = e < n_entries ? P.akey[e] : 0u;
        const bool keep = a != 0u && select_bin(a) <= bin_star;
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        int off = 0;
        if (lane == 0 && m) off = atomicAdd(&s_base, __popc(m));
        off = __shfl_sync(0xffffffffu, off, 0);
        if (keep) P.cand[off + __popc(m & ((1u << lane) - 1u))] = e;
    }
    __syncthreads();
    if (tid == 0) P.ticket[1] = s_base;
}

// ---- S2 + S3 without a sort: rank and admitted mass of every candidate ------------------------
// key order: a descending, then position ascending, then request ascending.
__device__ __forceinline__ bool key_le(uint32_t a2, int j2, int r2, uint32_t a1, int j1, int r1)
{
    // is key (a2, j2, r2) at or before key (a1, j1, r1) in the admission order?
    return a2 > a1 || (a2 == a1 && (j2 < j1 || (j2 == j1 && r2 <= r1)));
}

// Searches one sorted segment (SEG entries held one per lane starting at lane `base`, the first
// `cnt` of them candidates) for the number of entries at or before my key.  The common case needs
// only the strict comparison on a; a warp that sees an exact tie redoes the search with the full key.
template <int SEG>
__device__ __forceinline__ int segment_search(uint32_t ak, int base, int cnt, uint32_t a1, int j1, int r1,
                                              int j_base, int r2)
{
    // entries that are not candidates hold the key 0 and follow the candidates, so "a2 > a1" alone finds
    // the count: a halving search over places 0 .. SEG-1, then one look at the place it stopped at
    int pos = 0;
#pragma unroll
    for (int step = SEG / 2; step >= 1; step >>= 1) {
        const uint32_t a2 = __shfl_sync(0xffffffffu, ak, base + pos + step - 1);
        if (a2 > a1) pos += step;
    }
    if (__shfl_sync(0xffffffffu, ak, base + pos) > a1) ++pos;
    const uint32_t a_next = __shfl_sync(0xffffffffu, ak, base + (pos < SEG ? pos : SEG - 1));
    if (__any_sync(0xffffffffu, pos < cnt && a_next == a1)) {
        pos = 0;
#pragma unroll
        for (int step = SEG; step >= 1; step >>= 1) {
            const int probe = pos + step;
            const uint32_t a2 = __shfl_sync(0xffffffffu, ak, base + (probe <= SEG ? probe : SEG) - 1);
            if (probe <= cnt && key_le(a2, j_base + probe - 1, r2, a1, j1, r1)) pos = probe;
        }
    }
    return pos;
}

__device__ void sched_final_stage(const SchedParams& P);

template <int SEG>
__global__ void __launch_bounds__(kSchedThreads, 1) sched_rank_kernel(SchedParams P)
{
    constexpr int kWarps = kSchedThreads / 32;
    constexpr int kSegsPerTile = 32 / SEG;
    __shared__ unsigned int s_rank[kWarps][32];
    __shared__ unsigned long long s_mass[kWarps][32];
    __shared__ int s_is_last;
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tiles_per_req = P.gpad > 32 ? P.gpad / 32 : 1;
    const int n_cand = P.cand ? __ldcg(&P.ticket[1]) : P.n_tiles * 32;   // no selection: every entry

  for (int ctile = blockIdx.x; ctile * 32 < n_cand; ctile += gridDim.x) {
    // my candidate (one of the compacted entries worth ranking)
    const int ci = ctile * 32 + lane;
    const int e = ci < n_cand ? (P.cand ? __ldcg(&P.cand[ci]) : ci) : 0;   // flat padded entry index
    const uint32_t a1 = ci < n_cand ? P.akey[e] : 0u;
    const int r1 = e / P.gpad;
    const int j1 = e - r1 * P.gpad;

    unsigned int rank = 0;
    unsigned long long mass = 0ull;
    // the tiles of this warp, four at a time: their loads are issued together (one trip to the L2
    // instead of four in a row), then searched one after the other
    constexpr int kBatch = 4;
    for (int t0 = warp; t0 < P.n_tiles; t0 += kBatch * kWarps) {
        uint32_t akv[kBatch];
        unsigned long long pfv[kBatch];
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const int t = t0 + q * kWarps;
            akv[q] = t < P.n_tiles ? P.akey[t * 32 + lane] : 0u;
            pfv[q] = t < P.n_tiles ? P.pfix[t * 32 + lane] : 0ull;
        }
#pragma unroll
        for (int q = 0; q < kBatch; ++q) {
            const int t = t0 + q * kWarps;
            const uint32_t ak = akv[q];
            const unsigned long long pf = pfv[q];
            const unsigned valid = __ballot_sync(0xffffffffu, ak != 0u);
            if (valid == 0u) continue;                    // also a tile beyond the last one
#pragma unroll
            for (int sgi = 0; sgi < kSegsPerTile; ++sgi) {
                const int base = sgi * SEG;
                const unsigned segmask = (SEG == 32) ? 0xffffffffu : (((1u << SEG) - 1u) << base);
                const int cnt = __popc(valid & segmask);      // candidates form a prefix of the segment
                // a padded block shorter than a tile is exactly one segment (gpad == SEG): no runtime division
                const int r2 = SEG < 32 ? (t * 32 + base) / SEG : (tiles_per_req == 1 ? t : t / tiles_per_req);
                const int j_base = SEG < 32 ? 0 : (t - r2 * tiles_per_req) * 32;
                const int pos = segment_search<SEG>(ak, base, cnt, a1, j1, r1, j_base, r2);
                const unsigned long long m = __shfl_sync(0xffffffffu, pf, base + (pos > 0 ? pos - 1 : 0));
                if (pos > 0) { rank += (unsigned)pos; mass += m; }
            }
        }
    }
    s_rank[warp][lane] = rank;
    s_mass[warp][lane] = mass;
    __syncthreads();
    if (warp == 0 && a1 != 0u) {
        unsigned int rk = 0;
        unsigned long long ms = (unsigned long long)P.R << 40;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) { rk += s_rank[w][lane]; ms += s_mass[w][lane]; }
        // rk is the 1-based place of this candidate on the admission path, ms is T at that place
        P.t_by_rank[rk] = ms;
        P.owner_by_rank[rk] = r1;
    }
    __syncthreads();                           // s_rank / s_mass are reused by the next candidate tile
  }
    // the CTA that finishes last walks the path (no CTA ever waits for another)
    if (threadIdx.x == 0) {
        __threadfence();
        s_is_last = (atomicAdd(P.ticket, 1) == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    sched_final_stage(P);
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

// ---- S3 + S4: Theta path, stop rule, lengths, offsets (one CTA of 1024 threads) -------------
__device__ void sched_final_stage(const SchedParams& P)
{
    __shared__ unsigned long long s_warp_tot[32];
    __shared__ unsigned long long s_carry, s_T_best;
    __shared__ double s_theta_best;
    __shared__ int s_first_bad, s_istar, s_nE, s_status, s_done;
    __shared__ double s_red_theta[32];
    __shared__ int s_red_i[32];
    __shared__ unsigned long long s_red_T[32];

    __shared__ int s_len[kSmemLenCap];        // per-request lengths while R fits (else global out_len)
    const int tid = threadIdx.x;
    const int R = P.R;
    const bool len_in_smem = R <= kSmemLenCap;
    int* len_arr = len_in_smem ? s_len : P.out_len;
    if (tid == 0) { s_nE = 0; s_status = 0; s_first_bad = 0x7fffffff; s_done = 0; }
    // This stage is a chain of short steps, each of which would wait for its own trip to the L2: ask now
    // for what the first round of the path walk and of the length count will read (place tid + 1 on the
    // path; the by-rank arrays have an entry for every place, what lies beyond the admitted count is
    // loaded but never used).
    const int mt = P.max_tokens;
    const int n_places = P.n_tiles * 32;
    const int i_first = tid + 1;
    unsigned long long pre_Ti = 0ull, pre_Tp = 0ull;
    int pre_owner = 0;
    if (i_first <= n_places) {
        pre_Ti = P.t_by_rank[i_first];
        if (i_first > 1) pre_Tp = P.t_by_rank[i_first - 1];
        pre_owner = P.owner_by_rank[i_first];
    }
    const double pre_tab = P.table[R + i_first < mt ? R + i_first : mt];
    const double pre_tab_prev = P.table[R + i_first - 1 < mt ? R + i_first - 1 : mt];
    __syncthreads();
    {
        int n = 0, cl = 0;
        for (int r = tid; r < R; r += kSchedThreads) {
            const int c = P.cnt[r];
            n += c & 0x3fffffff;
            cl |= c >> 30;
            len_arr[r] = 0;
        }
        if (n) atomicAdd(&s_nE, n);
        if (cl) atomicOr(&s_status, DSPARK_DEV_CONF_CLAMPED);
    }
    __syncthreads();

    const int nE = s_nE;
    long long cap = (long long)P.budget - (long long)R;
    if (cap < 0) { cap = 0; if (tid == 0) s_status |= DSPARK_DEV_BUDGET_LT_R; }
    const int N = (int)(nE < cap ? nE : cap);
    const unsigned long long T0 = (unsigned long long)R << 40;
    if (tid == 0) {
        s_T_best = T0;
        s_theta_best = __dmul_rn(__ull2double_rn(T0), P.table[R < mt ? R : mt]);
        s_istar = 0;
    }
    __syncthreads();

    for (int base = 0; base < N; base += kSchedThreads) {
        const int i = base + tid + 1;                 // 1-based admitted count
        const bool valid = i <= N;
        unsigned long long Ti = 0ull, Tp = 0ull;
        double theta_i = 0.0;
        const bool first_round = base == 0;
        if (valid) {
            Ti = first_round ? pre_Ti : P.t_by_rank[i];
            Tp = (i == 1) ? T0 : (first_round ? pre_Tp : P.t_by_rank[i - 1]);
            const int B = R + i;
            theta_i = __dmul_rn(__ull2double_rn(Ti), first_round ? pre_tab : P.table[B < mt ? B : mt]);
        }
        if (P.mode == DSPARK_SCHED_EARLY_STOP) {
            if (valid) {
                const int Bp = R + i - 1;
                const double theta_prev = __dmul_rn(__ull2double_rn(Tp), first_round ? pre_tab_prev : P.table[Bp < mt ? Bp : mt]);
                if (!(theta_i > theta_prev)) atomicMin(&s_first_bad, i);
            }
            __syncthreads();
            const int fb = s_first_bad;
            const int istar = (fb != 0x7fffffff) ? fb - 1 : (base + kSchedThreads < N ? base + kSchedThreads : N);
            if (valid && i == istar) { s_T_best = Ti; s_theta_best = theta_i; s_istar = i; }
            if (fb != 0x7fffffff && tid == 0) s_done = 1;
        } else if (P.mode == DSPARK_SCHED_GLOBAL || P.mode == kModeAsync) {
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
        __syncthreads();
        if (s_done) break;
    }
    __syncthreads();
    if (P.mode == kModeAsync) {
        // Section 5.2: the admission count found on the current confidences becomes the capacity of
        // the step after next; this step admits the top K by current scores with the capacity that
        // was stored two steps ago.
        if (tid == 0) {
            const int slot = 1 + (P.async_state[0] & 1);
            int K = P.async_state[slot];
            K = K < 0 ? 0 : K;
            const int use = N < K ? N : K;
            P.async_state[slot] = s_istar;
            P.async_state[0] += 1;
            s_istar = use;
            s_T_best = use > 0 ? P.t_by_rank[use] : T0;
            const int B = R + use;
            s_theta_best = __dmul_rn(__ull2double_rn(s_T_best), P.table[B < mt ? B : mt]);
        }
        __syncthreads();
    }
    const int istar = s_istar;

    // ---- lengths l*_r = admitted candidates of request r -----------------------------------
    for (int k = tid + 1; k <= istar; k += kSchedThreads) atomicAdd(&len_arr[k == i_first ? pre_owner : P.owner_by_rank[k]], 1);
    __syncthreads();
    if (len_in_smem)
        for (int r = tid; r < R; r += kSchedThreads) P.out_len[r] = s_len[r];

    // ---- row offsets: exclusive scan of (l*_r + 1) -------------------------------------------
    if (P.out_offsets) {
        if (tid == 0) s_carry = 0ull;
        __syncthreads();
        for (int base = 0; base < R; base += kSchedThreads) {
            const int r = base + tid;
            unsigned long long v = 0ull;
            if (r < R) v = (unsigned long long)((len_in_smem ? s_len[r] : __ldcg(&P.out_len[r])) + 1);
            unsigned long long incl = block_scan_u64(v, s_warp_tot) + s_carry;
            if (r < R) P.out_offsets[r] = (int32_t)(incl - v);
            if (r == R - 1) P.out_offsets[R] = (int32_t)incl;
            __syncthreads();
            if (tid == kSchedThreads - 1) s_carry = incl;
            __syncthreads();
        }
    }

    // ---- expected accepted length 1 + sum_{j < l*_r} a_{r,j} ---------------------------------
    if (P.out_exp) {
        for (int r = tid; r < R; r += kSchedThreads) {
            const int len = len_in_smem ? s_len[r] : __ldcg(&P.out_len[r]);
            double e = 1.0;
            for (int j = 0; j < len; ++j)
                e = __dadd_rn(e, (double)__uint_as_float(P.akey[(size_t)r * P.gpad + j]));
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

// No candidates at all (gamma = 0): only the final stage runs.
__global__ void __launch_bounds__(kSchedThreads, 1) sched_final_only_kernel(SchedParams P)
{
    pdl_wait();
    sched_final_stage(P);
}

__global__ void __launch_bounds__(kSchedThreads, 1)
build_offsets_kernel(const int32_t* __restrict__ lengths, int R, int32_t* __restrict__ offsets)
{
    __shared__ unsigned long long s_warp_tot[32];
    __shared__ unsigned long long s_carry;
    pdl_wait();
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

// Padded geometry: positions per request, requests after padding, tiles of 32 entries.
struct SchedGeom { int gpad, seg, R_pad, n_tiles; size_t akey, pfix, cnt, tbr, obr, cand, ticket, total; };
static SchedGeom sched_geom(int R, int gamma)
{
    SchedGeom g;
    int gp = 1;
    if (gamma <= 32) { while (gp < gamma) gp <<= 1; } else { gp = (gamma + 31) / 32 * 32; }
    g.gpad = gp;
    g.seg = gp < 32 ? gp : 32;
    const int req_per_tile = gp < 32 ? 32 / gp : 1;
    g.R_pad = (R + req_per_tile - 1) / req_per_tile * req_per_tile;
    const size_t n_entries = (size_t)g.R_pad * gp;
    g.n_tiles = (int)(n_entries / 32);
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    size_t o = 0;
    g.akey = o; o += up(n_entries * sizeof(uint32_t));
    g.pfix = o; o += up(n_entries * sizeof(unsigned long long));
    g.cnt = o;  o += up((size_t)R * sizeof(int32_t));
    g.tbr = o;  o += up((n_entries + 1) * sizeof(unsigned long long));
    g.obr = o;  o += up((n_entries + 1) * sizeof(int32_t));
    g.cand = o; o += up(n_entries * sizeof(int32_t));
    g.ticket = o; o += up(2 * sizeof(int));
    g.total = o;
    return g;
}

}  // namespace dspark

using namespace dspark;

extern "C" {

size_t dspark_schedule_workspace_bytes(int R, int gamma)
{
    if (R < 1 || gamma < 0) return 0;
    if (R > (1 << 20) || gamma > 4096 || (long long)R * gamma > (1 << 20)) return 0;
    return sched_geom(R, gamma).total;
}

static int schedule_launch(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                           int R, int gamma, int budget_tokens, int mode, int topk_K, int32_t* async_state,
                           int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                           float* out_expected_len, dspark_sched_info_t* out_info,
                           void* workspace, size_t workspace_bytes, void* stream)
{
    if (!prof || !out_len || (!conf && gamma > 0)) return DSPARK_ERR_INVALID_ARG;
    if (R < 1 || gamma < 0) return DSPARK_ERR_INVALID_ARG;
    if (R > (1 << 20) || gamma > 4096 || (long long)R * gamma > (1 << 20)) return DSPARK_ERR_SHAPE;
    const SchedGeom g = sched_geom(R, gamma);
    if (!workspace || workspace_bytes < g.total) return DSPARK_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return DSPARK_ERR_ALIGNMENT;

    int max_tokens = 0;
    const double* table = dspark_profile_table(prof, &max_tokens);
    unsigned char* ws = (unsigned char*)workspace;
    SchedParams P;
    P.conf = conf; P.draft_len = draft_len;
    P.R = R; P.gamma = gamma; P.budget = budget_tokens; P.mode = mode; P.topk = topk_K;
    P.table = table; P.max_tokens = max_tokens;
    P.out_len = out_len; P.out_offsets = out_row_offsets; P.out_surv = out_survival;
    P.out_exp = out_expected_len; P.info = out_info;
    P.async_state = async_state;
    P.gpad = g.gpad; P.seg = g.seg; P.n_tiles = g.n_tiles; P.R_pad = g.R_pad;
    P.akey = (uint32_t*)(ws + g.akey);
    P.pfix = (unsigned long long*)(ws + g.pfix);
    P.cnt = (int32_t*)(ws + g.cnt);
    P.t_by_rank = (unsigned long long*)(ws + g.tbr);
    P.owner_by_rank = (int32_t*)(ws + g.obr);
    {
        long long cap0 = (long long)budget_tokens - R;
        cap0 = cap0 < 0 ? 0 : cap0;
        const long long n_entries0 = (long long)g.n_tiles * 32;
        P.cand = (n_entries0 >= 8192 && cap0 * 2 <= n_entries0) ? (int32_t*)(ws + g.cand) : nullptr;
    }
    P.ticket = (int*)(ws + g.ticket);

    cudaStream_t s = (cudaStream_t)stream;
    KernelTimerScope timer(DSPARK_K_SCHEDULE, s);
    const int prep_warps = g.R_pad / (32 / g.seg);
    const int prep_ctas = (prep_warps + kPrepThreads / 32 - 1) / (kPrepThreads / 32);
    launch_pdl(sched_prep_kernel, dim3(prep_ctas), dim3(kPrepThreads), 0, s, P);
    if (g.n_tiles > 0 && gamma > 0) {
        // Ranking only the candidates that fit under the cap pays once the candidate set is large and
        // the cap cuts at least half of it; small problems rank every entry and save the extra kernel.
        long long cap = (long long)budget_tokens - R;
        cap = cap < 0 ? 0 : cap;
        const long long n_entries = (long long)g.n_tiles * 32;
        const bool select = n_entries >= 8192 && cap * 2 <= n_entries;
        long long want = g.n_tiles;
        if (select) {
            launch_pdl(sched_select_kernel, dim3(1), dim3(kSchedThreads), 0, s, P);
            want = (cap + n_entries / 16) / 32 + 1;    // the cap plus histogram slack; the kernel loops if more
        }
        const dim3 grid((unsigned)(want < g.n_tiles ? want : g.n_tiles)), block(kSchedThreads);
        switch (g.seg) {
            case 1: launch_pdl(sched_rank_kernel<1>, grid, block, 0, s, P); break;
            case 2: launch_pdl(sched_rank_kernel<2>, grid, block, 0, s, P); break;
            case 4: launch_pdl(sched_rank_kernel<4>, grid, block, 0, s, P); break;
            case 8: launch_pdl(sched_rank_kernel<8>, grid, block, 0, s, P); break;
            case 16: launch_pdl(sched_rank_kernel<16>, grid, block, 0, s, P); break;
            default: launch_pdl(sched_rank_kernel<32>, grid, block, 0, s, P); break;
        }
    } else {
        launch_pdl(sched_final_only_kernel, dim3(1), dim3(kSchedThreads), 0, s, P);
    }
    return launch_status();
}

int dspark_schedule(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                    int R, int gamma, int budget_tokens, int mode, int topk_K,
                    int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                    float* out_expected_len, dspark_sched_info_t* out_info,
                    void* workspace, size_t workspace_bytes, void* stream)
{
    if (mode != DSPARK_SCHED_EARLY_STOP && mode != DSPARK_SCHED_GLOBAL && mode != DSPARK_SCHED_TOPK)
        return DSPARK_ERR_INVALID_ARG;
    return schedule_launch(prof, conf, draft_len, R, gamma, budget_tokens, mode, topk_K, nullptr, out_len,
                           out_row_offsets, out_survival, out_expected_len, out_info, workspace, workspace_bytes,
                           stream);
}

__global__ void async_state_init_kernel(int32_t* state, int K)
{
    pdl_wait();
    if (threadIdx.x == 0) { state[0] = 0; state[1] = K; state[2] = K; state[3] = 0; }
}

int dspark_async_state_init(int32_t* state, int initial_K, void* stream)
{
    if (!state || initial_K < 0) return DSPARK_ERR_INVALID_ARG;
    launch_pdl(async_state_init_kernel, dim3(1), dim3(32), 0, (cudaStream_t)stream, state, initial_K);
    return launch_status();
}

int dspark_schedule_async(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                          int R, int gamma, int budget_tokens, int32_t* state,
                          int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                          float* out_expected_len, dspark_sched_info_t* out_info,
                          void* workspace, size_t workspace_bytes, void* stream)
{
    if (!state) return DSPARK_ERR_INVALID_ARG;
    return schedule_launch(prof, conf, draft_len, R, gamma, budget_tokens, kModeAsync, 0, state, out_len,
                           out_row_offsets, out_survival, out_expected_len, out_info, workspace, workspace_bytes,
                           stream);
}

int dspark_build_offsets(const int32_t* lengths, int R, int32_t* row_offsets, void* stream)
{
    if (!lengths || !row_offsets || R < 1) return DSPARK_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    KernelTimerScope timer(DSPARK_K_OFFSETS, s);
    launch_pdl(build_offsets_kernel, dim3(1), dim3(kSchedThreads), 0, s, lengths, R, row_offsets);
    return launch_status();
}

}  // extern "C"
