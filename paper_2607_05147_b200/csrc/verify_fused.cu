// Single-launch verifier: the whole of dspark_verify / dspark_verify_per_request / dspark_verify_greedy
// in one persistent kernel (acceptance rule of Section 2.1, bonus token of Section 1, flat ragged rows of
// Section 5.3).
//
// The streamed pass of verify.cu stays as it is -- persistent CTAs, a producer warp feeding a ring of 32 KB
// stages with 1-D bulk async copies, eight consumer warps reducing one 4 KB block each, units handed out by a
// grid-wide counter -- but nothing waits for a kernel boundary any more:
//   * units are handed out request-major (target row and draft row of a position next to each other), so
//     requests complete one after the other while the pass is still streaming;
//   * every block ends with one ticket (an atomic add on a counter of its position).  The warp that draws the
//     last ticket of a position combines the block statistics into row statistics and runs the accept test;
//     the warp that completes the last position of a request finds the first rejection, writes the accepted
//     prefix and either draws the bonus token on the spot or publishes the rejected position as a task;
//   * CTAs that find the statistics units exhausted draw residual units (task, 16 KB piece of the row pair)
//     from a second counter; the warp that completes the last block of a task draws the corrected token.
// Nobody waits for a ticket: only a producer that holds a residual unit whose task is not yet published polls
// (bounded) for it, and it can only be waiting for warps that are already running.
#include <cstdio>

#include "verify_device.cuh"

namespace dspark {

constexpr int kUnitEnd = 0, kUnitStats = 1, kUnitResid = 2;
constexpr long long kResidBit = 1ll << 62, kEndCode = -1;

struct __align__(16) FusedSlot {     // what the producer tells the consumers about a stage
    int kind, piece;
    int sigma;                       // statistics row of the unit's stream
    int r, j, len, lo;               // request, position, draft positions of the request, its first target row
    int tok;                         // draft token of the position (-1: bonus row)
    int is_draft;
    float scale;                     // log2(e) / T of the request
    unsigned int g;                  // first stream of the request
    int pad;
    FusedTask task;                  // residual unit: the task it belongs to
};

__device__ __forceinline__ int atom_add_acq_rel(int* p, int v)
{
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
__device__ __forceinline__ int ld_acquire(const int* p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(int* p, int v)
{
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// A mbarrier wait that also gives up when the CTA's abort flag is raised.
__device__ __forceinline__ bool mbar_wait_abortable(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t limit)
{
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 63u) == 63u && *abort_flag) return false;
    }
    return false;
}

// Poll limits: the entry waits (a consumer waiting for data, the producer waiting for a free stage, for the
// launch tag or for a residual task) can be shortened for diagnostics; the producer's wait for copies it has
// already issued always keeps the long bound, so that no copy can land in a CTA that has left.
__device__ uint32_t g_entry_poll_limit = kWaitPollLimit;

// ---------------------------------------------------------------------------------------
// Stream prefix.  Request r owns the streams [gb[r], gb[r+1]): sampling 2 len + 1 (target and draft row of
// every position interleaved, then the bonus row), greedy len + 1.  A request whose offsets are unusable
// owns none; one whose streams would not fit the statistics arrays (only possible with inconsistent
// offsets) is dropped as well.  CTA-wide; total_fit and n_dead are returned to every thread.
// ---------------------------------------------------------------------------------------
constexpr int kConsumerThreads = kConsumerWarps * 32;
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }

template <bool kGreedy>
__device__ void build_prefix(const FusedParams& F, int n_rows, unsigned int* gb, bool write_outputs,
                             unsigned int* s_fit, int* s_dead)
{
    // called by the consumer warps only (threads 0 .. kConsumerThreads-1); results in *s_fit, *s_dead (shared)
    __shared__ unsigned long long s_w[kConsumerWarps];
    __shared__ unsigned long long s_carry;
    const VerifyParams& P = F.P;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { s_carry = 0ull; *s_fit = 0u; *s_dead = 0; }
    consumer_sync();
    for (int base = 0; base < P.R; base += kConsumerThreads) {
        const int r = base + tid;
        unsigned long long cnt = 0ull;
        bool ok = false;
        if (r < P.R) {
            const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
            ok = lo >= 0 && hi - lo >= 1 && hi <= n_rows;
            if (!kGreedy) ok = ok && lo - r >= 0 && (hi - 1 - r) <= n_rows - P.R;
            if (ok) cnt = kGreedy ? (unsigned long long)(hi - lo) : 2ull * (unsigned long long)(hi - lo) - 1ull;
        }
        unsigned long long x = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += t;
        }
        if (lane == 31) s_w[warp] = x;
        consumer_sync();
        unsigned long long before = s_carry;
        for (int w = 0; w < warp; ++w) before += s_w[w];
        const unsigned long long excl = before + x - cnt, incl = before + x;
        if (r < P.R) {
            gb[r] = excl > 0xFFFFFFFFull ? 0xFFFFFFFFu : (unsigned int)excl;
            if (ok && incl <= (unsigned long long)F.stream_cap) {
                atomicMax(s_fit, (unsigned int)incl);
            } else {
                atomicAdd(s_dead, 1);
                if (write_outputs) P.accepted_len[r] = 0;
            }
        }
        consumer_sync();
        if (tid == kConsumerThreads - 1) s_carry = incl;
        consumer_sync();
    }
    if (tid == 0) gb[P.R] = s_carry > 0xFFFFFFFFull ? 0xFFFFFFFFu : (unsigned int)s_carry;
    consumer_sync();
    if (write_outputs && tid == 0 && *s_dead > 0) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
}

// Largest r in [0, R) with gb[r] <= sigma (gb non-decreasing, gb[0] = 0).
__device__ __forceinline__ int find_request(const unsigned int* gb, int R, unsigned int sigma)
{
    int lo = 0, hi = R;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (gb[mid] <= sigma) lo = mid; else hi = mid;
    }
    return lo;
}

__device__ __forceinline__ float request_scale(const VerifyParams& P, int r)
{
    if (!P.req_temp) return P.scale;
    const float T = P.req_temp[r];
    return (T > 0.0f && T < INFINITY) ? (float)(1.4426950408889634 / (double)T) : 1.0f;
}

// ---------------------------------------------------------------------------------------
// Inverse CDF inside one block held lane-strided in registers (vector k of lane l is vector k*32+l of the
// block; vectors past the end of the row hold -inf and weigh nothing).  f(xt, xd) is the weight of an element.
// Running sums are fp64.  Returns the element index inside the block; when rounding between the block value
// of level 1 and these sums leaves no crossing, the last element with positive weight.
// ---------------------------------------------------------------------------------------
template <int kElem>
__device__ __forceinline__ float vec_elem(const uint4& q, int e)
{
    if (kElem == 4) return __uint_as_float(word_of(q, e));
    const uint32_t w = word_of(q, e >> 1);
    return (e & 1) ? bf16hi(w) : bf16lo(w);
}

template <int kElem, int kVec, typename F>
__device__ __forceinline__ int level2_registers(const uint4 (&vt)[kVec], const uint4 (&vd)[kVec], int lane, double thr, F f)
{
    constexpr int kPer = 16 / kElem;
    double xs[kVec];
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        double s = 0.0;
#pragma unroll
        for (int e = 0; e < kPer; ++e) s += (double)f(vec_elem<kElem>(vt[k], e), vec_elem<kElem>(vd[k], e));
        xs[k] = s;
    }
    double run = 0.0;
    int kc = -1;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        const double ct = warp_sum_f64(xs[k]);
        if (kc < 0) { if (run + ct > thr) kc = k; else run += ct; }
    }
    int l = -1;
    if (kc >= 0) {
        double xc = 0.0;
#pragma unroll
        for (int k = 0; k < kVec; ++k) if (k == kc) xc = xs[k];
        const double incl = warp_incl_scan_f64(xc, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, run + incl > thr);
        if (hit) {
            l = __ffs(hit) - 1;
            run += __shfl_sync(0xffffffffu, incl - xc, l);
        } else {
            kc = -1;                                  // the chunk total crossed, the lane sums do not: rounding
        }
    }
    if (kc < 0) {                                     // last vector with positive weight
        run = -1.0;                                   // every positive weight crosses: the walk below stops at the last one
        thr = INFINITY;
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            const unsigned pos = __ballot_sync(0xffffffffu, xs[k] > 0.0);
            if (pos) { kc = k; l = 31 - __clz(pos); }
        }
        if (kc < 0) return 0;
    }
    uint4 a = vt[0], b = vd[0];
#pragma unroll
    for (int k = 1; k < kVec; ++k) if (k == kc) { a = vt[k]; b = vd[k]; }
    int found = -1, lastpos = -1;
    double acc = run;
#pragma unroll
    for (int e = 0; e < kPer; ++e) {
        const float w = f(vec_elem<kElem>(a, e), vec_elem<kElem>(b, e));
        if (w > 0.f) lastpos = e;
        acc += (double)w;
        if (found < 0 && acc > thr) found = e;
    }
    if (found < 0) found = lastpos >= 0 ? lastpos : kPer - 1;
    found = __shfl_sync(0xffffffffu, found, l);
    return (kc * 32 + l) * kPer + found;
}

// Draw from p of one target row in vocabulary order: level 1 over the block masses of its saved statistics,
// level 2 inside the one block that holds the crossing (4 KB re-read).  One warp.
template <int kElem>
__device__ int draw_from_p(const VerifyParams& P, long long stat_row, long long target_row, float cp, float scale, double u, int lane)
{
    const float2* st = P.stats_t + stat_row * P.nblk;
    auto mass = [&](int i) { const float2 e = __ldcg(&st[i]); return e.x > kNegInf ? e.y * ex2_approx(e.x - cp) : 0.f; };
    double before, tot;
    int b;
    if (P.nblk <= 256) {
        float xr[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { const int i = k * 32 + lane; xr[k] = i < P.nblk ? mass(i) : 0.f; }
        b = level1_registers(xr, P.nblk, lane, u, before, tot);
    } else {
        tot = warp_total(P.nblk, lane, mass);
        b = level1_memory(P.nblk, lane, mass, u * tot, before);
    }
    if (!(tot > 0.0) || !(tot < INFINITY)) return 0;         // cannot happen for a usable row
    const double thr_local = u * tot - before;
    const int e0 = b * P.epb;
    const int cnt = (P.V - e0) < P.epb ? (P.V - e0) : P.epb;
    uint4 v[kStatVec];
    GlobalFetch<kElem> f{P.target + target_row * P.tstride_bytes + (long long)e0 * kElem};
    load_block<kElem, kStatVec>(f, cnt * kElem, lane, v);
    const float nc = -cp;
    return e0 + level2_registers<kElem, kStatVec>(v, v, lane, thr_local,
                                                  [&](float xt, float) { return ex2_approx(__fmaf_rn(xt, scale, nc)); });
}

// ---------------------------------------------------------------------------------------
// What the warp that completes a residual task does: the corrected token from norm(max(0, p - q)).
// ---------------------------------------------------------------------------------------
template <int kElem>
__device__ __noinline__ void resid_epilogue(const FusedParams& F, const FusedTask ft)
{
    const VerifyParams& P = F.P;
    const int lane = threadIdx.x & 31;
    __threadfence();
    const ResidTask& t = ft.t;
    const float* wb = P.wblk + (long long)t.wslot * P.nblk_r;
    auto wv = [&](int i) { return __ldcg(&wb[i]); };
    const double u = (double)t.u;
    double before, tot;
    int b;
    if (P.nblk_r <= 256) {
        float xr[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { const int i = k * 32 + lane; xr[k] = i < P.nblk_r ? wv(i) : 0.f; }
        b = level1_registers(xr, P.nblk_r, lane, u, before, tot);
    } else {
        tot = warp_total(P.nblk_r, lane, wv);
        b = level1_memory(P.nblk_r, lane, wv, u * tot, before);
    }
    int token;
    if (!(tot > 0.0) || !(tot < INFINITY)) {
        // empty residual (p and q agree to rounding): draw from p of that row with the same uniform
        token = draw_from_p<kElem>(P, ft.sigma_t, t.row_t, t.cp, t.scale, u, lane);
    } else {
        ResidConst K;
        K.set(t.scale, t.cp, t.inv_zp, t.cq, t.inv_zq, kNegInf);
        const int e0 = b * P.epb_r;
        const int cnt = (P.V - e0) < P.epb_r ? (P.V - e0) : P.epb_r;
        uint4 vt[kResidVec], vd[kResidVec];
        GlobalFetch<kElem> ft0{P.target + (long long)t.row_t * P.tstride_bytes + (long long)e0 * kElem};
        GlobalFetch<kElem> fd0{P.draft + t.row_d * P.dstride_bytes + (long long)e0 * kElem};
        load_block<kElem, kResidVec>(ft0, cnt * kElem, lane, vt);
        load_block<kElem, kResidVec>(fd0, cnt * kElem, lane, vd);
        token = e0 + level2_registers<kElem, kResidVec>(vt, vd, lane, u * tot - before,
                                                        [&](float xt, float xd) { return resid_elem(xt, xd, K); });
    }
    if (lane == 0) P.out_tokens[t.row_t] = token;
}

// ---------------------------------------------------------------------------------------
// What the warp that completes the last position of a request does (sampling): first rejection, accepted
// prefix, then the bonus draw or the publication of the rejected position as a residual task.
// ---------------------------------------------------------------------------------------
template <int kElem>
__device__ __noinline__ void request_epilogue(const FusedParams& F, int r, int len, int lo, unsigned int g, float scale_f)
{
    const VerifyParams& P = F.P;
    const int lane = threadIdx.x & 31;
    __threadfence();
    int bad = 0;
    for (int i = lane; i < len; i += 32) {
        const int d = P.draft_tokens[lo + i];
        if (d < 0 || d >= P.V) bad |= DSPARK_DEV_BAD_TOKEN;
    }
    bad = __reduce_or_sync(0xffffffffu, bad);
    if (P.req_temp) {
        const float T = P.req_temp[r];
        if (!(T > 0.0f) || !(T < INFINITY)) bad |= DSPARK_DEV_BAD_TEMPERATURE;
    }
    int n = len, first_bad = 0x7fffffff;
    bool bonus_bad = false;
    for (int base = 0; base <= len; base += 32) {
        const int jj = base + lane;
        const int fl = jj <= len ? __ldcg(&F.pos[g + 2u * (unsigned)jj].flags) : 0;
        const unsigned rej = __ballot_sync(0xffffffffu, (fl & kPosRejected) != 0);
        const unsigned bd = __ballot_sync(0xffffffffu, (fl & kPosBad) != 0 && jj < len);
        bonus_bad |= __any_sync(0xffffffffu, (fl & kPosBad) != 0 && jj == len);
        if (rej && n == len) n = base + __ffs(rej) - 1;
        if (bd && first_bad == 0x7fffffff) first_bad = base + __ffs(bd) - 1;
    }
    const bool want_all = (P.out_p != nullptr) || (P.out_q != nullptr);
    // Which rows void the request: with the probability outputs every draft position counts; without them
    // verification ends at the first rejection and only an unusable row before it does.  The row that emits
    // the token must be usable in any case (a rejected position is, or it would not have been tested).
    const bool bad_row = (want_all ? first_bad != 0x7fffffff : first_bad < n) || (n == len && bonus_bad);
    if (bad || bad_row) {
        for (int i = lane; i <= len; i += 32) P.out_tokens[lo + i] = -1;
        if (lane == 0) {
            atomicOr(P.dev_status, bad ? bad : DSPARK_DEV_BAD_ROW);
            P.accepted_len[r] = 0;
        }
    } else {
        for (int i = lane; i <= len; i += 32) P.out_tokens[lo + i] = i < n ? P.draft_tokens[lo + i] : -1;
        float ua, ur;
        philox_uniforms(P.seed, (uint32_t)r, (uint32_t)n, ua, ur);
        const unsigned int sn = g + 2u * (unsigned)n;
        const float cp = __ldcg(&F.pos[sn].cp), inv_zp = __ldcg(&F.pos[sn].inv_zp);
        if (lane == 0) P.accepted_len[r] = n;
        if (n < len) {
            __syncwarp();
            if (lane == 0) {
                FusedTask ft;
                ft.t.request = r; ft.t.row_t = lo + n;
                ft.t.row_d = (P.draft_row_start ? P.draft_row_start[r] : (long long)(lo - r)) + n;
                ft.t.cp = cp; ft.t.inv_zp = inv_zp;
                ft.t.cq = __ldcg(&F.pos[sn].cq); ft.t.inv_zq = __ldcg(&F.pos[sn].inv_zq);
                ft.t.u = ur; ft.t.scale = scale_f; ft.t.wslot = r; ft.t.tau = kNegInf;
                ft.sigma_t = (int)sn; ft.ready = 0; ft.pad[0] = ft.pad[1] = 0;
                const int slot = atomicAdd(&P.counters[0], 1);
                F.tasks[slot] = ft;
                __threadfence();                      // the accepted prefix written by the other lanes goes first too
                st_release(&F.tasks[slot].ready, 1);
            }
        } else {
            const int token = draw_from_p<kElem>(P, (long long)sn, (long long)lo + n, cp, scale_f, (double)ur, lane);
            if (lane == 0) P.out_tokens[lo + n] = token;
        }
    }
    __syncwarp();
    if (lane == 0) { __threadfence(); atomicAdd(&P.counters[kHdrDecided], 1); }
}

// What the warp that draws the last block ticket of a position does (sampling): row statistics from block
// statistics, p(x), q(x), the accept test; then its own ticket on the request.
template <int kElem>
__device__ __noinline__ void position_epilogue(const FusedParams& F, int r, int j, int len, int lo, unsigned int g, float scale_f)
{
    const VerifyParams& P = F.P;
    const int lane = threadIdx.x & 31;
    __threadfence();
    const unsigned int st = g + 2u * (unsigned)j;
    const bool is_draft_pos = j < len;
    RowAcc A, D;
    combine_rows(P.stats_t + (long long)st * P.nblk, is_draft_pos ? P.stats_t + (long long)(st + 1u) * P.nblk : nullptr,
                 P.nblk, lane, A, D);
    int last = 0;
    if (lane == 0) {
        PosRec rec;
        rec.cp = A.C; rec.cq = D.C; rec.inv_zp = 0.f; rec.inv_zq = 0.f; rec.flags = 0;
        rec.pad[0] = rec.pad[1] = rec.pad[2] = 0;
        const bool ok_t = row_usable(A.C, A.S), ok_d = !is_draft_pos || row_usable(D.C, D.S);
        if (ok_t) rec.inv_zp = (float)(1.0 / A.S);
        if (is_draft_pos && ok_d) rec.inv_zq = (float)(1.0 / D.S);
        if (!ok_t || !ok_d) {
            rec.flags = kPosBad;
        } else if (is_draft_pos) {
            const int d = P.draft_tokens[lo + j];
            if (d >= 0 && d < P.V) {
                const double scale_d = (double)scale_f;
                const double xt = (double)__ldcg(&F.xtok[st]), xd = (double)__ldcg(&F.xtok[st + 1u]);
                const double p = exp2(xt * scale_d - (double)A.C) / A.S;
                const double q = exp2(xd * scale_d - (double)D.C) / D.S;
                if (P.out_p) P.out_p[lo + j] = (float)p;
                if (P.out_q) P.out_q[lo + j] = (float)q;
                float ua, ur;
                philox_uniforms(P.seed, (uint32_t)r, (uint32_t)j, ua, ur);
                if (!((double)ua * q < p)) rec.flags = kPosRejected;
            }
        }
        F.pos[st] = rec;
        last = atom_add_acq_rel(&F.req_ticket[r], 1) == len;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) request_epilogue<kElem>(F, r, len, lo, g, scale_f);
}

// Greedy: the row argmax from its block statistics, then the ticket on the request; the warp that completes
// the request finds the first draft token that differs from its row's argmax.
__device__ __noinline__ void greedy_request_epilogue(const FusedParams& F, int r, int len, int lo, unsigned int g)
{
    const VerifyParams& P = F.P;
    const int lane = threadIdx.x & 31;
    __threadfence();
    const GreedyRec* rec = reinterpret_cast<const GreedyRec*>(F.pos);
    int bad = 0;
    for (int i = lane; i < len; i += 32) {
        const int d = P.draft_tokens[lo + i];
        if (d < 0 || d >= P.V) bad = 1;
    }
    if (__any_sync(0xffffffffu, bad)) {
        for (int i = lane; i <= len; i += 32) P.out_tokens[lo + i] = -1;
        if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_TOKEN); P.accepted_len[r] = 0; }
        return;
    }
    int n = -1, emit = -1, status = 0;
    for (int base = 0; base <= len && n < 0; base += 32) {
        const int jj = base + lane;
        int am = 0, neg = 0, stop = 0;
        if (jj <= len) {
            const int* e = reinterpret_cast<const int*>(&rec[g + (unsigned)jj]);
            am = __ldcg(e); neg = __ldcg(e + 1);
            stop = (jj == len) || P.draft_tokens[lo + jj] != am;     // the bonus row always ends the scan
        }
        const unsigned hit = __ballot_sync(0xffffffffu, stop);
        const int upto = hit ? __ffs(hit) - 1 : 31;                   // rows up to the one that emits may raise the flag
        if (__any_sync(0xffffffffu, neg && lane <= upto)) status |= DSPARK_DEV_ALL_NEG_INF;
        if (hit) { n = base + upto; emit = __shfl_sync(0xffffffffu, am, upto); }
    }
    for (int i = lane; i <= len; i += 32) P.out_tokens[lo + i] = i < n ? P.draft_tokens[lo + i] : (i == n ? emit : -1);
    if (lane == 0) {
        P.accepted_len[r] = n;
        if (status) atomicOr(P.dev_status, status);
    }
}

__device__ __noinline__ void greedy_position_epilogue(const FusedParams& F, int r, int j, int len, int lo, unsigned int g)
{
    const VerifyParams& P = F.P;
    const int lane = threadIdx.x & 31;
    __threadfence();
    const float2* st = P.stats_t + (long long)(g + (unsigned)j) * P.nblk;
    float best = kNegInf;
    int bi = 0x7fffffff;
    for (int b = lane; b < P.nblk; b += 32) {          // lane-strided: ascending indices per lane
        const float2 e = __ldcg(&st[b]);
        const int idx = __float_as_int(e.y);
        if (e.x > best || (e.x == best && idx < bi)) { best = e.x; bi = idx; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    int last = 0;
    if (lane == 0) {
        GreedyRec e;
        e.all_neg_inf = (best == kNegInf);
        e.argmax = e.all_neg_inf ? 0 : bi;
        reinterpret_cast<GreedyRec*>(F.pos)[g + (unsigned)j] = e;
        last = atom_add_acq_rel(&F.req_ticket[r], 1) == len;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) greedy_request_epilogue(F, r, len, lo, g);
}

// ---------------------------------------------------------------------------------------
// The kernel
// ---------------------------------------------------------------------------------------
template <int kElem, bool kGreedy>
__global__ void __launch_bounds__(kStreamThreads, 3) verify_fused_kernel(const __grid_constant__ FusedParams F)
{
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ FusedSlot s_unit[kStages];
    __shared__ int s_abort, s_tag_seen, s_dead;
    __shared__ unsigned int s_fit;
    __shared__ long long s_first[kStages];

    const VerifyParams& P = F.P;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kConsumerWarps); }
        s_abort = 0; s_tag_seen = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait();                                  // everything below reads what earlier kernels wrote

    volatile int* abort_flag = &s_abort;
    volatile int* tag_seen = &s_tag_seen;
    const uint32_t entry_limit = g_entry_poll_limit;
    int* hdr = P.counters;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const bool smem_prefix = F.gbase_g == nullptr;
    unsigned int* gb_s = reinterpret_cast<unsigned int*>(stage_mem + kStages * kStageBytes);
    const unsigned int* gb = smem_prefix ? gb_s : F.gbase_g;
    unsigned long long* ctr_s = unit_counter<kModeStats>(P);
    unsigned long long* ctr_r = unit_counter<kModeResid>(P);
    unsigned long long* tag_units = unit_tag(P);          // published once the unit counters are zero
    unsigned long long* tag_state = unit_tag(P) + 1;      // published once tickets, queue and stream prefix are set

    // Start-up.  Every unit is drawn from a counter: a unit that belonged to a CTA by its index could belong to
    // a CTA that is not resident yet (another kernel holds the SMs) while resident CTAs wait for the request it
    // is part of.  CTA 0, which is dispatched first, zeroes the unit counters and publishes the first tag at
    // once; the producer of every CTA draws its first two units as soon as it sees that tag, while the
    // consumer warps set up the stream prefix.  CTA 0 then clears the tickets and publishes the second tag,
    // which everybody looks for before touching a ticket or the residual queue.
    if (warp == kConsumerWarps) {
        if (lane == 0) {
            bool ok = true;
            if (blockIdx.x == 0) {
                hdr[0] = 0; *ctr_s = 0ull; *ctr_r = 0ull;
                hdr[kHdrExit] = 0; hdr[kHdrAbort] = 0;
                if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
                __threadfence();
                atomicExch(tag_units, P.launch_tag);
            } else {
                ok = false;
                for (uint32_t i = 0; i < entry_limit && !ok; ++i) {
                    unsigned long long v;
                    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(tag_units) : "memory");
                    ok = v == P.launch_tag;
                }
                if (!ok) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
            }
            s_first[0] = ok ? (long long)atomicAdd(ctr_s, 1ull) : kEndCode;
            s_first[1] = ok ? (long long)atomicAdd(ctr_s, 1ull) : kEndCode;
        }
    } else {
        if (blockIdx.x == 0) {
            for (int i = tid; i < F.stream_cap; i += kConsumerThreads) F.pos_ticket[i] = 0;
            for (int i = tid; i < P.R; i += kConsumerThreads) {
                F.req_ticket[i] = 0;
                if (!kGreedy) { F.resid_ticket[i] = 0; F.tasks[i].ready = 0; }
            }
        }
        if (smem_prefix || blockIdx.x == 0)
            build_prefix<kGreedy>(F, n_rows, smem_prefix ? gb_s : F.gbase_g, blockIdx.x == 0, &s_fit, &s_dead);
        if (blockIdx.x == 0) {
            __threadfence();
            consumer_sync();
            if (tid == 0) {
                hdr[kHdrDecided] = s_dead;
                hdr[kHdrTotalFit] = (int)s_fit;
                hdr[kHdrDead] = s_dead;
                __threadfence();
                atomicExch(tag_state, P.launch_tag);
                *tag_seen = 1;
            }
        } else if (!smem_prefix && tid == 0) {
            // the stream prefix lives in global memory and is CTA 0's to build: nothing can be mapped before it is there
            if (wait_for_tag(tag_state, P.launch_tag)) { *tag_seen = 1; s_fit = (unsigned int)__ldcg(&hdr[kHdrTotalFit]); }
            else { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); s_fit = 0u; *abort_flag = 1; }
        }
    }
    __syncthreads();
    const unsigned int total_fit = s_fit;

    const int nblk = P.nblk, nblk_r = P.nblk_r;
    const int ppr = (nblk + kConsumerWarps - 1) / kConsumerWarps;
    const int ppr_r = (nblk_r + kConsumerWarps - 1) / kConsumerWarps;
    const long long total_units = (long long)total_fit * ppr;

    // lane 0 of a warp: make sure the second tag has been seen by this CTA (bounded); false: give up
    auto ensure_tag = [&]() -> bool {
        if (*tag_seen) return true;
        for (uint32_t i = 0; i < entry_limit; ++i) {
            unsigned long long v;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(tag_state) : "memory");
            if (v == P.launch_tag) { *tag_seen = 1; return true; }
        }
        atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT);
        hdr[kHdrAbort] = 1;
        *abort_flag = 1;
        return false;
    };

    if (warp == kConsumerWarps) {
        // ---------------- producer warp: lane 0 draws the units and issues the copies ----------------
        const uint64_t pol_first = l2_policy_evict_first();
        bool stats_done = false;
        int it = 0;
        // the next unit of this CTA from the grid-wide counters (lane 0)
        auto draw = [&]() -> long long {
            if (!stats_done) {
                const long long x = (long long)atomicAdd(ctr_s, 1ull);
                if (x < total_units) return x;
                stats_done = true;
            }
            if (kGreedy || !ensure_tag()) return kEndCode;
            return kResidBit | (long long)atomicAdd(ctr_r, 1ull);
        };
        // one turn of the pipeline with the unit held in `mine`; `mine` then receives the unit of the turn
        // after next
        auto turn = [&](long long& mine) -> bool {
            const int st = it % kStages;
            const uint32_t ph = (uint32_t)(it / kStages) & 1u;
            FusedSlot slot = {};
            const unsigned char *src0 = nullptr, *src1 = nullptr;
            int bytes = 0;
            slot.kind = kUnitEnd;
            if (lane == 0 && !*abort_flag) {
                const long long code = mine;
                if (code >= 0 && code < kResidBit) {
                    const unsigned int sigma = (unsigned int)(code / ppr);
                    slot.kind = kUnitStats;
                    slot.piece = (int)(code - (long long)sigma * ppr);
                    slot.sigma = (int)sigma;
                    const int r = find_request(gb, P.R, sigma);
                    const unsigned int g = gb[r], cnt = gb[r + 1] - g, k = sigma - g;
                    const int lo = __ldg(&P.row_offsets[r]);
                    slot.r = r; slot.g = g; slot.lo = lo;
                    if (kGreedy) { slot.j = (int)k; slot.len = (int)cnt - 1; slot.is_draft = 0; }
                    else { slot.j = (int)(k >> 1); slot.len = (int)((cnt - 1u) >> 1); slot.is_draft = (int)(k & 1u); }
                    slot.tok = slot.j < slot.len ? __ldg(&P.draft_tokens[lo + slot.j]) : -1;
                    slot.scale = kGreedy ? 1.0f : request_scale(P, r);
                    const long long off = (long long)slot.piece * kStageBytes;
                    const long long rem = (long long)P.row_bytes - off;
                    bytes = (int)(rem < kStageBytes ? rem : kStageBytes);
                    if (slot.is_draft) {
                        const long long row = (P.draft_row_start ? P.draft_row_start[r] : (long long)(lo - r)) + slot.j;
                        src0 = P.draft + row * P.dstride_bytes + off;
                    } else {
                        src0 = P.target + (long long)(lo + slot.j) * P.tstride_bytes + off;
                    }
                } else if (code >= kResidBit) {
                    const long long v = code - kResidBit;
                    const long long ti = v / ppr_r;
                    if (ti < P.R) {
                        // the task may not be published yet: its request is still being streamed or decided
                        int state = 0;                 // 1: task published, 2: there is no such task
                        const uint32_t task_limit = entry_limit < (1u << 19) ? entry_limit : (1u << 19);
                        for (uint32_t i = 0; i < task_limit && state == 0; ++i) {
                            if (ld_acquire(&F.tasks[ti].ready)) state = 1;
                            else if (ld_acquire(&hdr[kHdrDecided]) >= P.R && ti >= (long long)ld_acquire(&hdr[0])) state = 2;
                            else if (ld_acquire(&hdr[kHdrAbort])) { *abort_flag = 1; state = 2; }
                            else __nanosleep(64);
                        }
                        if (state == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); hdr[kHdrAbort] = 1; *abort_flag = 1; }
                        const bool have = state == 1;
                        if (have) {
                            slot.kind = kUnitResid;
                            slot.piece = (int)(v - ti * ppr_r);
                            slot.task = F.tasks[ti];
                            const long long off = (long long)slot.piece * (kStageBytes / 2);
                            const long long rem = (long long)P.row_bytes - off;
                            bytes = (int)(rem < kStageBytes / 2 ? rem : kStageBytes / 2);
                            src0 = P.target + (long long)slot.task.t.row_t * P.tstride_bytes + off;
                            src1 = P.draft + slot.task.t.row_d * P.dstride_bytes + off;
                        }
                    }
                }
            }
            const int kind = __shfl_sync(0xffffffffu, slot.kind, 0);
            if (!__all_sync(0xffffffffu, mbar_wait_abortable(&empty_bar[st], ph ^ 1u, abort_flag, entry_limit))) {
                if (lane == 0 && !*abort_flag) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); hdr[kHdrAbort] = 1; *abort_flag = 1; }
                return false;
            }
            if (lane == 0) {
                s_unit[st] = slot;                 // read by the consumers after the barrier below completes
                if (kind != kUnitEnd) {
                    unsigned char* dst = stage_mem + st * kStageBytes;
                    if (kind == kUnitStats) {
                        mbar_arrive_expect_tx(&full_bar[st], (uint32_t)bytes);
                        bulk_g2s_hint(dst, src0, (uint32_t)bytes, &full_bar[st], pol_first);
                    } else {
                        mbar_arrive_expect_tx(&full_bar[st], (uint32_t)(2 * bytes));
                        bulk_g2s_hint(dst, src0, (uint32_t)bytes, &full_bar[st], pol_first);
                        bulk_g2s_hint(dst + kStageBytes / 2, src1, (uint32_t)bytes, &full_bar[st], pol_first);
                    }
                    mine = draw();                 // needed two turns from now
                } else {
                    mbar_arrive(&full_bar[st]);    // end marker: no data follows
                }
            }
            __syncwarp();
            if (kind != kUnitEnd) ++it;
            return kind != kUnitEnd;
        };
        static_assert(kStages == 2, "the producer keeps one pending unit per stage");
        // Units are taken up in the order they were drawn (a CTA stops at the first unit that does not exist,
        // so nothing drawn earlier may still be pending then).
        long long unit_a = s_first[0], unit_b = s_first[1];
        if (lane == 0) {
            if (unit_a >= total_units) { stats_done = true; unit_a = draw(); }
            if (unit_b >= 0 && unit_b < kResidBit && unit_b >= total_units) { stats_done = true; unit_b = draw(); }
        }
        while (turn(unit_a) && turn(unit_b)) {}
        if (*abort_flag) {
            // leave only after every copy already issued has landed (bounded, never shortened)
            for (int k = 0; k < kStages && k < it; ++k) {
                const int jt = it - 1 - k;
                mbar_wait_bounded(&full_bar[jt % kStages], (uint32_t)(jt / kStages) & 1u);
            }
        }
    } else {
        // ---------------- consumer warps --------------------------------------------------------------
        for (int it = 0;; ++it) {
            const int st = it % kStages;
            const uint32_t ph = (uint32_t)(it / kStages) & 1u;
            if (*abort_flag) break;
            if (!__all_sync(0xffffffffu, mbar_wait_abortable(&full_bar[st], ph, abort_flag, entry_limit))) {
                if (lane == 0 && !*abort_flag) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); hdr[kHdrAbort] = 1; *abort_flag = 1; }
                break;
            }
            const int kind = s_unit[st].kind;
            if (kind == kUnitEnd) break;
            const int piece = s_unit[st].piece;
            const int b = piece * kConsumerWarps + warp;
            if (kind == kUnitStats) {
                const int sigma = s_unit[st].sigma, r = s_unit[st].r, j = s_unit[st].j, len = s_unit[st].len;
                const int lo = s_unit[st].lo, tok = s_unit[st].tok, is_draft = s_unit[st].is_draft;
                const unsigned int g = s_unit[st].g;
                const float scale = s_unit[st].scale;
                const bool live = b < nblk;
                if (live) {
                    const unsigned char* sp = stage_mem + st * kStageBytes + warp * kStatBlockBytes;
                    const int rem = P.row_bytes - b * kStatBlockBytes;
                    const int nbytes = rem < kStatBlockBytes ? rem : kStatBlockBytes;
                    uint4 v[kStatVec];
                    load_block<kElem, kStatVec>(SmemFetch{sp}, nbytes, lane, v);
                    const float2 e = kGreedy ? block_argmax<kElem, kStatVec>(v, b * P.epb, lane)
                                             : block_stats<kElem, kStatVec>(v, scale);
                    if (lane == 0) {
                        P.stats_t[(long long)sigma * nblk + b] = e;
                        // the logit at the draft token, while its block is on chip
                        if (!kGreedy && tok >= b * P.epb && tok < (b + 1) * P.epb) {
                            const int idx = tok - b * P.epb;
                            F.xtok[sigma] = kElem == 2 ? __uint_as_float((uint32_t)reinterpret_cast<const unsigned short*>(sp)[idx] << 16)
                                                       : reinterpret_cast<const float*>(sp)[idx];
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
                if (live) {
                    int last = 0;
                    if (lane == 0 && ensure_tag()) {
                        const int expected = (!kGreedy && j < len) ? 2 * nblk : nblk;
                        last = atom_add_acq_rel(&F.pos_ticket[sigma - is_draft], 1) == expected - 1;
                    }
                    last = __shfl_sync(0xffffffffu, last, 0);
                    if (last) {
                        if (kGreedy) greedy_position_epilogue(F, r, j, len, lo, g);
                        else position_epilogue<kElem>(F, r, j, len, lo, g, scale);
                    }
                }
            } else if (!kGreedy) {
                const FusedTask ft = s_unit[st].task;
                const bool live = b < nblk_r;
                if (live) {
                    const unsigned char* sp = stage_mem + st * kStageBytes + warp * kResidBlockBytes;
                    const int rem = P.row_bytes - b * kResidBlockBytes;
                    const int nbytes = rem < kResidBlockBytes ? rem : kResidBlockBytes;
                    uint4 vt[kResidVec], vd[kResidVec];
                    load_block<kElem, kResidVec>(SmemFetch{sp}, nbytes, lane, vt);
                    load_block<kElem, kResidVec>(SmemFetch{sp + kStageBytes / 2}, nbytes, lane, vd);
                    ResidConst K;
                    K.set(ft.t.scale, ft.t.cp, ft.t.inv_zp, ft.t.cq, ft.t.inv_zq, kNegInf);
                    const float w = block_resid<kElem, kResidVec, false>(vt, vd, K);
                    if (lane == 0) P.wblk[(long long)ft.t.wslot * nblk_r + b] = w;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
                if (live) {
                    int last = 0;
                    if (lane == 0) last = atom_add_acq_rel(&F.resid_ticket[ft.t.request], 1) == nblk_r - 1;
                    last = __shfl_sync(0xffffffffu, last, 0);
                    if (last) resid_epilogue<kElem>(F, ft);
                }
            }
        }
    }

    // The last CTA to leave clears the launch tag, so that a replayed CUDA graph (same tag every time) finds
    // the cell empty.  A CTA counts itself out only after it has seen the tag: CTA 0 zeroes the count before
    // it publishes the tag.
    __syncthreads();
    if (tid == 0 && ensure_tag()) {
        __threadfence();
        if (atomicAdd(&hdr[kHdrExit], 1) == (int)gridDim.x - 1) { *tag_units = 0ull; *tag_state = 0ull; }
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
static constexpr size_t kFusedSmemMax = (size_t)kStages * kStageBytes + (((size_t)kGbaseSmemMaxR + 1) * sizeof(unsigned int) + 15) / 16 * 16;

template <int kElem, bool kGreedy>
static cudaError_t set_fused_attr()
{
    return cudaFuncSetAttribute(verify_fused_kernel<kElem, kGreedy>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFusedSmemMax);
}

struct FusedDevice { int sms; bool attrs_set; };
static FusedDevice* fused_device()
{
    static FusedDevice info[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    FusedDevice& d = info[dev];
    if (d.sms == 0) cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    if (!d.attrs_set) {
        d.attrs_set = set_fused_attr<2, false>() == cudaSuccess && set_fused_attr<4, false>() == cudaSuccess &&
                      set_fused_attr<2, true>() == cudaSuccess && set_fused_attr<4, true>() == cudaSuccess;
        if (!d.attrs_set) return nullptr;
    }
    return &d;
}

int fused_verify_launch(const FusedParams& F, bool greedy, long long max_units, cudaStream_t stream)
{
    FusedDevice* d = fused_device();
    if (!d) return launch_status() == DSPARK_OK ? DSPARK_ERR_CUDA : DSPARK_ERR_CUDA;
    long long g = (long long)d->sms * 3;
    if (g > max_units) g = max_units;
    if (g < 1) g = 1;
    const size_t smem = (size_t)kStages * kStageBytes +
                        (F.gbase_g ? 0 : (((size_t)F.P.R + 1) * sizeof(unsigned int) + 15) / 16 * 16);
    const dim3 grid((unsigned)g), block(kStreamThreads);
    if (F.P.elem == 2) {
        if (greedy) launch_pdl(verify_fused_kernel<2, true>, grid, block, smem, stream, F);
        else launch_pdl(verify_fused_kernel<2, false>, grid, block, smem, stream, F);
    } else {
        if (greedy) launch_pdl(verify_fused_kernel<4, true>, grid, block, smem, stream, F);
        else launch_pdl(verify_fused_kernel<4, false>, grid, block, smem, stream, F);
    }
    return launch_status();
}

}  // namespace dspark
