// Device-side building blocks of the verifier kernels (verify.cu): batch parameters, per-block statistics / argmax / residual arithmetic, the
// combination of block statistics into row statistics, and the two-level inverse CDF.
#pragma once

#include <cuda_bf16.h>
#include <math.h>

#include <type_traits>

#include "common.cuh"

namespace dspark {

constexpr int kModeStats = 0, kModeGreedy = 1, kModeResid = 2, kModeHist = 3;
constexpr uint32_t kWindowDense = 0x80000000u;   // flag in TruncRow::size
constexpr int kHistBins = 1024;              // keys next to the row maximum that the streamed threshold search resolves
constexpr int kTaskNone = 0, kTaskResid = 1, kTaskBonus = 2;
constexpr int kCtrBonus = 12;                // header cell: bonus rows queued for the second pass (from the back of the queue)
constexpr int kSkipBonusSmemBytes = 9 * 1024;    // shared memory behind the stages for the offsets and that table
constexpr int kCtrRetry = 13;                // header cell: rows the threshold search looks at a second time
constexpr int kCellRetryUnits = 5;           // 64-bit header cell: unit counter of that second histogram pass
constexpr int kSkipBonusMaxRequests = 2048;  // the statistics pass keeps (row_offsets[r] - r) of the batch behind its stages
constexpr int kDecideThreads = 256;
constexpr float kNegInf = -INFINITY;

struct __align__(16) ResidTask {     // one rejected request queued for the residual pass
    int32_t request;
    int32_t row_t;                   // target row of the rejected position
    int64_t row_d;                   // physical draft row
    float cp, inv_zp, cq, inv_zq;    // row references (log2 domain) and 1 / row sums
    float u;                         // resample uniform of the rejected position
    float scale;                     // log2(e) / T of this request
    int32_t wslot;                   // which row of the block-sum array receives the result
    float tau;                       // truncation threshold of the target row (-inf: none): p = 0 below it
};

struct __align__(16) RequestRec {    // what the finalize kernel needs per request (written by decide)
    int32_t kind;                    // kTaskNone / kTaskResid / kTaskBonus
    int32_t row_t;                   // target row that emits the token
    int64_t row_d;                   // physical draft row of the rejected position
    float cp, inv_zp, cq, inv_zq;    // row references (log2 domain) and 1 / row sums
    float u;                         // resample uniform
    float scale;                     // log2(e) / T of this request
    float tau;                       // truncation threshold of the target row (-inf: none)
    int32_t pad;
};

struct __align__(16) TruncRow {      // per target row, for the streamed threshold search of top-k / top-p
    uint32_t kmax;                   // key of the row maximum
    uint32_t size;                   // keys in the window next to the maximum (0: row not truncated); bit 31: a wide
                                     // window of positive values only (counted without the branch, see consume_block)
    uint32_t cut2;                   // lowest value of the window, bf16 pattern in both halves
    float scale;                     // log2(e) / T
    float C;                         // row reference (log2 domain) of the statistics
    float Z;                         // row sum relative to C
    int32_t k;                       // top-k (0: off)
    float p;                         // top-p (>= 1: off)
};

struct VerifyParams {
    const unsigned char* target;
    const unsigned char* draft;
    long long tstride_bytes, dstride_bytes;
    int V, elem, row_bytes;
    int nblk, epb;                            // statistics blocks per row, elements per block
    int nblk_r, epb_r;                        // residual blocks per row, elements per block
    const int32_t* row_offsets;
    const int64_t* draft_row_start;
    const int32_t* draft_tokens;
    int R, n_rows_cap;
    float scale;                              // log2(e) / T (one temperature for the batch)
    const float* req_temp;                    // or: device [R] temperatures, one per request
    float* row_scale_t;                       // workspace: per target row / per draft row log2(e) / T
    float* row_scale_d;
    unsigned long long seed;
    int32_t* accepted_len;
    int32_t* out_tokens;
    float* out_p;
    float* out_q;
    int32_t* dev_status;
    // workspace
    int resid_cap;                            // capacity of the residual queue (R, or rows for c*)
    int* counters;                            // [0] queued residual tasks, [1] dev_status stand-in
    float2* stats_t;
    float2* stats_d;
    float2* stats_b;                          // [R][nblk]: block statistics of a bonus row streamed by the second pass, by
                                              // request (the draw kernel asks for them before it knows the row)
    ResidTask* resid;                         // queue of rejected requests (decide -> residual pass)
    RequestRec* req;                          // per request: outcome of decide for the finalize kernel
    unsigned long long launch_tag;            // unique per call: see unit_counter()
    float* wblk;                              // per request: residual block sums
    const float* tau;                         // per target row: top-k / top-p threshold (NULL: no truncation)
    int req_scale_smem;                       // 1: with that table, the requests' exponent scales are kept beside it and the
                                              // statistics pass needs no per-row scales (one temperature per request)
    int req_table;                            // statistics pass without the bonus rows: entries of the request-of-position
                                              // table kept in shared memory (0: none, the request is searched for)
    int skip_bonus;                           // 1: the statistics pass leaves the bonus rows out; the second pass streams
                                              // them for the requests that accepted every draft token (a rejected
                                              // request never needs its bonus row)
    const float2* draft_stats;                // per physical draft row: (reference, sum) handed over by the drafter (NULL:
                                              // the statistics pass streams the draft rows as well)
    TruncRow* trunc_rows;                     // workspace of the streamed threshold search
    unsigned int* trunc_bins;                 // [n_rows][kHistBins] key counts
    int32_t* trunc_flag;                      // [n_rows] 1: no window resolved the row (per-row search); 2: between the
                                              // two looks, the row waits for its deeper window
    int32_t* retry_rows;                      // rows of the second look (their number: counters[kCtrRetry])
    double* trunc_z;                          // [n_rows] mass of the kept set relative to the row reference, from the key
                                              // counts (<= 0: take the row's block sums); NULL without the streamed search
    int hist_retry;                           // histogram pass: 1 = second look, streams retry_rows only
};

template <int kMode> struct ModeCfg {
    static constexpr int kSrc = (kMode == kModeResid) ? 2 : 1;
    static constexpr int kVec = (kMode == kModeResid) ? kResidVec : kStatVec;
    static constexpr int kBlockBytes = kVec * 512;
    static constexpr int kPieceBytes = kBlockBytes * kConsumerWarps;   // per source
    static_assert(kPieceBytes * kSrc == kStageBytes, "a stage holds one piece of every source");
};

// ---------------------------------------------------------------------------------------
// Row bookkeeping shared by the kernels
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ int device_rows(const VerifyParams& P, bool* bad)
{
    int n = P.row_offsets[P.R];
    *bad = (n < P.R || n > P.n_rows_cap);
    return n < 0 ? 0 : (n > P.n_rows_cap ? P.n_rows_cap : n);
}

// Physical draft row of compact draft index ds (only needed with draft_row_start).
__device__ __forceinline__ long long draft_phys_row(const VerifyParams& P, int ds)
{
    if (!P.draft_row_start) return ds;
    int lo = 0, hi = P.R;                      // largest r with row_offsets[r] - r <= ds
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (P.row_offsets[mid] - mid <= ds) lo = mid; else hi = mid;
    }
    int j = ds - (P.row_offsets[lo] - lo);
    int len = P.row_offsets[lo + 1] - P.row_offsets[lo] - 1;
    if (j < 0 || j >= len) return -1;          // inconsistent offsets: caller substitutes a safe row
    return P.draft_row_start[lo] + j;
}

// Number of row streams a streamed pass walks.
template <int kMode>
__device__ __forceinline__ int stream_count(const VerifyParams& P, int n_rows)
{
    if (kMode == kModeStats) {
        const int nd = n_rows > P.R ? n_rows - P.R : 0;           // draft positions = target rows that are not bonus rows
        return (P.skip_bonus ? nd : n_rows) + (P.draft_stats ? 0 : nd);
    }
    if (kMode == kModeHist && P.hist_retry) {
        const int nr = __ldcg(&P.counters[kCtrRetry]);
        return nr < 0 ? 0 : (nr > n_rows ? n_rows : nr);
    }
    if (kMode == kModeGreedy || kMode == kModeHist) return n_rows;
    const int nq = __ldcg(&P.counters[0]);
    return nq > P.resid_cap ? P.resid_cap : (nq < 0 ? 0 : nq);
}

// Unit counters of the bulk-copy passes (64-bit cells behind the two int counters).  The residual and
// histogram passes find theirs zeroed by the statistics pass of the same call.  The statistics / greedy
// pass has no kernel of the call before it (a reset kernel would add a kernel boundary, 1.3 us, to every
// call), so its CTA 0 zeroes the counter and then publishes the call's launch tag -- a 64-bit value no
// earlier call used -- in the cell next to it; a CTA draws from the counter only after it has seen the tag
// (its first two units need no draw, so in practice nobody waits).  CTAs are dispatched in index order,
// CTA 0 is running before any other can ask; the wait is bounded all the same.  The kernel that follows
// the pass in every call clears the tag, so a replayed CUDA graph (same tag each time) starts clean.
template <int kMode>
__device__ __forceinline__ unsigned long long* unit_counter(const VerifyParams& P)
{
    return reinterpret_cast<unsigned long long*>(P.counters) +
           (kMode == kModeResid ? 2 : (kMode == kModeHist ? (P.hist_retry ? kCellRetryUnits : 3) : 1));
}
__device__ __forceinline__ unsigned long long* unit_tag(const VerifyParams& P)
{
    return reinterpret_cast<unsigned long long*>(P.counters) + 4;
}
struct __align__(16) UnitSlot {    // what the producer tells the consumers about a stage
    int s, piece;
    float scale;
    int pad;
    ResidTask task;                // residual pass: the task of stream s (loaded once per unit, not once per warp)
    TruncRow trunc;                // histogram pass: the window of row s (likewise)
};

// Walks the units (stream s, piece) owned by this CTA: unit index = s * ppr + piece, advancing by
// gridDim.x units per step without divisions.
struct UnitCursor {
    int s, piece, step_s, step_p, ppr;
    __device__ __forceinline__ void init(int ppr_)
    {
        ppr = ppr_;
        s = (int)blockIdx.x / ppr; piece = (int)blockIdx.x - s * ppr;
        step_s = (int)gridDim.x / ppr; step_p = (int)gridDim.x - step_s * ppr;
    }
    __device__ __forceinline__ void next()
    {
        s += step_s; piece += step_p;
        if (piece >= ppr) { piece -= ppr; ++s; }
    }
};

// ---------------------------------------------------------------------------------------
// Per-lane view of one block: kVec x 16 B, vector k of lane l is vector k*32+l of the block
// ---------------------------------------------------------------------------------------
template <int kElem> __device__ __forceinline__ uint32_t fill_word() { return kElem == 2 ? 0xFF80FF80u : 0xFF800000u; }

struct SmemFetch {
    const unsigned char* blk;
    __device__ __forceinline__ uint4 operator()(int vec, int) const { return *(const uint4*)(blk + vec * 16); }
};

template <int kElem>
struct GlobalFetch {
    const unsigned char* blk;     // block start in global memory (any alignment of kElem)
    __device__ __forceinline__ uint4 operator()(int vec, int nbytes) const
    {
        const int off = vec * 16;
        const unsigned char* p = blk + off;
        if (off + 16 <= nbytes && ((uintptr_t)p & 15u) == 0) return __ldg((const uint4*)p);
        uint32_t w[4] = {fill_word<kElem>(), fill_word<kElem>(), fill_word<kElem>(), fill_word<kElem>()};
        if (kElem == 4) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (off + (e + 1) * 4 <= nbytes) w[e] = __ldg((const uint32_t*)(p + e * 4));
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (off + (e + 1) * 2 <= nbytes) {
                    uint32_t h = __ldg((const unsigned short*)(p + e * 2));
                    w[e >> 1] = (e & 1) ? ((w[e >> 1] & 0x0000FFFFu) | (h << 16)) : ((w[e >> 1] & 0xFFFF0000u) | h);
                }
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

template <int kElem, int kVec, typename Fetch>
__device__ __forceinline__ void load_block(const Fetch& f, int nbytes, int lane, uint4 (&v)[kVec])
{
    if (nbytes == kVec * 512) {                  // full block: no per-vector tests
#pragma unroll
        for (int k = 0; k < kVec; ++k) v[k] = f(k * 32 + lane, nbytes);
    } else {
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            const int vec = k * 32 + lane;
            const uint32_t fw = fill_word<kElem>();
            v[k] = (vec * 16 < nbytes) ? f(vec, nbytes) : make_uint4(fw, fw, fw, fw);
        }
    }
}

__device__ __forceinline__ uint32_t word_of(const uint4& q, int i)
{
    return i == 0 ? q.x : (i == 1 ? q.y : (i == 2 ? q.z : q.w));
}
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b)
{
    __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162*>(&a), *reinterpret_cast<const __nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}

// Sampling statistics of one block: reference c = max(x) * scale (warp-uniform) and
// s = sum over the block of 2^(x*scale - c): exactly one exponential per element; the
// multiply-adds and the accumulation run as packed f32x2 instructions.
template <int kElem, int kVec>
__device__ __forceinline__ float2 block_stats(const uint4 (&v)[kVec], float scale)
{
    float mx;
    if (kElem == 2) {
        uint32_t m0 = v[0].x, m1 = v[0].y;
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            m0 = bf16x2_max(m0, v[k].x); m1 = bf16x2_max(m1, v[k].y);
            m0 = bf16x2_max(m0, v[k].z); m1 = bf16x2_max(m1, v[k].w);
        }
        m0 = bf16x2_max(m0, m1);
        mx = fmaxf(bf16lo(m0), bf16hi(m0));
    } else {
        float a = kNegInf, b = kNegInf;
#pragma unroll
        for (int k = 0; k < kVec; ++k) {
            a = fmaxf(a, __uint_as_float(v[k].x)); b = fmaxf(b, __uint_as_float(v[k].y));
            a = fmaxf(a, __uint_as_float(v[k].z)); b = fmaxf(b, __uint_as_float(v[k].w));
        }
        mx = fmaxf(a, b);
    }
    const float wmax = warp_max_f32(mx);
    if (wmax == kNegInf) {
        // nothing above -inf in this block: no mass -- unless a NaN hides behind the maximum (max drops NaN
        // operands; with a finite maximum the NaN would reach the sum below and flag the row by itself)
        bool nan = false;
#pragma unroll
        for (int k = 0; k < kVec; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t w = word_of(v[k], i);
                if (kElem == 2) nan |= (w & 0x7FFFu) > 0x7F80u || ((w >> 16) & 0x7FFFu) > 0x7F80u;
                else nan |= (w & 0x7FFFFFFFu) > 0x7F800000u;
            }
        return __any_sync(0xffffffffu, nan) ? make_float2(NAN, NAN) : make_float2(kNegInf, 0.0f);
    }
    const float c = __fmul_rn(wmax, scale);
    const uint64_t s2 = pack2(scale, scale), nc2 = pack2(-c, -c);
    uint64_t acc0 = pack2(0.f, 0.f), acc1 = acc0;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        if (kElem == 2) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t w = word_of(v[k], i);
                float t0, t1;
                unpack2(fma2(pack2(bf16lo(w), bf16hi(w)), s2, nc2), t0, t1);
                const uint64_t e2 = pack2(ex2_approx(t0), ex2_approx(t1));
                if (i & 1) acc1 = add2(acc1, e2); else acc0 = add2(acc0, e2);
            }
        } else {
            float t0, t1, t2, t3;
            unpack2(fma2(pack2(__uint_as_float(v[k].x), __uint_as_float(v[k].y)), s2, nc2), t0, t1);
            unpack2(fma2(pack2(__uint_as_float(v[k].z), __uint_as_float(v[k].w)), s2, nc2), t2, t3);
            acc0 = add2(acc0, pack2(ex2_approx(t0), ex2_approx(t1)));
            acc1 = add2(acc1, pack2(ex2_approx(t2), ex2_approx(t3)));
        }
    }
    float a0, a1, b0, b1;
    unpack2(acc0, a0, a1);
    unpack2(acc1, b0, b1);
    const float s = warp_sum_f32((a0 + a1) + (b0 + b1));
    return make_float2(c, s);
}

// Greedy statistics of one block: (max, lowest index attaining it); NaN never wins.
template <int kElem, int kVec>
__device__ __forceinline__ float2 block_argmax(const uint4 (&v)[kVec], int elem_base, int lane)
{
    constexpr int kPerVec = 16 / kElem;
    float best = kNegInf;
    int bi = 0x7fffffff;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        const int base = elem_base + (k * 32 + lane) * kPerVec;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w = word_of(v[k], i);
            if (kElem == 2) {
                float x0 = bf16lo(w), x1 = bf16hi(w);
                if (x0 > best) { best = x0; bi = base + 2 * i; }
                if (x1 > best) { best = x1; bi = base + 2 * i + 1; }
            } else {
                float x = __uint_as_float(w);
                if (x > best) { best = x; bi = base + i; }
            }
        }
    }
    const float wmax = warp_max_f32(best);
    const unsigned cand = (best == wmax) ? (unsigned)bi : 0x7fffffffu;
    const unsigned widx = __reduce_min_sync(0xffffffffu, cand);
    return make_float2(wmax, __int_as_float((int)widx));
}

// Residual max(0, p - q) of two neighbouring elements, packed; p = 2^(xt*scale-cp) * inv_zp,
// q likewise.  Every operation is a single IEEE-rounded step, so the scalar form below gives
// bit-identical values (the finalize kernel relies on that).
struct ResidConst {
    uint64_t s2, ncp2, ncq2, izp2, nizq2;
    float scale, cp, cq, inv_zp, inv_zq, tau;
    __device__ __forceinline__ void set(float scale_, float cp_, float inv_zp_, float cq_, float inv_zq_, float tau_)
    {
        scale = scale_; cp = cp_; cq = cq_; inv_zp = inv_zp_; inv_zq = inv_zq_; tau = tau_;
        s2 = pack2(scale, scale); ncp2 = pack2(-cp, -cp); ncq2 = pack2(-cq, -cq);
        izp2 = pack2(inv_zp, inv_zp); nizq2 = pack2(-inv_zq, -inv_zq);
    }
};
// A target logit below the truncation threshold of its row counts as -inf (p = 0): top-k / top-p.
__device__ __forceinline__ float cut_below(float x, float tau) { return x >= tau ? x : kNegInf; }

template <bool kCut>
__device__ __forceinline__ uint64_t resid_pair(uint64_t xt2, uint64_t xd2, const ResidConst& K)
{
    float a0, a1, b0, b1;
    if (kCut) {                    // without truncation (tau = -inf) the cut is the identity on every usable row
        unpack2(xt2, a0, a1);
        xt2 = pack2(cut_below(a0, K.tau), cut_below(a1, K.tau));
    }
    unpack2(fma2(xt2, K.s2, K.ncp2), a0, a1);
    unpack2(fma2(xd2, K.s2, K.ncq2), b0, b1);
    const uint64_t ep2 = pack2(ex2_approx(a0), ex2_approx(a1));
    const uint64_t eq2 = pack2(ex2_approx(b0), ex2_approx(b1));
    float w0, w1;
    unpack2(fma2(ep2, K.izp2, mul2(eq2, K.nizq2)), w0, w1);
    return pack2(fmaxf(w0, 0.0f), fmaxf(w1, 0.0f));
}
__device__ __forceinline__ float resid_elem(float xt, float xd, const ResidConst& K)
{
    const float ep = ex2_approx(__fmaf_rn(cut_below(xt, K.tau), K.scale, -K.cp));
    const float eq = ex2_approx(__fmaf_rn(xd, K.scale, -K.cq));
    return fmaxf(__fmaf_rn(ep, K.inv_zp, __fmul_rn(eq, -K.inv_zq)), 0.0f);
}

template <int kElem, int kVec, bool kCut>
__device__ __forceinline__ float block_resid(const uint4 (&vt)[kVec], const uint4 (&vd)[kVec], const ResidConst& K)
{
    uint64_t acc0 = pack2(0.f, 0.f), acc1 = acc0;
#pragma unroll
    for (int k = 0; k < kVec; ++k) {
        if (kElem == 2) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t a = word_of(vt[k], i), b = word_of(vd[k], i);
                const uint64_t w2 = resid_pair<kCut>(pack2(bf16lo(a), bf16hi(a)), pack2(bf16lo(b), bf16hi(b)), K);
                if (i & 1) acc1 = add2(acc1, w2); else acc0 = add2(acc0, w2);
            }
        } else {
            acc0 = add2(acc0, resid_pair<kCut>(pack2(__uint_as_float(vt[k].x), __uint_as_float(vt[k].y)),
                                         pack2(__uint_as_float(vd[k].x), __uint_as_float(vd[k].y)), K));
            acc1 = add2(acc1, resid_pair<kCut>(pack2(__uint_as_float(vt[k].z), __uint_as_float(vt[k].w)),
                                         pack2(__uint_as_float(vd[k].z), __uint_as_float(vd[k].w)), K));
        }
    }
    float a0, a1, b0, b1;
    unpack2(acc0, a0, a1);
    unpack2(acc1, b0, b1);
    return warp_sum_f32((a0 + a1) + (b0 + b1));
}

// What a consumer warp does with its block of the unit (stream s, piece).
template <int kElem, int kMode, typename Fetch>
__device__ __forceinline__ void consume_block(const VerifyParams& P, int s, int piece, int n_rows,
                                              int warp, int lane, const Fetch& f0, const Fetch& f1, float scale,
                                              const ResidTask* task = nullptr, const TruncRow* trunc = nullptr,
                                              unsigned int* shared_bins = nullptr)
{
    using M = ModeCfg<kMode>;
    if constexpr (kMode == kModeResid && std::is_same<Fetch, SmemFetch>::value) {
        if (task && task->row_d < 0) {
            // a bonus row inside the second pass (bulk-copy pipeline only): the stage holds a 32 KB piece of the row,
            // one 4 KB statistics block per warp (f0 points at this warp's 2 KB residual block)
            const int b4 = piece * kConsumerWarps + warp;
            if (b4 >= P.nblk) return;
            const int rem4 = P.row_bytes - b4 * kStatBlockBytes;
            uint4 v4[kStatVec];
            load_block<kElem, kStatVec>(SmemFetch{f0.blk + warp * (kStatBlockBytes - M::kBlockBytes)},
                                        rem4 < kStatBlockBytes ? rem4 : kStatBlockBytes, lane, v4);
            const float2 st = block_stats<kElem, kStatVec>(v4, task->scale);
            if (lane == 0) P.stats_b[(long long)task->wslot * P.nblk + b4] = st;
            return;
        }
    }
    const int nblk = (kMode == kModeResid) ? P.nblk_r : P.nblk;
    const int b = piece * kConsumerWarps + warp;
    if (b >= nblk) return;
    const int rem = P.row_bytes - b * M::kBlockBytes;
    const int nbytes = rem < M::kBlockBytes ? rem : M::kBlockBytes;
    uint4 v[M::kVec];
    load_block<kElem, M::kVec>(f0, nbytes, lane, v);
    if (kMode == kModeStats) {
        const float2 st = block_stats<kElem, M::kVec>(v, scale);
        if (lane == 0) {
            float2* dst = (s < n_rows) ? P.stats_t + (long long)s * nblk : P.stats_d + (long long)(s - n_rows) * nblk;
            dst[b] = st;
        }
    } else if (kMode == kModeGreedy) {
        const float2 st = block_argmax<kElem, M::kVec>(v, b * P.epb, lane);
        if (lane == 0) P.stats_t[(long long)s * nblk + b] = st;
    } else if (kMode == kModeHist) {
        // bf16 rows only.  Count the keys within the window next to the row maximum: a packed compare rejects the
        // pairs below it, the others take one atomic per token -- on the unit's histogram in shared memory where the
        // caller keeps one (it adds the non-empty bins to the row's counts afterwards), else on the row's counts.
        const TruncRow tr = trunc ? *trunc : P.trunc_rows[s];
        if (tr.size == 0u) return;
        unsigned int* bins = shared_bins ? shared_bins : P.trunc_bins + (long long)s * kHistBins;
        if (tr.size & kWindowDense) {
            // A wide window holds a good part of the row's tokens, and the branch below would be taken by some
            // thread of the warp for every pair.  All its values are positive, where the key distance is the
            // distance of the bit patterns: two subtractions, two compares and two predicated adds per pair
            // (a negative value or a NaN wraps to a distance beyond the window).
            const uint32_t bmax = tr.kmax & 0x7FFFu, size = tr.size & ~kWindowDense;
#pragma unroll
            for (int k = 0; k < M::kVec; ++k) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint32_t w = word_of(v[k], i);
                    const uint32_t d0 = bmax - (w & 0xFFFFu), d1 = bmax - (w >> 16);
                    if (d0 < size) atomicAdd(&bins[d0], 1u);
                    if (d1 < size) atomicAdd(&bins[d1], 1u);
                }
            }
            return;
        }
        const __nv_bfloat162 cut2 = *reinterpret_cast<const __nv_bfloat162*>(&tr.cut2);
#pragma unroll
        for (int k = 0; k < M::kVec; ++k) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t w = word_of(v[k], i);
                if (__hge2_mask(*reinterpret_cast<const __nv_bfloat162*>(&w), cut2)) {
                    const uint32_t d0 = tr.kmax - bf16_key(w & 0xFFFFu), d1 = tr.kmax - bf16_key(w >> 16);
                    if (d0 < tr.size) atomicAdd(&bins[d0], 1u);
                    if (d1 < tr.size) atomicAdd(&bins[d1], 1u);
                }
            }
        }
    } else {
        uint4 vd[M::kVec];
        load_block<kElem, M::kVec>(f1, nbytes, lane, vd);
        const ResidTask t = task ? *task : P.resid[s];
        ResidConst K;
        K.set(t.scale, t.cp, t.inv_zp, t.cq, t.inv_zq, t.tau);
        const float w = (t.tau == kNegInf) ? block_resid<kElem, M::kVec, false>(v, vd, K)
                                           : block_resid<kElem, M::kVec, true>(v, vd, K);
        if (lane == 0) P.wblk[(long long)t.wslot * nblk + b] = w;
    }
}

// Exponent scale log2(e)/T of row stream s (per-request temperatures are expanded per row).
template <int kMode>
__device__ __forceinline__ float stream_scale(const VerifyParams& P, int s, int n_rows, int n_streams)
{
    if (kMode != kModeStats || !P.req_temp || s >= n_streams) return P.scale;
    return (s < n_rows) ? __ldcg(&P.row_scale_t[s]) : __ldcg(&P.row_scale_d[s - n_rows]);
}

// Source addresses of a unit (producer / direct path).
template <int kMode>
__device__ __forceinline__ void unit_sources(const VerifyParams& P, int s, int piece, int n_rows,
                                             const unsigned char*& src0, const unsigned char*& src1, int& bytes,
                                             const ResidTask* task = nullptr, long long draft_row = -2)
{
    using M = ModeCfg<kMode>;
    const long long off = (long long)piece * M::kPieceBytes;
    const long long rem = (long long)P.row_bytes - off;
    bytes = (int)(rem < M::kPieceBytes ? rem : M::kPieceBytes);
    src1 = nullptr;
    if (kMode == kModeResid) {
        const ResidTask t = task ? *task : P.resid[s];
        src0 = P.target + (long long)t.row_t * P.tstride_bytes + off;
        src1 = t.row_d >= 0 ? P.draft + t.row_d * P.dstride_bytes + off : nullptr;   // a bonus row: the target row alone
    } else if (s < n_rows) {
        src0 = P.target + (long long)s * P.tstride_bytes + off;
    } else {
        // draft_row: the physical row where the caller has found it already (-1: inconsistent offsets), else -2
        const long long phys = draft_row != -2 ? draft_row : draft_phys_row(P, s - n_rows);
        src0 = (phys >= 0 ? P.draft + phys * P.dstride_bytes : P.target) + off;
    }
}

// ---------------------------------------------------------------------------------------
// Row statistics from block statistics: reference C = max_b c_b, sum S = sum_b s_b 2^(c_b-C).
// One pass over the entries (4 per lane in flight), online rescaling per lane, then a warp
// combine.  Called by one full warp; the result is valid in every lane.
// ---------------------------------------------------------------------------------------
struct RowAcc {
    float C;
    double S;
    __device__ __forceinline__ void init() { C = kNegInf; S = 0.0; }
    __device__ __forceinline__ void add(float2 e)
    {
        if (e.x != e.x || e.y != e.y) { S = NAN; return; }      // a NaN anywhere must survive
        if (!(e.x > kNegInf)) return;                           // empty block
        if (e.x > C) { S *= (double)ex2_approx(C - e.x); C = e.x; }   // C = -inf: factor 0, S was 0
        S += (double)(e.y * ex2_approx(e.x - C));
    }
    __device__ __forceinline__ void finish()
    {
        const float Cw = warp_max_f32(C);
        double s = (C > kNegInf) ? S * (double)ex2_approx(C - Cw) : (S != S ? S : 0.0);
        S = warp_sum_f64(s);
        C = Cw;
    }
};

__device__ __forceinline__ void combine_rows(const float2* __restrict__ a, const float2* __restrict__ b,
                                             int nblk, int lane, RowAcc& A, RowAcc& Bc)
{
    A.init(); Bc.init();
    for (int base = 0; base < nblk; base += 128) {
        float2 ea[4], eb[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int i = base + k * 32 + lane;
            ea[k] = (i < nblk) ? __ldcg(&a[i]) : make_float2(kNegInf, 0.f);
            eb[k] = (b && i < nblk) ? __ldcg(&b[i]) : make_float2(kNegInf, 0.f);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) { A.add(ea[k]); Bc.add(eb[k]); }
    }
    A.finish();
    if (b) Bc.finish();
}

__device__ __forceinline__ float load_logit(const unsigned char* base, long long row, long long stride_bytes,
                                            int elem, int v)
{
    const unsigned char* p = base + row * stride_bytes + (long long)v * elem;
    if (elem == 2) return __uint_as_float((uint32_t)__ldg((const unsigned short*)p) << 16);
    return __ldg((const float*)p);
}

__device__ __forceinline__ bool row_usable(float C, double S)
{
    return C > kNegInf && C < INFINITY && S > 0.0 && S < INFINITY;   // false for NaN
}

// ---------------------------------------------------------------------------------------
// Inverse CDF in vocabulary order, two levels, one warp:
//   level 1  over per-block values (residual block sums, or block masses of p).  Up to 256 blocks
//            are held in registers, lane-strided (value k of lane l is block k*32+l): chunk totals
//            by warp reduction, then one warp scan inside the chunk that holds the crossing.
//            Longer rows walk memory in chunks of 32 blocks.
//   level 2  inside that one block: every lane copies its own contiguous run of raw logits into a
//            padded (bank-conflict-free) strip of shared memory, sums its values, the warp scans
//            the lane sums, and the lane that holds the crossing walks its cached values.
// All running sums are fp64 sums of the fp32 values in index order.
// ---------------------------------------------------------------------------------------
template <typename F>
__device__ __forceinline__ double warp_total(int n, int lane, F val)
{
    double t = 0.0;
#pragma unroll 4
    for (int i = lane; i < n; i += 32) t += (double)val(i);
    return warp_sum_f64(t);
}

__device__ __forceinline__ double warp_incl_scan_f64(double x, int lane)
{
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += t;
    }
    return x;
}

// Level 1 from registers: x[k] = value of block k*32+lane (0 beyond n), n <= 256.  thr = u * total.
// Returns the block index (never -1 when total > 0: falls back to the last positive block), and the
// exclusive sum before it.
__device__ __forceinline__ int level1_registers(const float (&x)[8], int n, int lane, double u, double& before,
                                                double& total)
{
    double ct[8];
    total = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) { ct[k] = (k * 32 < n) ? warp_sum_f64((double)x[k]) : 0.0; total += ct[k]; }
    const double thr = u * total;
    double run = 0.0;
    int kc = -1;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        if (kc < 0 && k * 32 < n) {
            if (run + ct[k] > thr) kc = k; else run += ct[k];
        }
    }
    int lastp = -1;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const unsigned pos = __ballot_sync(0xffffffffu, x[k] > 0.f);
        if (pos) lastp = k * 32 + (31 - __clz(pos));
    }
    if (kc < 0) { before = total; return lastp >= 0 ? lastp : 0; }      // only by rounding
    float xc = 0.f;
#pragma unroll
    for (int k = 0; k < 8; ++k) if (k == kc) xc = x[k];
    const double incl = warp_incl_scan_f64((double)xc, lane);
    const unsigned hit = __ballot_sync(0xffffffffu, run + incl > thr && kc * 32 + lane < n);
    int l;
    if (hit) l = __ffs(hit) - 1;
    else { const unsigned pos = __ballot_sync(0xffffffffu, xc > 0.f); l = pos ? 31 - __clz(pos) : 0; }
    before = run + __shfl_sync(0xffffffffu, incl - (double)xc, l);
    return kc * 32 + l;
}

// Level 1 from memory for rows with more than 256 blocks: first index i in [0, n) whose inclusive
// running sum exceeds thr, else the last positive index.
template <typename F>
__device__ __forceinline__ int level1_memory(int n, int lane, F val, double thr, double& before)
{
    double run = 0.0;
    int lastp = -1;
    for (int c0 = 0; c0 < n; c0 += 32) {
        const int i = c0 + lane;
        const float x = i < n ? val(i) : 0.f;
        const double incl = warp_incl_scan_f64((double)x, lane);
        const unsigned pos = __ballot_sync(0xffffffffu, x > 0.f);
        if (pos) lastp = c0 + (31 - __clz(pos));
        const unsigned hit = __ballot_sync(0xffffffffu, run + incl > thr && i < n);
        if (hit) {
            const int l = __ffs(hit) - 1;
            before = run + __shfl_sync(0xffffffffu, incl - (double)x, l);
            return c0 + l;
        }
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    before = run;
    return lastp >= 0 ? lastp : 0;
}

// Shared-memory strip of one warp for level 2.
template <int kElem>
struct Level2Scratch {
    static constexpr int kWordsStat = kStatBlockBytes / 32 / 4;      // raw words per lane, 4 KB block
    static constexpr int kPerStat = kStatBlockBytes / 32 / kElem;    // elements per lane, 4 KB block
    uint32_t raw_t[32 * (kWordsStat + 1)];
    uint32_t raw_d[32 * (kWordsStat / 2 + 1)];
    float w[32 * (kPerStat + 1)];
};

// Copies this lane's run (kWords 32-bit words starting at element e_lane of `row`) into its strip.
template <int kElem, int kWords>
__device__ __forceinline__ void stage_own_run(const unsigned char* row, int e_lane, int n_mine, uint32_t* strip)
{
    const unsigned char* p = row + (long long)e_lane * kElem;
    constexpr int kPer = kWords * 4 / kElem;
    if (n_mine == kPer && ((uintptr_t)p & 15u) == 0) {
#pragma unroll
        for (int v = 0; v < kWords / 4; ++v) {
            const uint4 q = __ldg((const uint4*)(p + 16 * v));
            strip[4 * v] = q.x; strip[4 * v + 1] = q.y; strip[4 * v + 2] = q.z; strip[4 * v + 3] = q.w;
        }
    } else if (kElem == 4) {
        for (int k = 0; k < n_mine; ++k) strip[k] = __ldg((const uint32_t*)(p + 4 * k));
    } else {
        for (int k = 0; k < n_mine; k += 2) {
            uint32_t lo = __ldg((const unsigned short*)(p + 2 * k));
            uint32_t hi = (k + 1 < n_mine) ? __ldg((const unsigned short*)(p + 2 * k + 2)) : 0xFF80u;
            strip[k >> 1] = lo | (hi << 16);
        }
    }
}
template <int kElem>
__device__ __forceinline__ float strip_elem(const uint32_t* strip, int k)
{
    if (kElem == 4) return __uint_as_float(strip[k]);
    const uint32_t w = strip[k >> 1];
    return (k & 1) ? bf16hi(w) : bf16lo(w);
}

// Level 2 over one block of kBlockBytes per row starting at element e0 (cnt valid elements): lane l
// owns elements [l*per, (l+1)*per).  f(xt, xd) is the value of an element.  Returns the element
// index inside the block.
template <int kElem, int kBlockBytes, bool kTwoRows, typename F>
__device__ __forceinline__ int level2_block(const unsigned char* trow, const unsigned char* drow, int e0, int cnt,
                                            int lane, double thr, F f, Level2Scratch<kElem>& S)
{
    constexpr int kWords = kBlockBytes / 32 / 4;
    constexpr int kPer = kBlockBytes / 32 / kElem;
    const int i0 = lane * kPer;
    int n_mine = cnt - i0;
    n_mine = n_mine < 0 ? 0 : (n_mine > kPer ? kPer : n_mine);
    uint32_t* st = S.raw_t + lane * (kWords + 1);
    uint32_t* sd = S.raw_d + lane * (kWords + 1);
    float* sw = S.w + lane * (kPer + 1);
    stage_own_run<kElem, kWords>(trow, e0 + i0, n_mine, st);
    if (kTwoRows) stage_own_run<kElem, kWords>(drow, e0 + i0, n_mine, sd);
    double mine = 0.0;
    int lastp = -1;
#pragma unroll 4
    for (int k = 0; k < n_mine; ++k) {
        const float w = f(strip_elem<kElem>(st, k), kTwoRows ? strip_elem<kElem>(sd, k) : 0.f);
        sw[k] = w;
        mine += (double)w;
        if (w > 0.f) lastp = i0 + k;
    }
    const double incl = warp_incl_scan_f64(mine, lane);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lastp = max(lastp, __shfl_xor_sync(0xffffffffu, lastp, o));
    const unsigned hit = __ballot_sync(0xffffffffu, incl > thr && n_mine > 0);
    if (!hit) return lastp >= 0 ? lastp : 0;              // only by rounding between the two levels
    // the whole warp scans the cached values of the lane that holds the crossing
    const int src = __ffs(hit) - 1;
    const double run0 = __shfl_sync(0xffffffffu, incl - mine, src);
    const int n_src = __shfl_sync(0xffffffffu, n_mine, src);
    const float* ssrc = S.w + src * (kPer + 1);
    __syncwarp();
    double run = run0;
    int found = -1;
#pragma unroll
    for (int c = 0; c < kPer; c += 32) {
        const float w = (c + lane < n_src) ? ssrc[c + lane] : 0.f;
        const double inc = warp_incl_scan_f64((double)w, lane);
        const unsigned h2 = __ballot_sync(0xffffffffu, run + inc > thr && c + lane < n_src);
        if (found < 0 && h2) found = c + __ffs(h2) - 1;
        run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (found < 0) found = n_src - 1;                     // only by rounding between the two sums
    return src * kPer + found;
}


// Workspace of the verifiers (caller-provided, any content on entry), offsets in bytes.
struct Workspace {
    size_t counters, stats_t, stats_d, stats_b, resid, req, wblk, scale_t, scale_d, tau, trunc_rows, trunc_bins, trunc_flag, retry_rows, trunc_z;
    size_t total;
};
inline Workspace workspace_layout(int R, int n_rows, int V)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t nblk = (size_t)blocks_per_row(V, 4, kStatBlockBytes);
    const size_t nblk_r = (size_t)blocks_per_row(V, 4, kResidBlockBytes);
    Workspace w;
    size_t o = 0;
    w.counters = o; o += up(64 * sizeof(int));
    w.stats_t = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.stats_d = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.stats_b = o;  o += up((size_t)R * nblk * sizeof(float2));
    w.resid = o;    o += up((size_t)R * sizeof(ResidTask));
    w.req = o;      o += up((size_t)R * sizeof(RequestRec));
    w.wblk = o;     o += up((size_t)R * nblk_r * sizeof(float));
    w.scale_t = o;  o += up((size_t)n_rows * sizeof(float));
    w.scale_d = o;  o += up((size_t)n_rows * sizeof(float));
    w.tau = o;      o += up((size_t)n_rows * sizeof(float));
    w.trunc_rows = o; o += up((size_t)n_rows * sizeof(TruncRow));
    w.trunc_bins = o; o += up((size_t)n_rows * kHistBins * sizeof(unsigned int));
    w.trunc_flag = o; o += up((size_t)(n_rows + 2) * sizeof(int32_t));   // + the fallback's row counter and row count
    w.retry_rows = o; o += up((size_t)n_rows * sizeof(int32_t));
    w.trunc_z = o;    o += up((size_t)n_rows * sizeof(double));
    w.total = o;
    return w;
}

// Scratch of greedy verification alone (what dspark_verify_greedy_static must fit into its array): the header
// and the per-block (max, argmax) of every target row.
struct GreedyWorkspace { size_t counters, stats, total; };
inline GreedyWorkspace greedy_workspace_layout(int n_rows, int V, int elem)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t nblk = (size_t)blocks_per_row(V, elem, kStatBlockBytes);
    GreedyWorkspace w;
    size_t o = 0;
    w.counters = o; o += up(64 * sizeof(int));
    w.stats = o;    o += up((size_t)n_rows * nblk * sizeof(float2));
    w.total = o;
    return w;
}

}  // namespace dspark
