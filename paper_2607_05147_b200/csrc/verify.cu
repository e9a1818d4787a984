// dspark_verify / dspark_verify_greedy: the fused ragged-batch speculative verifier
// (acceptance rule of Section 2.1; bonus token of Section 1; flat ragged rows of Section 4.3).
//
// Pass structure (all on the caller's stream, no host round trip):
//   stream   every target / draft row is read from HBM exactly once.  A row is cut into
//            4 KB blocks; one warp reduces one block to (reference, sum of 2^(x*scale-ref))
//            [sampling] or (max, lowest argmax) [greedy].  Persistent CTAs; a producer warp
//            feeds a ring of 32 KB shared-memory stages with 1-D bulk async copies
//            (cp.async.bulk + mbarrier), eight consumer warps drain it.  The 32 KB units are
//            handed out through a grid-wide counter, so all CTAs finish together.
//   decide   one CTA per request: combines block statistics into row statistics, gathers
//            p(x), q(x), runs the accept tests (Philox), finds the first rejection, writes the
//            accepted prefix, and queues a rejected position for the residual pass.
//   residual second read of the rejected position's row pair only: per-2KB-block sums of
//            max(0, p - q), same bulk-copy pipeline with two sources per stage.
//   finalize one warp per request: inverse CDF over block values (residual sums, or the saved
//            statistics of the bonus row), then inside the one block that holds the crossing.
#include <cuda_bf16.h>
#include <cstdio>
#include <math.h>

#include "common.cuh"

namespace dspark {

constexpr int kModeStats = 0, kModeGreedy = 1, kModeResid = 2, kModeHist = 3;
constexpr int kHistBins = 1024;              // keys next to the row maximum that the streamed threshold search resolves
constexpr int kTaskNone = 0, kTaskResid = 1, kTaskBonus = 2;
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
    uint32_t size;                   // keys in the window next to the maximum (0: row not truncated)
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
    ResidTask* resid;                         // queue of rejected requests (decide -> residual pass)
    RequestRec* req;                          // per request: outcome of decide for the finalize kernel
    unsigned long long launch_tag;            // unique per call: see unit_counter()
    float* wblk;                              // per request: residual block sums
    const float* tau;                         // per target row: top-k / top-p threshold (NULL: no truncation)
    TruncRow* trunc_rows;                     // workspace of the streamed threshold search
    unsigned int* trunc_bins;                 // [n_rows][kHistBins] key counts
    int32_t* trunc_flag;                      // [n_rows] 1: the window did not resolve the row (per-row search)
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
    if (kMode == kModeStats) return n_rows + (n_rows > P.R ? n_rows - P.R : 0);
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
    return reinterpret_cast<unsigned long long*>(P.counters) + (kMode == kModeResid ? 2 : (kMode == kModeHist ? 3 : 1));
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
                                              const ResidTask* task = nullptr)
{
    using M = ModeCfg<kMode>;
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
        // bf16 rows only.  Count the keys within the window next to the row maximum: a packed compare rejects
        // almost every pair, the few tokens of the tail take one atomic each.
        const TruncRow tr = P.trunc_rows[s];
        if (tr.size == 0u) return;
        const __nv_bfloat162 cut2 = *reinterpret_cast<const __nv_bfloat162*>(&tr.cut2);
        unsigned int* bins = P.trunc_bins + (long long)s * kHistBins;
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
                                             const ResidTask* task = nullptr)
{
    using M = ModeCfg<kMode>;
    const long long off = (long long)piece * M::kPieceBytes;
    const long long rem = (long long)P.row_bytes - off;
    bytes = (int)(rem < M::kPieceBytes ? rem : M::kPieceBytes);
    src1 = nullptr;
    if (kMode == kModeResid) {
        const ResidTask t = task ? *task : P.resid[s];
        src0 = P.target + (long long)t.row_t * P.tstride_bytes + off;
        src1 = P.draft + t.row_d * P.dstride_bytes + off;
    } else if (s < n_rows) {
        src0 = P.target + (long long)s * P.tstride_bytes + off;
    } else {
        const long long phys = draft_phys_row(P, s - n_rows);
        src0 = (phys >= 0 ? P.draft + phys * P.dstride_bytes : P.target) + off;
    }
}

// ---------------------------------------------------------------------------------------
// Streamed pass, bulk-copy pipeline: kStages x 32 KB of shared memory per CTA.
// ---------------------------------------------------------------------------------------
template <int kElem, int kMode>
__global__ void __launch_bounds__(kStreamThreads, 3) stream_bulk_kernel(VerifyParams P)
{
    using M = ModeCfg<kMode>;
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ UnitSlot s_unit[kStages];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kConsumerWarps); }
        s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait();                                  // everything below reads what earlier kernels wrote

    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (kMode != kModeResid && kMode != kModeHist && blockIdx.x == 0 && tid == 0) {
        P.counters[0] = 0;                       // residual queue, filled by the decide kernel
        *unit_counter<kModeResid>(P) = 0ull;     // unit counters of the passes that follow this one in the call
        *unit_counter<kModeHist>(P) = 0ull;
        *unit_counter<kMode>(P) = 0ull;          // and this pass's own, published by the tag
        __threadfence();
        atomicExch(unit_tag(P), P.launch_tag);
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int n_streams = stream_count<kMode>(P, n_rows);
    const int nblk = (kMode == kModeResid) ? P.nblk_r : P.nblk;
    const int ppr = (nblk + kConsumerWarps - 1) / kConsumerWarps;
    const long long total = (long long)n_streams * ppr;
    volatile int* abort_flag = &s_abort;

    if (warp == kConsumerWarps) {
        // ---------------- producer warp: lane 0 draws the units and issues the copies ----
        // The first kStages units of a CTA follow from its index; every further one comes from a counter
        // shared by the grid, so an SM that gets its data sooner takes more units and all CTAs finish
        // together.  A draw is issued right after the copies of a turn and is needed two turns later.
        unsigned long long* ctr = unit_counter<kMode>(P);
        // logit rows are read once (a rejected pair twice): their lines are the first to go, so that what the
        // short kernels of the step keep re-reading -- statistics, tokens, offsets, scheduler state -- stays in L2
        const uint64_t pol_first = l2_policy_evict_first();
        bool counter_ready = (kMode == kModeResid || kMode == kModeHist);    // zeroed by an earlier kernel
        int it = 0;
        // one turn of the pipeline with the unit held in `mine`; `mine` then receives the unit of the turn after
        // next (the first kStages units of a CTA are fixed, so the stages fill without waiting for the counter)
        auto turn = [&](long long& mine) -> bool {
            const long long u = __shfl_sync(0xffffffffu, mine, 0);
            const int st = it % kStages;
            const uint32_t ph = (uint32_t)(it / kStages) & 1u;
            const bool live = u < total;
            UnitSlot slot;
            const unsigned char *src0 = nullptr, *src1 = nullptr;
            int bytes = 0;
            if (lane == 0) {
                if (live) {
                    slot.s = total <= 0x7fffffffll ? (int)((unsigned)u / (unsigned)ppr) : (int)(u / ppr);
                    slot.piece = (int)(u - (long long)slot.s * ppr);
                    if (kMode == kModeResid) slot.task = P.resid[slot.s];
                    unit_sources<kMode>(P, slot.s, slot.piece, n_rows, src0, src1, bytes, kMode == kModeResid ? &slot.task : nullptr);
                    slot.scale = stream_scale<kMode>(P, slot.s, n_rows, n_streams);
                } else {
                    slot.s = -1; slot.piece = 0; slot.scale = 0.f;
                }
            }
            if (*abort_flag) return false;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&empty_bar[st], ph ^ 1u))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                return false;
            }
            if (lane == 0) {
                // read by the consumers after the barrier below completes
                s_unit[st].s = slot.s; s_unit[st].piece = slot.piece; s_unit[st].scale = slot.scale;
                if (kMode == kModeResid) s_unit[st].task = slot.task;
                if (live) {
                    unsigned char* dst = stage_mem + st * kStageBytes;
                    mbar_arrive_expect_tx(&full_bar[st], (uint32_t)(bytes * M::kSrc));
                    bulk_g2s_hint(dst, src0, (uint32_t)bytes, &full_bar[st], pol_first);
                    if (M::kSrc == 2) bulk_g2s_hint(dst + M::kPieceBytes, src1, (uint32_t)bytes, &full_bar[st], pol_first);
                    if (!counter_ready && !(counter_ready = wait_for_tag(unit_tag(P), P.launch_tag))) {
                        atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT);
                        *abort_flag = 1;
                        mine = total;
                    } else {
                        mine = (long long)gridDim.x * kStages + (long long)atomicAdd(ctr, 1ull);   // needed two turns from now
                    }
                } else {
                    mbar_arrive(&full_bar[st]);    // end marker: no data follows
                }
            }
            __syncwarp();
            if (live) ++it;
            return live;
        };
        static_assert(kStages == 2, "the producer keeps one pending unit per stage");
        long long unit_a = blockIdx.x, unit_b = (long long)blockIdx.x + gridDim.x;
        while (turn(unit_a) && turn(unit_b)) {}
        if (*abort_flag) {
            // leave only after every copy already issued has landed (bounded)
            for (int k = 0; k < kStages && k < it; ++k) {
                const int jt = it - 1 - k;
                mbar_wait_bounded(&full_bar[jt % kStages], (uint32_t)(jt / kStages) & 1u);
            }
        }
    } else {
        // ---------------- consumer warps --------------------------------------------------
        for (int it = 0;; ++it) {
            const int st = it % kStages;
            const uint32_t ph = (uint32_t)(it / kStages) & 1u;
            if (*abort_flag) break;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&full_bar[st], ph))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                break;
            }
            const int unit_s = s_unit[st].s, unit_piece = s_unit[st].piece;
            const float unit_scale = s_unit[st].scale;
            if (unit_s < 0) break;
            unsigned char* sp = stage_mem + st * kStageBytes + warp * M::kBlockBytes;
            SmemFetch f0{sp}, f1{sp + M::kPieceBytes};
            consume_block<kElem, kMode>(P, unit_s, unit_piece, n_rows, warp, lane, f0, f1, unit_scale,
                                        kMode == kModeResid ? &s_unit[st].task : nullptr);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[st]);
        }
    }
}

// Streamed pass without the bulk copy: each warp loads its block straight from global
// memory (16-byte loads where the address allows, element loads otherwise).  Taken when
// a pointer, stride or row length breaks the 16-byte rules of the bulk copy.
template <int kElem, int kMode>
__global__ void __launch_bounds__(kConsumerWarps * 32, 2) stream_direct_kernel(VerifyParams P)
{
    using M = ModeCfg<kMode>;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_wait();
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (kMode != kModeResid && kMode != kModeHist && blockIdx.x == 0 && tid == 0) {
        P.counters[0] = 0;
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int n_streams = stream_count<kMode>(P, n_rows);
    const int nblk = (kMode == kModeResid) ? P.nblk_r : P.nblk;
    UnitCursor cur;
    cur.init((nblk + kConsumerWarps - 1) / kConsumerWarps);
    for (; cur.s < n_streams; cur.next()) {
        const unsigned char *src0, *src1;
        int bytes;
        unit_sources<kMode>(P, cur.s, cur.piece, n_rows, src0, src1, bytes);
        GlobalFetch<kElem> f0{src0 + warp * M::kBlockBytes};
        GlobalFetch<kElem> f1{(kMode == kModeResid ? src1 : src0) + warp * M::kBlockBytes};
        consume_block<kElem, kMode>(P, cur.s, cur.piece, n_rows, warp, lane, f0, f1,
                                    stream_scale<kMode>(P, cur.s, n_rows, n_streams));
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

// ---------------------------------------------------------------------------------------
// top-k / top-p truncation of the target distribution inside the verifier (bf16 rows).
// The kept set of a row is {v : x_v >= tau}; tau is found exactly on the 16-bit keys:
//   trunc_prep    per target row: row maximum m (recovered exactly from the statistics: the reference
//                 c = m * scale determines the bf16 value m), the window of keys between m and m - 8 T (at
//                 most kHistBins keys), zeroed counters;
//   stream<Hist>  one more streamed pass over the target rows counts the keys inside the window;
//   trunc_scan    per row: masses count * 2^(value * scale - C), prefix sums, the top-k and top-p
//                 thresholds; a row whose threshold lies beyond the window is flagged for the per-row
//                 search of truncate.cu (flat rows: rare);
//   trunc_sums    per (row, block): the block sum of the statistics restricted to x >= tau (only blocks
//                 whose maximum reaches tau are read again).
// ---------------------------------------------------------------------------------------
struct TruncArgs {
    const int32_t* top_k; const float* top_p; const float* temperatures; float temperature;
    float* tau;                       // per target row
};

__global__ void __launch_bounds__(256) trunc_prep_kernel(VerifyParams P, TruncArgs T)
{
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (row >= n_rows) return;
    int lo = 0, hi = P.R;                                   // largest r with row_offsets[r] <= row
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (P.row_offsets[mid] <= row) lo = mid; else hi = mid;
    }
    const int r = lo;
    const int k = T.top_k ? T.top_k[r] : 0;
    const float pf = T.top_p ? T.top_p[r] : 1.f;
    const float temp = T.temperatures ? T.temperatures[r] : T.temperature;
    RowAcc A, D;
    combine_rows(P.stats_t + (long long)row * P.nblk, nullptr, P.nblk, lane, A, D);
    TruncRow tr;
    tr.kmax = 0u; tr.size = 0u; tr.cut2 = 0u; tr.scale = 0.f; tr.C = A.C; tr.Z = (float)A.S; tr.k = 0; tr.p = 1.f;
    const bool use_k = k > 0 && k < P.V, use_p = pf < 1.f;
    if ((use_k || use_p) && temp > 0.f && temp < INFINITY && row_usable(A.C, A.S)) {
        const float scale = (float)(1.4426950408889634 / (double)temp);
        const __nv_bfloat16 mb = __float2bfloat16_rn(A.C / scale);      // the bf16 maximum behind c = m * scale
        const float m = __bfloat162float(mb);
        const uint32_t kmax = bf16_key((uint32_t)__bfloat16_as_ushort(mb));
        float lo_val = m - 8.f * temp;
        if (use_k && k <= P.nblk) {
            // every block maximum is an element of the row, so the k-th largest logit is at least the k-th
            // largest block maximum: the window reaches down to it (rank by counting, 64-128 blocks)
            const float2* st = P.stats_t + (long long)row * P.nblk;
            float kth = kNegInf;
            if (P.nblk <= 128) {                             // block references in registers, compared through shuffles
                float c[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) c[q] = (q * 32 + lane < P.nblk) ? __ldcg(&st[q * 32 + lane]).x : kNegInf;
                int rank[4] = {0, 0, 0, 0};                  // blocks that come before mine in descending order
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2) {
                    if (q2 * 32 >= P.nblk) break;
                    for (int l2 = 0; l2 < 32; ++l2) {
                        const float cj = __shfl_sync(0xffffffffu, c[q2], l2);
                        const int j = q2 * 32 + l2;
#pragma unroll
                        for (int q = 0; q < 4; ++q) rank[q] += (cj > c[q]) || (cj == c[q] && j < q * 32 + lane);
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (q * 32 + lane < P.nblk && rank[q] == k - 1) kth = c[q];
            } else {
                for (int b0 = lane; b0 < P.nblk; b0 += 32) {
                    const float cb = __ldcg(&st[b0]).x;
                    int rank = 0;
                    for (int j = 0; j < P.nblk; ++j) {
                        const float cj = __ldcg(&st[j]).x;
                        rank += (cj > cb) || (cj == cb && j < b0);
                    }
                    if (rank == k - 1) kth = cb;
                }
            }
            kth = warp_max_f32(kth);
            if (kth > kNegInf) lo_val = fminf(lo_val, __bfloat162float(__float2bfloat16_rn(kth / scale)));
        }
        const uint32_t klo = bf16_key((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rd(lo_val)));
        uint32_t size = kHistBins;
        if (klo <= kmax && kmax - klo + 1u < (uint32_t)kHistBins) size = kmax - klo + 1u;
        if (size > kmax + 1u) size = kmax + 1u;                          // keys 0 .. kmax exist
        const uint32_t cb = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(bf16_key_value(kmax - (size - 1u))));
        tr.kmax = kmax; tr.size = size; tr.cut2 = cb | (cb << 16); tr.scale = scale;
        tr.k = use_k ? k : 0; tr.p = use_p ? pf : 1.f;
        unsigned int* bins = P.trunc_bins + (long long)row * kHistBins;
        for (uint32_t i = lane; i < size; i += 32) bins[i] = 0u;
    }
    if (lane == 0) { P.trunc_rows[row] = tr; T.tau[row] = kNegInf; P.trunc_flag[row] = 0; }
    if (row == 0 && lane == 0) P.trunc_flag[P.n_rows_cap] = 0;          // work counter of the per-row fallback
}

constexpr int kScanThreads = 256;
__global__ void __launch_bounds__(kScanThreads) trunc_scan_kernel(VerifyParams P, TruncArgs T)
{
    constexpr int kPer = kHistBins / kScanThreads;
    __shared__ unsigned long long s_c[kScanThreads / 32];
    __shared__ double s_m[kScanThreads / 32];
    __shared__ int s_hit_k, s_hit_p;
    __shared__ double s_zk;
    pdl_wait();
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    bool bad_rows;
    if (row >= device_rows(P, &bad_rows)) return;
    const TruncRow tr = P.trunc_rows[row];
    if (tr.size == 0u) return;
    if (tid == 0) { s_hit_k = 0x7fffffff; s_hit_p = 0x7fffffff; }
    const unsigned int* bins = P.trunc_bins + (long long)row * kHistBins;
    unsigned int cnt[kPer];
    double mass[kPer];
    unsigned long long lc = 0ull;
    double lm = 0.0;
#pragma unroll
    for (int j = 0; j < kPer; ++j) {
        const uint32_t d = (uint32_t)(tid * kPer + j);
        cnt[j] = d < tr.size ? __ldcg(&bins[d]) : 0u;
        // mass of a key relative to the row reference C, as the statistics count it
        mass[j] = cnt[j] ? (double)cnt[j] * (double)exp2f(__fmaf_rn(bf16_key_value(tr.kmax - d), tr.scale, -tr.C)) : 0.0;
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
    if (lane == 31) { s_c[warp] = ic; s_m[warp] = im; }
    __syncthreads();
    unsigned long long bc = 0ull;
    double bm = 0.0;
    for (int x = 0; x < warp; ++x) { bc += s_c[x]; bm += s_m[x]; }
    const unsigned long long c_excl = bc + (ic - lc);
    const double m_excl = bm + (im - lm);
    // top-k: the first key at which the running count reaches k
    if (tr.k > 0) {
        unsigned long long c = c_excl;
        int mine = 0x7fffffff;
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            c += cnt[j];
            if (mine == 0x7fffffff && cnt[j] && c >= (unsigned long long)tr.k) mine = tid * kPer + j;
        }
        mine = __reduce_min_sync(0xffffffffu, mine);
        if (lane == 0 && mine != 0x7fffffff) atomicMin(&s_hit_k, mine);
    }
    __syncthreads();
    const int dk = s_hit_k;
    if (tr.k > 0 && dk == 0x7fffffff) {                     // the k-th largest key lies beyond the window
        if (tid == 0) P.trunc_flag[row] = 1;
        return;
    }
    if (tr.k > 0 && dk / kPer == tid) {                     // mass of the top-k set
        double q = m_excl;
        for (int j = 0; j <= dk % kPer; ++j) q += mass[j];
        s_zk = q;
    }
    __syncthreads();
    int dist = tr.k > 0 ? dk : 0x7fffffff;
    if (tr.p < 1.f) {
        if (!(tr.p > 0.f)) {
            dist = 0;                                       // only the maximum
        } else {
            const double thr = (double)tr.p * (tr.k > 0 ? s_zk : (double)tr.Z);
            double q = m_excl;
            int mine = 0x7fffffff;
#pragma unroll
            for (int j = 0; j < kPer; ++j) {
                q += mass[j];
                if (mine == 0x7fffffff && cnt[j] && q >= thr) mine = tid * kPer + j;
            }
            mine = __reduce_min_sync(0xffffffffu, mine);
            if (lane == 0 && mine != 0x7fffffff) atomicMin(&s_hit_p, mine);
            __syncthreads();
            const int dp = s_hit_p;
            if (dp == 0x7fffffff && tr.k == 0) {            // the nucleus reaches beyond the window
                if (tid == 0) P.trunc_flag[row] = 1;
                return;
            }
            if (dp < dist) dist = dp;
        }
    }
    if (tid == 0 && dist != 0x7fffffff) T.tau[row] = bf16_key_value(tr.kmax - (uint32_t)dist);
}

// One warp per (target row, statistics block): s = sum over x >= tau of 2^(x * scale - c).
__global__ void __launch_bounds__(256) trunc_sums_kernel(VerifyParams P, TruncArgs T)
{
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x;
    const int b = blockIdx.y * 8 + (threadIdx.x >> 5);
    bool bad_rows;
    if (row >= device_rows(P, &bad_rows) || b >= P.nblk) return;
    const float tau = T.tau[row];
    if (!(tau > kNegInf) || P.trunc_flag[row]) return;       // untouched row, or left to the per-row search
    const TruncRow tr = P.trunc_rows[row];
    float2* st = P.stats_t + (long long)row * P.nblk + b;
    const float2 e = *st;
    float sum = 0.f;
    if (e.x > kNegInf && e.x >= __fmul_rn(tau, tr.scale)) {
        const unsigned char* base = P.target + (long long)row * P.tstride_bytes;
        const int e0 = b * P.epb;
        const int cnt = (P.V - e0) < P.epb ? (P.V - e0) : P.epb;
        const uint64_t sc2 = pack2(tr.scale, tr.scale), nc2 = pack2(-e.x, -e.x);
        uint64_t acc = pack2(0.f, 0.f);
        const bool vec = (((uintptr_t)(base + (long long)e0 * 2)) & 15u) == 0;
        for (int i = lane * 8; i < cnt; i += 256) {
            uint32_t w[4];
            if (vec && i + 8 <= cnt) {
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (long long)(e0 + i) * 2));
                w[0] = v.x; w[1] = v.y; w[2] = v.z; w[3] = v.w;
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int a = i + 2 * q;
                    const uint32_t l = a < cnt ? reinterpret_cast<const unsigned short*>(base)[e0 + a] : 0xFF80u;
                    const uint32_t h = a + 1 < cnt ? reinterpret_cast<const unsigned short*>(base)[e0 + a + 1] : 0xFF80u;
                    w[q] = l | (h << 16);
                }
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float t0, t1;
                unpack2(fma2(pack2(cut_below(bf16lo(w[q]), tau), cut_below(bf16hi(w[q]), tau)), sc2, nc2), t0, t1);
                acc = add2(acc, pack2(ex2_approx(t0), ex2_approx(t1)));
            }
        }
        float a0, a1;
        unpack2(acc, a0, a1);
        sum = warp_sum_f32(a0 + a1);
    }
    if (lane == 0) st->y = sum;
}

// ---------------------------------------------------------------------------------------
// Per-request temperatures: expands T_r into one exponent scale log2(e)/T_r per target row and per
// draft row (the streamed pass walks rows, not requests).  One thread per request.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) row_scale_kernel(VerifyParams P)
{
    pdl_wait();
    const int r = blockIdx.x * 256 + threadIdx.x;
    if (r >= P.R) return;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    if (lo < 0 || hi - lo < 1 || hi > n_rows || lo - r < 0 || (hi - 1 - r) > n_rows - P.R) return;
    const float T = P.req_temp[r];
    const float scale = (T > 0.0f && T < INFINITY) ? (float)(1.4426950408889634 / (double)T) : 1.0f;
    for (int i = lo; i < hi; ++i) P.row_scale_t[i] = scale;
    for (int i = lo - r; i < hi - 1 - r; ++i) P.row_scale_d[i] = scale;
}

// ---------------------------------------------------------------------------------------
// decide: one CTA per request, one warp per position (eight per round): row statistics from
// block statistics, p(x), q(x), accept test, first rejection n_r; the accepted prefix is written.
// Position j = len is the bonus row (statistics only).  Every request leaves a record for the
// finalize kernel; a rejected one is also queued for the residual pass.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kDecideThreads) decide_kernel(VerifyParams P)
{
    constexpr int kWarps = kDecideThreads / 32;
    __shared__ int s_first, s_bad, s_have_fin;
    __shared__ int s_first_bad;      // first position with an unusable target or draft row among those looked at
    __shared__ float s_Ct[kWarps], s_Cd[kWarps];
    __shared__ double s_St[kWarps], s_Sd[kWarps];
    __shared__ float s_fin_C[2];     // [0] target, [1] draft statistics of the row that emits the token
    __shared__ double s_fin_S[2];

    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) *unit_tag(P) = 0ull;      // the streamed pass of this call is over
    const int r = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    // the request's rows must lie inside the batch, and so must its draft rows (compact index lo - r)
    if (lo < 0 || hi - lo < 1 || hi > n_rows || lo - r < 0 || (hi - 1 - r) > n_rows - P.R) {
        if (tid == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
        return;
    }
    const int len = hi - lo - 1;
    const long long drow0 = P.draft_row_start ? P.draft_row_start[r] : (long long)(lo - r);
    if (tid == 0) { s_first = len; s_bad = 0; s_have_fin = 0; s_first_bad = 0x7fffffff; }
    __syncthreads();
    for (int i = tid; i <= len; i += kDecideThreads) {
        P.out_tokens[lo + i] = -1;
        if (i < len) {
            const int d = P.draft_tokens[lo + i];
            if (d < 0 || d >= P.V) atomicOr(&s_bad, DSPARK_DEV_BAD_TOKEN);
        }
    }
    __syncthreads();
    const bool want_all = (P.out_p != nullptr) || (P.out_q != nullptr);
    float scale_f = P.scale;
    int bad_request = s_bad;                     // a request reports everything that is wrong with it
    if (P.req_temp) {
        const float T = P.req_temp[r];
        if (!(T > 0.0f) || !(T < INFINITY)) bad_request |= DSPARK_DEV_BAD_TEMPERATURE;
        else scale_f = (float)(1.4426950408889634 / (double)T);
    }
    if (bad_request) {
        if (tid == 0) { atomicOr(P.dev_status, bad_request); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
        return;
    }
    const double scale_d = (double)scale_f;

    for (int j0 = 0; j0 <= len; j0 += kWarps) {
        const int j = j0 + warp;
        if (j <= len) {
            const bool is_draft_pos = j < len;
            // the two logits at the draft token do not depend on the statistics: fetch them first
            float xt = 0.f, xd = 0.f;
            if (is_draft_pos && lane == 0) {
                const int d = P.draft_tokens[lo + j];
                xt = load_logit(P.target, lo + j, P.tstride_bytes, P.elem, d);
                xd = load_logit(P.draft, drow0 + j, P.dstride_bytes, P.elem, d);
            }
            RowAcc A, D;
            combine_rows(P.stats_t + (long long)(lo + j) * P.nblk,
                         is_draft_pos ? P.stats_d + (long long)(lo - r + j) * P.nblk : nullptr, P.nblk, lane, A, D);
            if (!is_draft_pos) {
                // bonus row: leave its block masses (relative to the row reference) where the finalize
                // kernel looks for block values; a rejected request overwrites them in the residual pass
                const float2* st = P.stats_t + (long long)(lo + j) * P.nblk;
                float* wb = P.wblk + (long long)r * P.nblk_r;
                for (int b = lane; b < P.nblk; b += 32) {
                    const float2 e = __ldcg(&st[b]);
                    wb[b] = (e.x > kNegInf && A.C > kNegInf) ? e.y * ex2_approx(e.x - A.C) : 0.f;
                }
            }
            if (lane == 0) {
                s_Ct[warp] = A.C; s_St[warp] = A.S; s_Cd[warp] = D.C; s_Sd[warp] = D.S;
                if (is_draft_pos) {
                    if (!row_usable(A.C, A.S) || !row_usable(D.C, D.S)) {
                        atomicMin(&s_first_bad, j);
                    } else {
                        // truncated target (top-k / top-p): the row sum A.S already covers the kept set only
                        const bool cut = P.tau && xt < P.tau[lo + j];
                        const double p = cut ? 0.0 : exp2((double)xt * scale_d - (double)A.C) / A.S;
                        const double q = exp2((double)xd * scale_d - (double)D.C) / D.S;
                        if (P.out_p) P.out_p[lo + j] = (float)p;
                        if (P.out_q) P.out_q[lo + j] = (float)q;
                        float ua, ur;
                        philox_uniforms(P.seed, (uint32_t)r, (uint32_t)j, ua, ur);
                        if (!((double)ua * q < p)) atomicMin(&s_first, j);     // rejected
                    }
                }
            }
        }
        __syncthreads();
        const int first = s_first;
        const bool in_round = first >= j0 && first < j0 + kWarps;
        if (tid == 0 && in_round && !s_have_fin) {      // the row that emits the token sits in this round
            const int w = first - j0;
            s_fin_C[0] = s_Ct[w]; s_fin_S[0] = s_St[w]; s_fin_C[1] = s_Cd[w]; s_fin_S[1] = s_Sd[w];
            s_have_fin = 1;
        }
        // Which rows void the request: with the probability outputs every draft position is evaluated, and an
        // unusable row anywhere voids it; without them verification ends at the first rejection, and only an
        // unusable row before it counts (the warps of this round that looked further do not change the result)
        const int first_bad = s_first_bad;
        const bool void_req = want_all ? first_bad != 0x7fffffff : first_bad < first;
        const bool stop = void_req || (!want_all && first < len);
        __syncthreads();                         // everyone has read the flags before the next round updates them
        if (stop) break;
    }

    if (tid != 0) return;
    const int n = s_first;
    RequestRec rec;
    rec.kind = kTaskNone; rec.row_t = lo + n; rec.row_d = drow0 + n;
    rec.cp = rec.cq = 0.f; rec.inv_zp = rec.inv_zq = 1.f; rec.u = 0.f; rec.scale = scale_f; rec.pad = 0;
    rec.tau = kNegInf;
    const bool void_req = want_all ? s_first_bad != 0x7fffffff : s_first_bad < n;
    if (void_req || !s_have_fin || !row_usable(s_fin_C[0], s_fin_S[0]) ||
        (n < len && !row_usable(s_fin_C[1], s_fin_S[1]))) {
        atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW);
        P.accepted_len[r] = 0;
    } else {
        for (int i = 0; i < n; ++i) P.out_tokens[lo + i] = P.draft_tokens[lo + i];
        float ua, ur;
        philox_uniforms(P.seed, (uint32_t)r, (uint32_t)n, ua, ur);
        P.accepted_len[r] = n;
        rec.u = ur;
        if (P.tau) rec.tau = P.tau[rec.row_t];
        rec.cp = s_fin_C[0]; rec.inv_zp = (float)(1.0 / s_fin_S[0]);
        if (n < len) {
            rec.cq = s_fin_C[1]; rec.inv_zq = (float)(1.0 / s_fin_S[1]);
            rec.kind = kTaskResid;
            const int slot = atomicAdd(&P.counters[0], 1);
            ResidTask q;
            q.request = r; q.row_t = rec.row_t; q.row_d = rec.row_d;
            q.cp = rec.cp; q.inv_zp = rec.inv_zp; q.cq = rec.cq; q.inv_zq = rec.inv_zq;
            q.u = ur; q.scale = scale_f; q.wslot = r; q.tau = rec.tau;
            P.resid[slot] = q;
        } else {
            rec.kind = kTaskBonus;
        }
    }
    P.req[r] = rec;
}

// ---------------------------------------------------------------------------------------
// finalize: one warp per request draws the token that follows the accepted prefix: from
// norm(max(0, p - q)) of the rejected position (block sums from the residual pass), or the bonus
// token from p of the last row (block statistics saved by the streamed pass).
// ---------------------------------------------------------------------------------------
constexpr int kFinalizeWarps = 2;
template <int kElem>
__global__ void __launch_bounds__(kFinalizeWarps * 32) finalize_kernel(VerifyParams P)
{
    __shared__ Level2Scratch<kElem> s_scr[kFinalizeWarps];
    pdl_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int r = blockIdx.x * kFinalizeWarps + warp;
    if (r >= P.R) return;
    // issue everything that does not depend on the record together with it: the block values of
    // this request (residual sums of a rejected position, or masses of the bonus row)
    const RequestRec rec = P.req[r];
    const float* wb = P.wblk + (long long)r * P.nblk_r;
    // the first 256 block values go to registers whatever the row length: a bonus draw uses the first nblk of
    // them (nblk <= 256 can go with nblk_r > 256), a residual draw all nblk_r when they fit
    float xr[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { const int i = k * 32 + lane; xr[k] = i < P.nblk_r ? __ldcg(&wb[i]) : 0.f; }
    if (rec.kind == kTaskNone) return;
    Level2Scratch<kElem>& S = s_scr[warp];
    const double u = (double)rec.u;
    const unsigned char* trow = P.target + (long long)rec.row_t * P.tstride_bytes;
    int token = -1;
    for (int attempt = 0; attempt < 2 && token < 0; ++attempt) {
        const bool resid = (rec.kind == kTaskResid) && attempt == 0;
        const int n1 = resid ? P.nblk_r : P.nblk;
        if (attempt == 1) {
            // empty residual (p and q agree to rounding): draw from p with the same u; the block masses
            // of that row are rebuilt from the saved statistics
            const float2* st = P.stats_t + (long long)rec.row_t * P.nblk;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = k * 32 + lane;
                float m = 0.f;
                if (i < P.nblk && P.nblk <= 256) { const float2 e = __ldcg(&st[i]); m = e.x > kNegInf ? e.y * ex2_approx(e.x - rec.cp) : 0.f; }
                xr[k] = m;
            }
        }
        double before, tot;
        int b;
        if (n1 <= 256) {
#pragma unroll
            for (int k = 0; k < 8; ++k) if (k * 32 + lane >= n1) xr[k] = 0.f;   // a bonus row has fewer blocks
            b = level1_registers(xr, n1, lane, u, before, tot);
        } else if (attempt == 0) {
            auto wv = [&](int i) { return __ldcg(&wb[i]); };
            tot = warp_total(n1, lane, wv);
            b = level1_memory(n1, lane, wv, u * tot, before);
        } else {
            const float2* st = P.stats_t + (long long)rec.row_t * P.nblk;
            auto mass = [&](int i) { const float2 e = __ldcg(&st[i]); return e.x > kNegInf ? e.y * ex2_approx(e.x - rec.cp) : 0.f; };
            tot = warp_total(n1, lane, mass);
            b = level1_memory(n1, lane, mass, u * tot, before);
        }
        if (!(tot > 0.0) || !(tot < INFINITY)) {
            if (!resid) token = 0;                           // cannot happen for a usable row
            continue;
        }
        const double thr_local = u * tot - before;
        if (resid) {
            ResidConst K;
            K.set(rec.scale, rec.cp, rec.inv_zp, rec.cq, rec.inv_zq, rec.tau);
            const int e0 = b * P.epb_r;
            const int cnt = (P.V - e0) < P.epb_r ? (P.V - e0) : P.epb_r;
            const unsigned char* drow = P.draft + rec.row_d * P.dstride_bytes;
            token = e0 + level2_block<kElem, kResidBlockBytes, true>(
                trow, drow, e0, cnt, lane, thr_local, [&](float xt, float xd) { return resid_elem(xt, xd, K); }, S);
        } else {
            // element masses relative to the row reference, like the block masses
            const float nc = -rec.cp, scale = rec.scale, tau = rec.tau;
            const int e0 = b * P.epb;
            const int cnt = (P.V - e0) < P.epb ? (P.V - e0) : P.epb;
            token = e0 + level2_block<kElem, kStatBlockBytes, false>(
                trow, nullptr, e0, cnt, lane, thr_local,
                [&](float xt, float) { return ex2_approx(__fmaf_rn(cut_below(xt, tau), scale, nc)); }, S);
        }
    }
    if (lane == 0) P.out_tokens[rec.row_t] = token;
}

// ---------------------------------------------------------------------------------------
// Analytical acceptance rate c* = 1 - 1/2 ||p_d - p_t||_1 = 1 - sum_v max(0, p_v - q_v)
// (Section 3.2.1, the confidence head's training label) for every draft position.  Reuses the
// streamed statistics and the residual pass: every draft position is queued as a residual task
// (slot = its compact draft index), then one warp per position sums the block values.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kDecideThreads) queue_all_positions_kernel(VerifyParams P, float* out_cstar)
{
    constexpr int kWarps = kDecideThreads / 32;
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) *unit_tag(P) = 0ull;      // the streamed pass of this call is over
    const int r = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (r == 0 && tid == 0) P.counters[0] = n_rows > P.R ? n_rows - P.R : 0;     // every draft position is a task
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    const bool ok = !(lo < 0 || hi - lo < 1 || hi > n_rows || lo - r < 0 || (hi - 1 - r) > n_rows - P.R);
    if (!ok) {
        if (tid == 0) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
        return;
    }
    const int len = hi - lo - 1;
    const long long drow0 = P.draft_row_start ? P.draft_row_start[r] : (long long)(lo - r);
    if (tid == 0) out_cstar[hi - 1] = NAN;                                       // bonus row: no draft distribution
    for (int j = warp; j < len; j += kWarps) {
        RowAcc A, D;
        combine_rows(P.stats_t + (long long)(lo + j) * P.nblk, P.stats_d + (long long)(lo - r + j) * P.nblk,
                     P.nblk, lane, A, D);
        if (lane == 0) {
            const bool usable = row_usable(A.C, A.S) && row_usable(D.C, D.S);
            if (!usable) atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW);
            ResidTask q;
            q.request = r; q.row_t = lo + j; q.row_d = drow0 + j;
            q.cp = A.C; q.cq = D.C;
            q.inv_zp = usable ? (float)(1.0 / A.S) : NAN;                       // NaN propagates to c*
            q.inv_zq = usable ? (float)(1.0 / D.S) : NAN;
            q.u = 0.f; q.scale = P.scale; q.wslot = lo - r + j; q.tau = kNegInf;
            P.resid[lo - r + j] = q;
        }
    }
}

__global__ void __launch_bounds__(kDecideThreads) cstar_reduce_kernel(VerifyParams P, float* out_cstar)
{
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int slot = blockIdx.x * (kDecideThreads / 32) + (threadIdx.x >> 5);
    int nq = __ldcg(&P.counters[0]);
    nq = nq > P.n_rows_cap ? P.n_rows_cap : nq;
    if (slot >= nq) return;
    const float* wb = P.wblk + (long long)slot * P.nblk_r;
    double w = 0.0;
#pragma unroll 4
    for (int b = lane; b < P.nblk_r; b += 32) w += (double)__ldcg(&wb[b]);
    w = warp_sum_f64(w);
    if (lane == 0) {
        const ResidTask t = P.resid[slot];
        const bool usable = t.inv_zp == t.inv_zp && t.inv_zq == t.inv_zq;      // NaN marks an unusable row
        out_cstar[t.row_t] = usable ? (float)(1.0 - w) : NAN;
    }
}

// ---------------------------------------------------------------------------------------
// greedy decide: one CTA per request, one warp per row (eight rows per round): the row argmax
// from its block statistics, then the first draft token that differs from it.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kDecideThreads) greedy_decide_kernel(VerifyParams P)
{
    constexpr int kWarps = kDecideThreads / 32;
    __shared__ int s_bad, s_first, s_am[kWarps], s_neg[kWarps], s_emit, s_status;
    pdl_wait();
    if (blockIdx.x == 0 && threadIdx.x == 0) *unit_tag(P) = 0ull;      // the streamed pass of this call is over
    const int r = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    if (lo < 0 || hi - lo < 1 || hi > n_rows) {
        if (tid == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS); P.accepted_len[r] = 0; }
        return;
    }
    const int len = hi - lo - 1;
    if (tid == 0) { s_bad = 0; s_first = 0x7fffffff; s_emit = -1; s_status = 0; }
    __syncthreads();
    for (int i = tid; i <= len; i += kDecideThreads) {
        P.out_tokens[lo + i] = -1;
        if (i < len) { const int d = P.draft_tokens[lo + i]; if (d < 0 || d >= P.V) s_bad = 1; }
    }
    __syncthreads();
    if (s_bad) {
        if (tid == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_TOKEN); P.accepted_len[r] = 0; }
        return;
    }
    for (int j0 = 0; j0 <= len; j0 += kWarps) {
        const int j = j0 + warp;
        if (j <= len) {
            const float2* st = P.stats_t + (long long)(lo + j) * P.nblk;
            float best = kNegInf;
            int bi = 0x7fffffff;
            for (int b = lane; b < P.nblk; b += 32) {      // lane-strided: ascending indices per lane
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
            if (lane == 0) {
                const int neg = (best == kNegInf);
                const int am = neg ? 0 : bi;
                s_am[warp] = am; s_neg[warp] = neg;
                // the bonus row always ends the scan; a draft row ends it on a mismatch
                if (j == len || P.draft_tokens[lo + j] != am) atomicMin(&s_first, j);
            }
        }
        __syncthreads();
        const int first = s_first;
        if (tid == 0) {
            // rows of this round up to the one that emits may raise the all -inf flag
            const int last_j = first < j0 + kWarps ? first : j0 + kWarps - 1;
            for (int w = 0; j0 + w <= last_j && w < kWarps; ++w) if (s_neg[w]) s_status |= DSPARK_DEV_ALL_NEG_INF;
            if (first < j0 + kWarps) s_emit = s_am[first - j0];
        }
        __syncthreads();
        if (first < j0 + kWarps) break;
    }
    const int n = s_first;
    for (int i = tid; i < n; i += kDecideThreads) P.out_tokens[lo + i] = P.draft_tokens[lo + i];
    if (tid == 0) {
        P.out_tokens[lo + n] = s_emit;
        P.accepted_len[r] = n;
        if (s_status) atomicOr(P.dev_status, s_status);
    }
}

// ---------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------
static int g_force_direct = 0;

struct DeviceInfo { int sms; bool attrs_set; };
static DeviceInfo& device_info()
{
    static DeviceInfo info[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    DeviceInfo& d = info[dev & 63];
    if (d.sms == 0) cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    return d;
}

template <int kElem, int kMode>
static cudaError_t set_smem_attr()
{
    return cudaFuncSetAttribute(stream_bulk_kernel<kElem, kMode>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kStages * kStageBytes);
}

static bool ensure_attrs()
{
    DeviceInfo& d = device_info();
    if (d.attrs_set) return true;
    bool ok = set_smem_attr<2, kModeStats>() == cudaSuccess && set_smem_attr<4, kModeStats>() == cudaSuccess &&
              set_smem_attr<2, kModeGreedy>() == cudaSuccess && set_smem_attr<4, kModeGreedy>() == cudaSuccess &&
              set_smem_attr<2, kModeResid>() == cudaSuccess && set_smem_attr<4, kModeResid>() == cudaSuccess &&
              set_smem_attr<2, kModeHist>() == cudaSuccess;
    d.attrs_set = ok;
    return ok;
}

template <int kElem, int kMode>
static void launch_stream(const VerifyParams& P, bool bulk, long long max_units, cudaStream_t s)
{
    const int sms = device_info().sms;
    if (bulk) {
        long long g = (long long)sms * 3;
        if (g > max_units) g = max_units;
        if (g < 1) g = 1;
        launch_pdl(stream_bulk_kernel<kElem, kMode>, dim3((unsigned)g), dim3(kStreamThreads), kStages * kStageBytes, s, P);
    } else {
        long long g = (long long)sms * 8;
        if (g > max_units) g = max_units;
        if (g < 1) g = 1;
        launch_pdl(stream_direct_kernel<kElem, kMode>, dim3((unsigned)g), dim3(kConsumerWarps * 32), 0, s, P);
    }
}

template <int kMode>
static void launch_stream_dtype(const VerifyParams& P, bool bulk, long long max_units, cudaStream_t s)
{
    if (P.elem == 2) launch_stream<2, kMode>(P, bulk, max_units, s);
    else launch_stream<4, kMode>(P, bulk, max_units, s);
}

struct Workspace {
    size_t counters, stats_t, stats_d, resid, req, wblk, scale_t, scale_d, tau, trunc_rows, trunc_bins, trunc_flag, total;
};
static Workspace workspace_layout(int R, int n_rows, int V)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t nblk = (size_t)blocks_per_row(V, 4, kStatBlockBytes);
    const size_t nblk_r = (size_t)blocks_per_row(V, 4, kResidBlockBytes);
    Workspace w;
    size_t o = 0;
    w.counters = o; o += up(64 * sizeof(int));
    w.stats_t = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.stats_d = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.resid = o;    o += up((size_t)R * sizeof(ResidTask));
    w.req = o;      o += up((size_t)R * sizeof(RequestRec));
    w.wblk = o;     o += up((size_t)R * nblk_r * sizeof(float));
    w.scale_t = o;  o += up((size_t)n_rows * sizeof(float));
    w.scale_d = o;  o += up((size_t)n_rows * sizeof(float));
    w.tau = o;      o += up((size_t)n_rows * sizeof(float));
    w.trunc_rows = o; o += up((size_t)n_rows * sizeof(TruncRow));
    w.trunc_bins = o; o += up((size_t)n_rows * kHistBins * sizeof(unsigned int));
    w.trunc_flag = o; o += up((size_t)(n_rows + 1) * sizeof(int32_t));   // + the fallback's row counter
    w.total = o;
    return w;
}

static bool aligned16(const void* p, long long stride_bytes, long long row_bytes)
{
    return (((uintptr_t)p) & 15u) == 0 && (stride_bytes & 15) == 0 && (row_bytes & 15) == 0;
}

static int fill_params(VerifyParams& P, const void* target, const void* draft, int dtype,
                       int64_t tstride, int64_t dstride, int V, const int32_t* row_offsets,
                       const int64_t* draft_row_start, const int32_t* draft_tokens, int R, int n_rows,
                       int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                       void* workspace, size_t workspace_bytes)
{
    if (!target || !row_offsets || !draft_tokens || !accepted_len || !out_tokens) return DSPARK_ERR_INVALID_ARG;
    if (dtype != DSPARK_F32 && dtype != DSPARK_BF16) return DSPARK_ERR_INVALID_ARG;
    if (R < 1 || V < 1 || n_rows < R) return DSPARK_ERR_INVALID_ARG;
    const int elem = dtype == DSPARK_BF16 ? 2 : 4;
    if ((long long)V * elem >= (1ll << 31) || tstride < V) return DSPARK_ERR_SHAPE;
    const Workspace w = workspace_layout(R, n_rows, V);
    if (!workspace || workspace_bytes < w.total) return DSPARK_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return DSPARK_ERR_ALIGNMENT;
    unsigned char* ws = (unsigned char*)workspace;
    P.target = (const unsigned char*)target;
    P.draft = (const unsigned char*)draft;
    P.tstride_bytes = (long long)tstride * elem;
    P.dstride_bytes = (long long)dstride * elem;
    P.V = V; P.elem = elem; P.row_bytes = V * elem;
    P.nblk = blocks_per_row(V, elem, kStatBlockBytes);
    P.epb = kStatBlockBytes / elem;
    P.nblk_r = blocks_per_row(V, elem, kResidBlockBytes);
    P.epb_r = kResidBlockBytes / elem;
    P.row_offsets = row_offsets; P.draft_row_start = draft_row_start; P.draft_tokens = draft_tokens;
    P.R = R; P.n_rows_cap = n_rows;
    P.scale = 1.0f; P.seed = 0;
    P.accepted_len = accepted_len; P.out_tokens = out_tokens; P.out_p = nullptr; P.out_q = nullptr;
    P.counters = (int*)(ws + w.counters);
    P.launch_tag = next_launch_tag();
    P.dev_status = dev_status ? dev_status : P.counters + 1;
    P.stats_t = (float2*)(ws + w.stats_t);
    P.stats_d = (float2*)(ws + w.stats_d);
    P.resid = (ResidTask*)(ws + w.resid);
    P.req = (RequestRec*)(ws + w.req);
    P.wblk = (float*)(ws + w.wblk);
    P.resid_cap = R;
    P.req_temp = nullptr;
    P.tau = nullptr;
    P.trunc_rows = (TruncRow*)(ws + w.trunc_rows);
    P.trunc_bins = (unsigned int*)(ws + w.trunc_bins);
    P.trunc_flag = (int32_t*)(ws + w.trunc_flag);
    P.row_scale_t = (float*)(ws + w.scale_t);
    P.row_scale_d = (float*)(ws + w.scale_d);
    return DSPARK_OK;
}

static long long pieces(int nblk) { return (nblk + kConsumerWarps - 1) / kConsumerWarps; }

}  // namespace dspark

using namespace dspark;

extern "C" {

size_t dspark_verify_workspace_bytes(int R, int n_rows, int V)
{
    if (R < 1 || n_rows < R || V < 1) return 0;
    return workspace_layout(R, n_rows, V).total;
}

int dspark_set_stream_path(int path)
{
    if (path != 0 && path != 1) return DSPARK_ERR_INVALID_ARG;
    g_force_direct = path;
    return DSPARK_OK;
}

int dspark_verify_greedy(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                         const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                         int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    VerifyParams P;
    int rc = fill_params(P, target_logits, nullptr, dtype, target_row_stride, 0, V, row_offsets, nullptr,
                         draft_tokens, R, n_rows, accepted_len, out_tokens, dev_status, workspace, workspace_bytes);
    if (rc != DSPARK_OK) return rc;
    if (!ensure_attrs()) return launch_status();
    cudaStream_t s = (cudaStream_t)stream;
    const bool bulk = !g_force_direct && aligned16(P.target, P.tstride_bytes, P.row_bytes);
    {
        KernelTimerScope timer(DSPARK_K_GREEDY_STREAM, s);
        launch_stream_dtype<kModeGreedy>(P, bulk, (long long)n_rows * pieces(P.nblk), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_GREEDY_DECIDE, s);
        launch_pdl(greedy_decide_kernel, dim3(R), dim3(kDecideThreads), 0, s, P);
    }
    return launch_status();
}

static int verify_launch(const void* target_logits, const void* draft_logits, int dtype,
                         int64_t target_row_stride, int64_t draft_row_stride, int V,
                         const int32_t* row_offsets, const int64_t* draft_row_start,
                         const int32_t* draft_tokens, int R, int n_rows,
                         float temperature, const float* req_temp, uint64_t seed,
                         int32_t* accepted_len, int32_t* out_tokens,
                         float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream,
                         const int32_t* top_k = nullptr, const float* top_p = nullptr)
{
    if (!draft_logits) return DSPARK_ERR_INVALID_ARG;
    const bool truncate = top_k || top_p;
    if (truncate && dtype != DSPARK_BF16) return DSPARK_ERR_SHAPE;   // the threshold search works on 16-bit keys
    if (!req_temp && (!(temperature > 0.0f) || !isfinite(temperature))) return DSPARK_ERR_INVALID_ARG;
    if (draft_row_stride < V) return DSPARK_ERR_SHAPE;
    VerifyParams P;
    int rc = fill_params(P, target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V,
                         row_offsets, draft_row_start, draft_tokens, R, n_rows, accepted_len, out_tokens,
                         dev_status, workspace, workspace_bytes);
    if (rc != DSPARK_OK) return rc;
    P.scale = req_temp ? 1.0f : (float)(1.4426950408889634 / (double)temperature);
    P.req_temp = req_temp;
    P.seed = seed;
    P.out_p = out_p_tok;
    P.out_q = out_q_tok;
    if (!ensure_attrs()) return launch_status();
    cudaStream_t s = (cudaStream_t)stream;
    const bool bulk = !g_force_direct && aligned16(P.target, P.tstride_bytes, P.row_bytes) &&
                      aligned16(P.draft, P.dstride_bytes, P.row_bytes);
    if (req_temp) {
        KernelTimerScope timer(DSPARK_K_ROW_SCALE, s);
        launch_pdl(row_scale_kernel, dim3((R + 255) / 256), dim3(256), 0, s, P);
    }
    {
        KernelTimerScope timer(DSPARK_K_STREAM, s);
        launch_stream_dtype<kModeStats>(P, bulk, (2ll * n_rows - R) * pieces(P.nblk), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    if (truncate) {
        // top-k / top-p of the target distribution without touching the rows: one kernel finds the threshold of
        // every target row and replaces the row's block sums by the sums over the kept set; from here on a
        // target logit below the threshold counts as -inf
        float* tau = (float*)((unsigned char*)workspace + workspace_layout(R, n_rows, V).tau);
        KernelTimerScope timer(DSPARK_K_TRUNCATE, s);
        TruncArgs T;
        T.top_k = top_k; T.top_p = top_p; T.temperatures = req_temp; T.temperature = temperature; T.tau = tau;
        launch_pdl(trunc_prep_kernel, dim3((n_rows + 7) / 8), dim3(256), 0, s, P, T);
        launch_stream<2, kModeHist>(P, bulk, (long long)n_rows * pieces(P.nblk), s);
        launch_pdl(trunc_scan_kernel, dim3(n_rows), dim3(kScanThreads), 0, s, P, T);
        launch_pdl(trunc_sums_kernel, dim3(n_rows, (P.nblk + 7) / 8), dim3(256), 0, s, P, T);
        // rows whose threshold lies beyond the window (flat rows): the per-row search
        rc = truncate_virtual_launch(P.target, P.tstride_bytes, V, row_offsets, R, n_rows, top_k, top_p, temperature,
                                     req_temp, tau, P.stats_t, P.nblk, P.epb, P.trunc_flag, s);
        if (rc != DSPARK_OK) return rc;
        P.tau = tau;
    }
    {
        KernelTimerScope timer(DSPARK_K_DECIDE, s);
        launch_pdl(decide_kernel, dim3(R), dim3(kDecideThreads), 0, s, P);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_RESIDUAL, s);
        launch_stream_dtype<kModeResid>(P, bulk, (long long)R * pieces(P.nblk_r), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_FINALIZE, s);
        const int grid = (R + kFinalizeWarps - 1) / kFinalizeWarps;
        if (P.elem == 2) launch_pdl(finalize_kernel<2>, dim3(grid), dim3(kFinalizeWarps * 32), 0, s, P);
        else launch_pdl(finalize_kernel<4>, dim3(grid), dim3(kFinalizeWarps * 32), 0, s, P);
    }
    return launch_status();
}


// ---------------------------------------------------------------------------------------
// dspark_verify_greedy_static: greedy verification for callers that must not allocate.
// Its scratch is this fixed array inside the library image instead of a caller workspace.
// ---------------------------------------------------------------------------------------
}  // extern "C"

namespace dspark {

constexpr size_t kStaticScratchBytes = DSPARK_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// The array's name is only a host-side handle; kernels need its device address, which is looked
// up once per device (with that device current) and cached.
static void* g_static_scratch_ptr[64] = {};

static int static_scratch_address(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return DSPARK_ERR_CUDA; }
    if (!g_static_scratch_ptr[dev]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) {
            fprintf(stderr, "dspark: cudaGetSymbolAddress(static scratch) failed: %s\n", cudaGetErrorString(e));
            cudaGetLastError();
            return DSPARK_ERR_CUDA;
        }
        g_static_scratch_ptr[dev] = ptr;
    }
    *out = g_static_scratch_ptr[dev];
    return DSPARK_OK;
}

}  // namespace dspark

extern "C" {

size_t dspark_verify_greedy_static_capacity(void) { return kStaticScratchBytes; }

int dspark_verify_greedy_static(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                                const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                                int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status, void* stream)
{
    if (R < 1 || n_rows < R || V < 1) return DSPARK_ERR_INVALID_ARG;
    const size_t need = workspace_layout(R, n_rows, V).total;
    if (need > kStaticScratchBytes) {
        fprintf(stderr, "dspark_verify_greedy_static: this batch needs %zu bytes of scratch, the built-in array "
                        "holds %zu; use dspark_verify_greedy with a caller workspace\n", need, kStaticScratchBytes);
        return DSPARK_ERR_STATIC_LIMIT;
    }
    void* scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != DSPARK_OK) return rc;
    // every statistic the decide kernel reads is rewritten by the stream kernel of this same call,
    // so nothing left by an earlier call needs clearing
    return dspark_verify_greedy(target_logits, dtype, target_row_stride, V, row_offsets, draft_tokens, R, n_rows,
                                accepted_len, out_tokens, dev_status, scratch, kStaticScratchBytes, stream);
}

int dspark_verify(const void* target_logits, const void* draft_logits, int dtype,
                  int64_t target_row_stride, int64_t draft_row_stride, int V,
                  const int32_t* row_offsets, const int64_t* draft_row_start,
                  const int32_t* draft_tokens, int R, int n_rows,
                  float temperature, uint64_t seed,
                  int32_t* accepted_len, int32_t* out_tokens,
                  float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                  void* workspace, size_t workspace_bytes, void* stream)
{
    return verify_launch(target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V, row_offsets,
                         draft_row_start, draft_tokens, R, n_rows, temperature, nullptr, seed, accepted_len,
                         out_tokens, out_p_tok, out_q_tok, dev_status, workspace, workspace_bytes, stream);
}

int dspark_verify_per_request(const void* target_logits, const void* draft_logits, int dtype,
                              int64_t target_row_stride, int64_t draft_row_stride, int V,
                              const int32_t* row_offsets, const int64_t* draft_row_start,
                              const int32_t* draft_tokens, int R, int n_rows,
                              const float* temperatures, uint64_t seed,
                              int32_t* accepted_len, int32_t* out_tokens,
                              float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                              void* workspace, size_t workspace_bytes, void* stream)
{
    if (!temperatures) return DSPARK_ERR_INVALID_ARG;
    return verify_launch(target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V, row_offsets,
                         draft_row_start, draft_tokens, R, n_rows, 1.0f, temperatures, seed, accepted_len,
                         out_tokens, out_p_tok, out_q_tok, dev_status, workspace, workspace_bytes, stream);
}

int dspark_verify_truncated(const void* target_logits, const void* draft_logits, int dtype,
                            int64_t target_row_stride, int64_t draft_row_stride, int V,
                            const int32_t* row_offsets, const int64_t* draft_row_start,
                            const int32_t* draft_tokens, int R, int n_rows,
                            float temperature, const float* temperatures, const int32_t* top_k, const float* top_p,
                            uint64_t seed, int32_t* accepted_len, int32_t* out_tokens,
                            float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                            void* workspace, size_t workspace_bytes, void* stream)
{
    return verify_launch(target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V, row_offsets,
                         draft_row_start, draft_tokens, R, n_rows, temperatures ? 1.0f : temperature, temperatures, seed,
                         accepted_len, out_tokens, out_p_tok, out_q_tok, dev_status, workspace, workspace_bytes, stream,
                         top_k, top_p);
}

static size_t accept_rate_extra(int n_rows, int V, size_t* resid_off, size_t* wblk_off)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t nblk_r = (size_t)blocks_per_row(V, 4, kResidBlockBytes);
    size_t o = 0;
    *resid_off = o; o += up((size_t)n_rows * sizeof(ResidTask));
    *wblk_off = o;  o += up((size_t)n_rows * nblk_r * sizeof(float));
    return o;
}

size_t dspark_accept_rate_workspace_bytes(int R, int n_rows, int V)
{
    if (R < 1 || n_rows < R || V < 1) return 0;
    size_t a, b;
    return workspace_layout(R, n_rows, V).total + accept_rate_extra(n_rows, V, &a, &b);
}

int dspark_accept_rate(const void* target_logits, const void* draft_logits, int dtype,
                       int64_t target_row_stride, int64_t draft_row_stride, int V,
                       const int32_t* row_offsets, const int64_t* draft_row_start, int R, int n_rows,
                       float temperature, float* out_cstar, int32_t* dev_status,
                       void* workspace, size_t workspace_bytes, void* stream)
{
    if (!draft_logits || !out_cstar) return DSPARK_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return DSPARK_ERR_INVALID_ARG;
    if (draft_row_stride < V) return DSPARK_ERR_SHAPE;
    if (R < 1 || n_rows < R || V < 1) return DSPARK_ERR_INVALID_ARG;
    size_t resid_off, wblk_off;
    const size_t base = workspace_layout(R, n_rows, V).total;
    const size_t extra = accept_rate_extra(n_rows, V, &resid_off, &wblk_off);
    if (!workspace || workspace_bytes < base + extra) return DSPARK_ERR_WORKSPACE;
    VerifyParams P;
    // the token / length outputs of the verifier are not produced here: the row_offsets pointer only
    // stands in for the non-null checks of the shared set-up and is never written through
    int rc = fill_params(P, target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V,
                         row_offsets, draft_row_start, row_offsets, R, n_rows,
                         const_cast<int32_t*>(row_offsets), const_cast<int32_t*>(row_offsets), dev_status,
                         workspace, workspace_bytes);
    if (rc != DSPARK_OK) return rc;
    P.accepted_len = nullptr; P.out_tokens = nullptr; P.draft_tokens = nullptr;
    P.scale = (float)(1.4426950408889634 / (double)temperature);
    P.resid = (ResidTask*)((unsigned char*)workspace + base + resid_off);
    P.wblk = (float*)((unsigned char*)workspace + base + wblk_off);
    P.resid_cap = n_rows;
    if (!ensure_attrs()) return launch_status();
    cudaStream_t s = (cudaStream_t)stream;
    const bool bulk = !g_force_direct && aligned16(P.target, P.tstride_bytes, P.row_bytes) &&
                      aligned16(P.draft, P.dstride_bytes, P.row_bytes);
    {
        KernelTimerScope timer(DSPARK_K_STREAM, s);
        launch_stream_dtype<kModeStats>(P, bulk, (2ll * n_rows - R) * pieces(P.nblk), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_DECIDE, s);
        launch_pdl(queue_all_positions_kernel, dim3(R), dim3(kDecideThreads), 0, s, P, out_cstar);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_RESIDUAL, s);
        launch_stream_dtype<kModeResid>(P, bulk, (long long)(n_rows - R > 0 ? n_rows - R : 1) * pieces(P.nblk_r), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_FINALIZE, s);
        const int warps = kDecideThreads / 32;
        const int grid = (n_rows - R + warps - 1) / warps;
        launch_pdl(cstar_reduce_kernel, dim3(grid > 0 ? grid : 1), dim3(kDecideThreads), 0, s, P, out_cstar);
    }
    return launch_status();
}

}  // extern "C"
