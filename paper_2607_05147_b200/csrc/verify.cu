// dspark_verify / dspark_verify_greedy: the fused ragged-batch speculative verifier
// (acceptance rule of Section 2.1; bonus token of Section 1; flat ragged rows of Section 4.3).
//
// Pass structure (all on the caller's stream, no host round trip):
//   stream   every target / draft row is read from HBM exactly once.  A row is cut into
//            2 KB blocks; one warp reduces one block to (reference, sum of 2^(x*scale-ref))
//            [sampling] or (max, lowest argmax) [greedy].  Persistent CTAs; a producer warp
//            feeds a ring of 16 KB shared-memory stages with 1-D bulk async copies
//            (cp.async.bulk + mbarrier), eight consumer warps drain it.
//   decide   one CTA per request: combines block statistics into row statistics, gathers
//            p(x), q(x), runs the accept tests (Philox), finds the first rejection, writes
//            the accepted prefix, and queues the rejected position for the residual pass.
//   residual second read of the rejected position's row pair only: per-block sums of
//            max(0, p - q), same bulk-copy pipeline with two sources per stage.
//   finalize one warp per request: inverse CDF over block sums, then inside one block.
#include <cuda_bf16.h>
#include <math.h>

#include "common.cuh"

namespace dspark {

constexpr int kModeStats = 0, kModeGreedy = 1, kModeResid = 2;
constexpr int kTaskNone = 0, kTaskResid = 1, kTaskBonus = 2;
constexpr int kDecideThreads = 256;
constexpr int kFinalizeThreads = 256;
constexpr float kNegInf = -INFINITY;

struct __align__(16) ResidTask {     // one rejected request queued for the residual pass
    int32_t request;
    int32_t row_t;                   // target row of the rejected position
    int64_t row_d;                   // physical draft row
    float cp, inv_zp, cq, inv_zq;    // row references (log2 domain) and 1 / row sums
};

struct __align__(16) RequestTask {   // what finalize needs per request
    int32_t kind;                    // kTaskNone / kTaskResid / kTaskBonus
    int32_t n;                       // accepted length
    int32_t slot;                    // index into the residual list (kTaskResid)
    float u;                         // resample uniform
    int64_t row_d;
    float cp, inv_zp, cq, inv_zq;
};

struct VerifyParams {
    const unsigned char* target;
    const unsigned char* draft;
    long long tstride_bytes, dstride_bytes;
    int V, elem, row_bytes, nblk, ppr, epb;   // epb = elements per block
    const int32_t* row_offsets;
    const int64_t* draft_row_start;
    const int32_t* draft_tokens;
    int R, n_rows_cap;
    float scale;                              // log2(e) / T
    unsigned long long seed;
    int32_t* accepted_len;
    int32_t* out_tokens;
    float* out_p;
    float* out_q;
    int32_t* dev_status;
    // workspace
    int* counters;                            // [0] number of queued residual tasks
    float2* stats_t;
    float2* stats_d;
    ResidTask* resid;
    RequestTask* req;
    float* wblk;
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

struct Unit {
    const unsigned char* src0;
    const unsigned char* src1;
    int piece;          // piece index inside the row
    int bytes;          // bytes of this piece (per source)
    long long out_row;  // row index into the statistics array (or residual slot)
    int is_draft;
    ResidTask task;
};

template <int kMode>
__device__ __forceinline__ int total_units(const VerifyParams& P, int n_rows)
{
    if (kMode == kModeStats) return (n_rows + (n_rows > P.R ? n_rows - P.R : 0)) * P.ppr;
    if (kMode == kModeGreedy) return n_rows * P.ppr;
    int nq = __ldcg(&P.counters[0]);
    return (nq > P.R ? P.R : nq) * P.ppr;
}

template <int kMode>
__device__ __forceinline__ void decode_unit(const VerifyParams& P, int u, int n_rows, bool need_src, Unit& U)
{
    const int s = u / P.ppr;
    U.piece = u - s * P.ppr;
    const long long off = (long long)U.piece * kPieceBytes;
    const long long rem = (long long)P.row_bytes - off;
    U.bytes = (int)(rem < kPieceBytes ? rem : kPieceBytes);
    U.src1 = nullptr;
    U.is_draft = 0;
    if (kMode == kModeResid) {
        U.task = P.resid[s];
        U.out_row = s;
        U.src0 = P.target + (long long)U.task.row_t * P.tstride_bytes + off;
        U.src1 = P.draft + U.task.row_d * P.dstride_bytes + off;
        return;
    }
    if (s < n_rows) {
        U.out_row = s;
        U.src0 = P.target + (long long)s * P.tstride_bytes + off;
    } else {
        const int ds = s - n_rows;
        U.out_row = ds;
        U.is_draft = 1;
        long long phys = need_src ? draft_phys_row(P, ds) : 0;
        U.src0 = (phys >= 0 ? P.draft + phys * P.dstride_bytes : P.target) + off;
    }
}

// ---------------------------------------------------------------------------------------
// Per-lane view of one 2 KB block: 4 x 16 B, vector k of lane l is vector k*32+l of the block
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

template <int kElem, typename Fetch>
__device__ __forceinline__ void load_block(const Fetch& f, int nbytes, int lane, uint4 (&v)[kVecPerLane])
{
#pragma unroll
    for (int k = 0; k < kVecPerLane; ++k) {
        const int vec = k * 32 + lane;
        const uint32_t fw = fill_word<kElem>();
        v[k] = (vec * 16 < nbytes) ? f(vec, nbytes) : make_uint4(fw, fw, fw, fw);
    }
}

__device__ __forceinline__ uint32_t word_of(const uint4& q, int i)
{
    return i == 0 ? q.x : (i == 1 ? q.y : (i == 2 ? q.z : q.w));
}

// Sampling statistics of one block: reference c = max(x) * scale (warp-uniform) and
// s = sum over the block of 2^(x*scale - c): exactly one exponential per element.
template <int kElem>
__device__ __forceinline__ float2 block_stats(const uint4 (&v)[kVecPerLane], float scale)
{
    float mx;
    if (kElem == 2) {
        __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&v[0].x);
#pragma unroll
        for (int k = 0; k < kVecPerLane; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint32_t w = word_of(v[k], i);
                m2 = __hmax2(m2, *reinterpret_cast<const __nv_bfloat162*>(&w));
            }
        uint32_t mw = *reinterpret_cast<uint32_t*>(&m2);
        mx = fmaxf(bf16lo(mw), bf16hi(mw));
    } else {
        mx = kNegInf;
#pragma unroll
        for (int k = 0; k < kVecPerLane; ++k)
#pragma unroll
            for (int i = 0; i < 4; ++i) mx = fmaxf(mx, __uint_as_float(word_of(v[k], i)));
    }
    const float wmax = warp_max_f32(mx);
    if (wmax == kNegInf) return make_float2(kNegInf, 0.0f);
    const float c = __fmul_rn(wmax, scale);
    const float nc = -c;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < kVecPerLane; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t w = word_of(v[k], i);
            if (kElem == 2) {
                acc[i] += ex2_approx(__fmaf_rn(bf16lo(w), scale, nc));
                acc[i] += ex2_approx(__fmaf_rn(bf16hi(w), scale, nc));
            } else {
                acc[i] += ex2_approx(__fmaf_rn(__uint_as_float(w), scale, nc));
            }
        }
    const float s = warp_sum_f32((acc[0] + acc[1]) + (acc[2] + acc[3]));
    return make_float2(c, s);
}

// Greedy statistics of one block: (max, lowest index attaining it); NaN never wins.
template <int kElem>
__device__ __forceinline__ float2 block_argmax(const uint4 (&v)[kVecPerLane], int elem_base, int lane)
{
    constexpr int kPerVec = 16 / kElem;
    float best = kNegInf;
    int bi = 0x7fffffff;
#pragma unroll
    for (int k = 0; k < kVecPerLane; ++k) {
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

// One element of the residual max(0, p - q), with the exact operation sequence the
// finalize kernel repeats.
__device__ __forceinline__ float resid_elem(float xt, float xd, float scale, const ResidTask& t)
{
    const float ep = ex2_approx(__fmaf_rn(xt, scale, -t.cp));
    const float eq = ex2_approx(__fmaf_rn(xd, scale, -t.cq));
    const float q = __fmul_rn(eq, t.inv_zq);
    return fmaxf(__fmaf_rn(ep, t.inv_zp, -q), 0.0f);
}

template <int kElem>
__device__ __forceinline__ float block_resid(const uint4 (&vt)[kVecPerLane], const uint4 (&vd)[kVecPerLane],
                                             float scale, const ResidTask& t)
{
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int k = 0; k < kVecPerLane; ++k)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t a = word_of(vt[k], i), b = word_of(vd[k], i);
            if (kElem == 2) {
                acc[i] += resid_elem(bf16lo(a), bf16lo(b), scale, t);
                acc[i] += resid_elem(bf16hi(a), bf16hi(b), scale, t);
            } else {
                acc[i] += resid_elem(__uint_as_float(a), __uint_as_float(b), scale, t);
            }
        }
    return warp_sum_f32((acc[0] + acc[1]) + (acc[2] + acc[3]));
}

// What a consumer warp does with its block of a unit.
template <int kElem, int kMode, typename Fetch>
__device__ __forceinline__ void consume_block(const VerifyParams& P, const Unit& U, int warp, int lane,
                                              const Fetch& f0, const Fetch& f1)
{
    const int b = U.piece * kConsumerWarps + warp;
    if (b >= P.nblk) return;
    const int blk_off = warp * kBlockBytes;
    const int nbytes = (U.bytes - blk_off) < kBlockBytes ? (U.bytes - blk_off) : kBlockBytes;
    uint4 v[kVecPerLane];
    load_block<kElem>(f0, nbytes, lane, v);
    if (kMode == kModeStats) {
        const float2 st = block_stats<kElem>(v, P.scale);
        if (lane == 0) (U.is_draft ? P.stats_d : P.stats_t)[U.out_row * P.nblk + b] = st;
    } else if (kMode == kModeGreedy) {
        const float2 st = block_argmax<kElem>(v, b * P.epb, lane);
        if (lane == 0) P.stats_t[U.out_row * P.nblk + b] = st;
    } else {
        uint4 vd[kVecPerLane];
        load_block<kElem>(f1, nbytes, lane, vd);
        const float w = block_resid<kElem>(v, vd, P.scale, U.task);
        if (lane == 0) P.wblk[U.out_row * P.nblk + b] = w;
    }
}

// ---------------------------------------------------------------------------------------
// Streamed pass, bulk-copy pipeline.  kStages x kSrc x 16 KB of shared memory per CTA.
// ---------------------------------------------------------------------------------------
template <int kElem, int kMode>
struct StreamCfg {
    static constexpr int kSrc = (kMode == kModeResid) ? 2 : 1;
    static constexpr int kStages = 6 / kSrc;
    static constexpr int kStageBytes = kSrc * kPieceBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes;
};

template <int kElem, int kMode>
__global__ void __launch_bounds__(kStreamThreads, 2) stream_bulk_kernel(VerifyParams P)
{
    using Cfg = StreamCfg<kElem, kMode>;
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[Cfg::kStages];
    __shared__ __align__(8) uint64_t empty_bar[Cfg::kStages];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < Cfg::kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kConsumerWarps); }
        s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();

    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (kMode != kModeResid && blockIdx.x == 0 && tid == 0) {
        P.counters[0] = 0;                       // residual queue, filled by the decide kernel
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int total = total_units<kMode>(P, n_rows);
    volatile int* abort_flag = &s_abort;

    if (warp == kConsumerWarps) {
        // ---------------- producer warp: lane 0 issues the copies -----------------------
        int it = 0;
        for (int u = blockIdx.x; u < total; u += gridDim.x, ++it) {
            const int s = it % Cfg::kStages;
            const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
            if (*abort_flag) break;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&empty_bar[s], ph ^ 1u))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                break;
            }
            Unit U;
            decode_unit<kMode>(P, u, n_rows, true, U);
            if (lane == 0) {
                unsigned char* dst = stage_mem + s * Cfg::kStageBytes;
                mbar_arrive_expect_tx(&full_bar[s], (uint32_t)(U.bytes * Cfg::kSrc));
                bulk_g2s(dst, U.src0, (uint32_t)U.bytes, &full_bar[s]);
                if (Cfg::kSrc == 2) bulk_g2s(dst + kPieceBytes, U.src1, (uint32_t)U.bytes, &full_bar[s]);
            }
            __syncwarp();
        }
        if (*abort_flag) {
            // leave only after every copy already issued has landed (bounded)
            for (int k = 0; k < Cfg::kStages && k < it; ++k) {
                const int jt = it - 1 - k;
                mbar_wait_bounded(&full_bar[jt % Cfg::kStages], (uint32_t)(jt / Cfg::kStages) & 1u);
            }
        }
    } else {
        // ---------------- consumer warps --------------------------------------------------
        int it = 0;
        for (int u = blockIdx.x; u < total; u += gridDim.x, ++it) {
            const int s = it % Cfg::kStages;
            const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
            if (*abort_flag) break;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&full_bar[s], ph))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                break;
            }
            Unit U;
            decode_unit<kMode>(P, u, n_rows, false, U);
            const unsigned char* st = stage_mem + s * Cfg::kStageBytes + warp * kBlockBytes;
            SmemFetch f0{st}, f1{st + kPieceBytes};
            consume_block<kElem, kMode>(P, U, warp, lane, f0, f1);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[s]);
        }
    }
}

// Streamed pass without the bulk copy: each warp loads its block straight from global
// memory (16-byte loads where the address allows, element loads otherwise).  Taken when
// a pointer, stride or row length breaks the 16-byte rules of the bulk copy.
template <int kElem, int kMode>
__global__ void __launch_bounds__(kConsumerWarps * 32, 2) stream_direct_kernel(VerifyParams P)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (kMode != kModeResid && blockIdx.x == 0 && tid == 0) {
        P.counters[0] = 0;
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int total = total_units<kMode>(P, n_rows);
    for (int u = blockIdx.x; u < total; u += gridDim.x) {
        Unit U;
        decode_unit<kMode>(P, u, n_rows, true, U);
        GlobalFetch<kElem> f0{U.src0 + warp * kBlockBytes};
        GlobalFetch<kElem> f1{(kMode == kModeResid ? U.src1 : U.src0) + warp * kBlockBytes};
        consume_block<kElem, kMode>(P, U, warp, lane, f0, f1);
    }
}

// ---------------------------------------------------------------------------------------
// Row statistics from block statistics: reference C = max_b c_b, sum S = sum_b s_b 2^(c_b-C).
// Called by one full warp; result valid in every lane.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void combine_row(const float2* __restrict__ st, int nblk, int lane, float& C, double& S)
{
    float c = kNegInf;
    for (int b = lane; b < nblk; b += 32) c = fmaxf(c, __ldcg(&st[b]).x);
    C = warp_max_f32(c);
    double s = 0.0;
    if (C > kNegInf) {
        for (int b = lane; b < nblk; b += 32) {
            const float2 e = __ldcg(&st[b]);
            if (e.x > kNegInf) s += (double)(e.y * ex2_approx(e.x - C));
            else if (e.y != e.y) s += (double)e.y;
        }
    }
    // a NaN anywhere (NaN reference or NaN sum) must survive
    for (int b = lane; b < nblk; b += 32) {
        const float2 e = __ldcg(&st[b]);
        if (e.x != e.x || e.y != e.y) s = NAN;
    }
    S = warp_sum_f64(s);
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
// decide: one CTA per request.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kDecideThreads) decide_kernel(VerifyParams P)
{
    __shared__ int s_first, s_bad;
    const int r = blockIdx.x;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kWarps = kDecideThreads / 32;

    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    // the request's rows must lie inside the batch, and so must its draft rows (compact index lo - r)
    if (lo < 0 || hi - lo < 1 || hi > n_rows || lo - r < 0 || (hi - 1 - r) > n_rows - P.R) {
        if (tid == 0) {
            atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
            P.accepted_len[r] = 0;
            P.req[r].kind = kTaskNone;
        }
        return;
    }
    const int len = hi - lo - 1;
    const long long drow0 = P.draft_row_start ? P.draft_row_start[r] : (long long)(lo - r);
    if (tid == 0) { s_first = len; s_bad = 0; }
    __syncthreads();
    for (int i = tid; i <= len; i += kDecideThreads) {
        P.out_tokens[lo + i] = -1;
        if (i < len) {
            const int d = P.draft_tokens[lo + i];
            if (d < 0 || d >= P.V) atomicOr(&s_bad, DSPARK_DEV_BAD_TOKEN);
        }
    }
    __syncthreads();
    if (s_bad) {
        if (tid == 0) { atomicOr(P.dev_status, s_bad); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
        return;
    }
    const bool want_all = (P.out_p != nullptr) || (P.out_q != nullptr);
    const double scale_d = (double)P.scale;

    for (int j0 = 0; j0 < len; j0 += kWarps) {
        const int j = j0 + warp;
        if (j < len) {
            float Cp, Cq; double Sp, Sq;
            combine_row(P.stats_t + (long long)(lo + j) * P.nblk, P.nblk, lane, Cp, Sp);
            combine_row(P.stats_d + (long long)(lo - r + j) * P.nblk, P.nblk, lane, Cq, Sq);
            if (lane == 0) {
                if (!row_usable(Cp, Sp) || !row_usable(Cq, Sq)) {
                    atomicOr(&s_bad, DSPARK_DEV_BAD_ROW);
                } else {
                    const int d = P.draft_tokens[lo + j];
                    const double xt = (double)load_logit(P.target, lo + j, P.tstride_bytes, P.elem, d);
                    const double xd = (double)load_logit(P.draft, drow0 + j, P.dstride_bytes, P.elem, d);
                    const double p = exp2(xt * scale_d - (double)Cp) / Sp;
                    const double q = exp2(xd * scale_d - (double)Cq) / Sq;
                    if (P.out_p) P.out_p[lo + j] = (float)p;
                    if (P.out_q) P.out_q[lo + j] = (float)q;
                    float ua, ur;
                    philox_uniforms(P.seed, (uint32_t)r, (uint32_t)j, ua, ur);
                    if (!((double)ua * q < p)) atomicMin(&s_first, j);     // rejected
                }
            }
        }
        __syncthreads();
        const bool stop = s_bad || (!want_all && s_first < len);
        __syncthreads();                         // everyone has read the flags before the next round updates them
        if (stop) break;
    }
    if (warp != 0) return;

    if (s_bad) {
        if (lane == 0) { atomicOr(P.dev_status, s_bad); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
        return;
    }
    const int n = s_first;
    float Cp; double Sp;
    combine_row(P.stats_t + (long long)(lo + n) * P.nblk, P.nblk, lane, Cp, Sp);
    if (!row_usable(Cp, Sp)) {
        if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
        return;
    }
    float Cq = 0.f; double Sq = 1.0;
    if (n < len) combine_row(P.stats_d + (long long)(lo - r + n) * P.nblk, P.nblk, lane, Cq, Sq);
    for (int i = lane; i < n; i += 32) P.out_tokens[lo + i] = P.draft_tokens[lo + i];
    if (lane == 0) {
        float ua, ur;
        philox_uniforms(P.seed, (uint32_t)r, (uint32_t)n, ua, ur);
        RequestTask t;
        t.n = n; t.u = ur; t.slot = -1;
        t.cp = Cp; t.inv_zp = (float)(1.0 / Sp);
        t.cq = Cq; t.inv_zq = (float)(1.0 / Sq);
        t.row_d = drow0 + n;
        if (n < len) {
            const int slot = atomicAdd(&P.counters[0], 1);
            ResidTask q;
            q.request = r; q.row_t = lo + n; q.row_d = t.row_d;
            q.cp = t.cp; q.inv_zp = t.inv_zp; q.cq = t.cq; q.inv_zq = t.inv_zq;
            P.resid[slot] = q;
            t.kind = kTaskResid; t.slot = slot;
        } else {
            t.kind = kTaskBonus;
        }
        P.req[r] = t;
        P.accepted_len[r] = n;
    }
}

// ---------------------------------------------------------------------------------------
// finalize: one warp per request.  Inverse CDF in vocabulary order: first over per-block
// sums (fp64 running sum), then over the elements of the one block that holds the crossing.
// ---------------------------------------------------------------------------------------

// Finds, over values val(b) for b in [0, n) taken in index order, the first index whose
// inclusive running sum exceeds thr.  Each lane owns a contiguous run.  Returns the index
// (or -1), the exclusive sum before it, and the grand total.
template <typename F>
__device__ __forceinline__ int warp_first_crossing(int n, int lane, double thr, F val, double& before, double& total,
                                                   int& last_positive)
{
    const int per = (n + 31) / 32;
    const int b0 = lane * per, b1 = (b0 + per < n) ? b0 + per : n;
    double mine = 0.0;
    int lastp = -1;
    for (int b = b0; b < b1; ++b) { const double x = val(b); mine += x; if (x > 0.0) lastp = b; }
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    total = __shfl_sync(0xffffffffu, incl, 31);
    const double excl = incl - mine;
    const unsigned hit = __ballot_sync(0xffffffffu, incl > thr && b0 < b1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lastp = max(lastp, __shfl_xor_sync(0xffffffffu, lastp, o));
    last_positive = lastp;
    if (!hit) { before = total; return -1; }
    const int src = __ffs(hit) - 1;
    int found = -1;
    double bef = 0.0;
    if (lane == src) {
        double run = excl;
        for (int b = b0; b < b1; ++b) {
            const double x = val(b);
            if (run + x > thr) { found = b; bef = run; break; }
            run += x;
        }
        if (found < 0) { found = b1 - 1; bef = run; }   // only by rounding between the two sums
    }
    found = __shfl_sync(0xffffffffu, found, src);
    before = __shfl_sync(0xffffffffu, bef, src);
    return found;
}

__global__ void __launch_bounds__(kFinalizeThreads) finalize_kernel(VerifyParams P)
{
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (kFinalizeThreads / 32) + (threadIdx.x >> 5);
    if (r >= P.R) return;
    const RequestTask t = P.req[r];
    if (t.kind == kTaskNone) return;
    const int lo = P.row_offsets[r];
    const int row_t = lo + t.n;
    int token = -1;
    bool from_p = (t.kind == kTaskBonus);

    ResidTask rt;
    rt.cp = t.cp; rt.inv_zp = t.inv_zp; rt.cq = t.cq; rt.inv_zq = t.inv_zq;

    if (t.kind == kTaskResid) {
        const float* wb = P.wblk + (long long)t.slot * P.nblk;
        double before, W;
        int lastp;
        // total first (thr depends on it), then the crossing
        warp_first_crossing(P.nblk, lane, INFINITY, [&](int b) { return (double)__ldcg(&wb[b]); }, before, W, lastp);
        if (!(W > 0.0) || !(W < INFINITY)) {
            from_p = true;                                   // empty residual: draw from p with the same u
        } else {
            const double thr = (double)t.u * W;
            int b = warp_first_crossing(P.nblk, lane, thr, [&](int bb) { return (double)__ldcg(&wb[bb]); }, before, W, lastp);
            if (b < 0) b = lastp;
            const int e0 = b * P.epb;
            const int ne = (P.V - e0) < P.epb ? (P.V - e0) : P.epb;
            auto w_of = [&](int e) {
                const float xt = load_logit(P.target, row_t, P.tstride_bytes, P.elem, e0 + e);
                const float xd = load_logit(P.draft, t.row_d, P.dstride_bytes, P.elem, e0 + e);
                return (double)resid_elem(xt, xd, P.scale, rt);
            };
            double bef2, tot2;
            int lp2;
            int e = warp_first_crossing(ne, lane, thr - before, w_of, bef2, tot2, lp2);
            if (e < 0) e = lp2 >= 0 ? lp2 : 0;
            token = e0 + e;
        }
    }
    if (from_p) {
        const float2* st = P.stats_t + (long long)row_t * P.nblk;
        const float C = t.cp;
        auto mass = [&](int b) {
            const float2 e = __ldcg(&st[b]);
            return e.x > kNegInf ? (double)(e.y * ex2_approx(e.x - C)) : 0.0;
        };
        double before, Z;
        int lastp;
        warp_first_crossing(P.nblk, lane, INFINITY, mass, before, Z, lastp);
        const double thr = (double)t.u * Z;
        int b = warp_first_crossing(P.nblk, lane, thr, mass, before, Z, lastp);
        if (b < 0) b = lastp >= 0 ? lastp : 0;
        const float2 sb = __ldcg(&st[b]);
        const int e0 = b * P.epb;
        const int ne = (P.V - e0) < P.epb ? (P.V - e0) : P.epb;
        // inside the block work in the block's own reference: divide the remaining mass by 2^(c_b - C)
        const double thr_local = (thr - before) / (double)ex2_approx(sb.x - C);
        const float nc = -sb.x;
        auto e_of = [&](int e) {
            const float x = load_logit(P.target, row_t, P.tstride_bytes, P.elem, e0 + e);
            return (double)ex2_approx(__fmaf_rn(x, P.scale, nc));
        };
        double bef2, tot2;
        int lp2;
        int e = warp_first_crossing(ne, lane, thr_local, e_of, bef2, tot2, lp2);
        if (e < 0) e = lp2 >= 0 ? lp2 : 0;
        token = e0 + e;
    }
    if (lane == 0) P.out_tokens[row_t] = token;
}

// ---------------------------------------------------------------------------------------
// greedy decide: one warp per request.
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kDecideThreads) greedy_decide_kernel(VerifyParams P)
{
    const int lane = threadIdx.x & 31;
    const int r = blockIdx.x * (kDecideThreads / 32) + (threadIdx.x >> 5);
    if (r >= P.R) return;
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
    if (lo < 0 || hi - lo < 1 || hi > n_rows) {
        if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS); P.accepted_len[r] = 0; }
        return;
    }
    const int len = hi - lo - 1;
    int bad = 0;
    for (int i = lane; i <= len; i += 32) {
        P.out_tokens[lo + i] = -1;
        if (i < len) { const int d = P.draft_tokens[lo + i]; if (d < 0 || d >= P.V) bad = 1; }
    }
    if (__any_sync(0xffffffffu, bad)) {
        if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_TOKEN); P.accepted_len[r] = 0; }
        return;
    }
    __syncwarp();
    int n = len, emitted = -1, status = 0;
    for (int j = 0; j <= len; ++j) {
        const float2* st = P.stats_t + (long long)(lo + j) * P.nblk;
        float best = kNegInf;
        int bi = 0x7fffffff;
        for (int b = lane; b < P.nblk; b += 32) {
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
        int am = bi;
        if (best == kNegInf) { am = 0; status |= DSPARK_DEV_ALL_NEG_INF; }
        if (j == len) { emitted = am; break; }
        if (P.draft_tokens[lo + j] != am) { n = j; emitted = am; break; }
    }
    for (int i = lane; i < n; i += 32) P.out_tokens[lo + i] = P.draft_tokens[lo + i];
    if (lane == 0) {
        P.out_tokens[lo + n] = emitted;
        P.accepted_len[r] = n;
        if (status) atomicOr(P.dev_status, status);
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
                                StreamCfg<kElem, kMode>::kSmemBytes);
}

static bool ensure_attrs()
{
    DeviceInfo& d = device_info();
    if (d.attrs_set) return true;
    bool ok = set_smem_attr<2, kModeStats>() == cudaSuccess && set_smem_attr<4, kModeStats>() == cudaSuccess &&
              set_smem_attr<2, kModeGreedy>() == cudaSuccess && set_smem_attr<4, kModeGreedy>() == cudaSuccess &&
              set_smem_attr<2, kModeResid>() == cudaSuccess && set_smem_attr<4, kModeResid>() == cudaSuccess;
    d.attrs_set = ok;
    return ok;
}

template <int kElem, int kMode>
static void launch_stream(const VerifyParams& P, bool bulk, long long max_units, cudaStream_t s)
{
    const int sms = device_info().sms;
    if (bulk) {
        long long g = (long long)sms * 2;
        if (g > max_units) g = max_units;
        if (g < 1) g = 1;
        stream_bulk_kernel<kElem, kMode><<<(int)g, kStreamThreads, StreamCfg<kElem, kMode>::kSmemBytes, s>>>(P);
    } else {
        long long g = (long long)sms * 8;
        if (g > max_units) g = max_units;
        if (g < 1) g = 1;
        stream_direct_kernel<kElem, kMode><<<(int)g, kConsumerWarps * 32, 0, s>>>(P);
    }
}

template <int kMode>
static void launch_stream_dtype(const VerifyParams& P, bool bulk, long long max_units, cudaStream_t s)
{
    if (P.elem == 2) launch_stream<2, kMode>(P, bulk, max_units, s);
    else launch_stream<4, kMode>(P, bulk, max_units, s);
}

struct Workspace {
    size_t counters, stats_t, stats_d, resid, req, wblk, total;
};
static Workspace workspace_layout(int R, int n_rows, int V)
{
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t nblk = (size_t)blocks_per_row(V, 4);
    Workspace w;
    size_t o = 0;
    w.counters = o; o += up(64 * sizeof(int));
    w.stats_t = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.stats_d = o;  o += up((size_t)n_rows * nblk * sizeof(float2));
    w.resid = o;    o += up((size_t)R * sizeof(ResidTask));
    w.req = o;      o += up((size_t)R * sizeof(RequestTask));
    w.wblk = o;     o += up((size_t)R * nblk * sizeof(float));
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
    P.nblk = blocks_per_row(V, elem);
    P.ppr = pieces_per_row(V, elem);
    P.epb = kBlockBytes / elem;
    P.row_offsets = row_offsets; P.draft_row_start = draft_row_start; P.draft_tokens = draft_tokens;
    P.R = R; P.n_rows_cap = n_rows;
    P.scale = 1.0f; P.seed = 0;
    P.accepted_len = accepted_len; P.out_tokens = out_tokens; P.out_p = nullptr; P.out_q = nullptr;
    P.counters = (int*)(ws + w.counters);
    P.dev_status = dev_status ? dev_status : P.counters + 1;
    P.stats_t = (float2*)(ws + w.stats_t);
    P.stats_d = (float2*)(ws + w.stats_d);
    P.resid = (ResidTask*)(ws + w.resid);
    P.req = (RequestTask*)(ws + w.req);
    P.wblk = (float*)(ws + w.wblk);
    return DSPARK_OK;
}

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
        launch_stream_dtype<kModeGreedy>(P, bulk, (long long)n_rows * P.ppr, s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_GREEDY_DECIDE, s);
        const int warps_per_cta = kDecideThreads / 32;
        greedy_decide_kernel<<<(R + warps_per_cta - 1) / warps_per_cta, kDecideThreads, 0, s>>>(P);
    }
    return launch_status();
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
    if (!draft_logits) return DSPARK_ERR_INVALID_ARG;
    if (!(temperature > 0.0f) || !isfinite(temperature)) return DSPARK_ERR_INVALID_ARG;
    if (draft_row_stride < V) return DSPARK_ERR_SHAPE;
    VerifyParams P;
    int rc = fill_params(P, target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V,
                         row_offsets, draft_row_start, draft_tokens, R, n_rows, accepted_len, out_tokens,
                         dev_status, workspace, workspace_bytes);
    if (rc != DSPARK_OK) return rc;
    P.scale = (float)(1.4426950408889634 / (double)temperature);
    P.seed = seed;
    P.out_p = out_p_tok;
    P.out_q = out_q_tok;
    if (!ensure_attrs()) return launch_status();
    cudaStream_t s = (cudaStream_t)stream;
    const bool bulk = !g_force_direct && aligned16(P.target, P.tstride_bytes, P.row_bytes) &&
                      aligned16(P.draft, P.dstride_bytes, P.row_bytes);
    {
        KernelTimerScope timer(DSPARK_K_STREAM, s);
        launch_stream_dtype<kModeStats>(P, bulk, (long long)(2ll * n_rows - R > 0 ? 2ll * n_rows - R : n_rows) * P.ppr, s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_DECIDE, s);
        decide_kernel<<<R, kDecideThreads, 0, s>>>(P);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_RESIDUAL, s);
        launch_stream_dtype<kModeResid>(P, bulk, (long long)R * P.ppr, s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_FINALIZE, s);
        const int warps_per_cta = kFinalizeThreads / 32;
        finalize_kernel<<<(R + warps_per_cta - 1) / warps_per_cta, kFinalizeThreads, 0, s>>>(P);
    }
    return launch_status();
}

}  // extern "C"
