// dspark_verify / dspark_verify_greedy: the fused ragged-batch speculative verifier
// (acceptance rule of Section 2.1; bonus token of Section 1; flat ragged rows of Section 5.3).
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
#include <cstdio>

#include "verify_device.cuh"

namespace dspark {

// ---------------------------------------------------------------------------------------
// Streamed pass, bulk-copy pipeline: kStages x 32 KB of shared memory per CTA.
// ---------------------------------------------------------------------------------------
// Poll limit of the entry waits of the streamed passes (a consumer waiting for data, the producer waiting for a
// free stage or for the launch tag).  dspark_set_wait_poll_limit shortens it for diagnostics; the producer's
// wait for copies it has already issued always keeps the long bound, so that no copy can land in the shared
// memory of a CTA that has left.
__device__ uint32_t g_entry_poll_limit = kWaitPollLimit;

// kReqScale (statistics pass only): one temperature per request, and every request's exponent scale kept in shared
// memory beside the request table (P.req_scale_smem); an instantiation of its own, so that the plain pass keeps its code.
template <int kElem, int kMode, bool kReqScale = false>
__global__ void __launch_bounds__(kStreamThreads, 3) stream_bulk_kernel(VerifyParams P)
{
    using M = ModeCfg<kMode>;
    extern __shared__ __align__(128) unsigned char stage_mem[];
    __shared__ __align__(8) uint64_t full_bar[kStages];
    __shared__ __align__(8) uint64_t empty_bar[kStages];
    __shared__ UnitSlot s_unit[kStages];
    __shared__ __align__(8) uint64_t hist_bar[2];
    __shared__ int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kConsumerWarps); }
        if (kMode == kModeHist) { mbar_init(&hist_bar[0], kConsumerWarps); mbar_init(&hist_bar[1], kConsumerWarps); }
        s_abort = 0;
        mbar_fence_init();
    }
    // histogram pass: two histograms of one unit each behind the stages (units alternate between them)
    unsigned int* unit_bins = reinterpret_cast<unsigned int*>(stage_mem + kStages * kStageBytes);
    if (kMode == kModeHist)
        for (int i = tid; i < 2 * kHistBins; i += kStreamThreads) unit_bins[i] = 0u;
    __syncthreads();
    pdl_wait();                                  // everything below reads what earlier kernels wrote

    const uint32_t entry_limit = g_entry_poll_limit;
    // Statistics pass without the bonus rows: every CTA keeps row_offsets[r] - r behind its stages (see below).  The
    // offsets are asked for before anything waits for the row count, so that the prologue costs one trip to the L2.
    constexpr int kPrefPer = (kSkipBonusMaxRequests + kStreamThreads) / kStreamThreads;
    int pref_reg[kPrefPer];
    float temp_reg[kPrefPer];                    // one temperature per request: they ride along (P.req_scale_smem)
    if (kMode == kModeStats && P.skip_bonus) {
#pragma unroll
        for (int k = 0; k < kPrefPer; ++k) {
            const int r = tid + k * kStreamThreads;
            pref_reg[k] = r <= P.R ? P.row_offsets[r] - r : 0;
            temp_reg[k] = (kReqScale && r < P.R) ? P.req_temp[r] : 1.0f;
        }
    }
    bool bad_rows;
    const int n_rows = device_rows(P, &bad_rows);
    if (kMode != kModeResid && kMode != kModeHist && blockIdx.x == 0 && tid == 0) {
        P.counters[0] = 0;                       // residual queue, filled by the decide kernel
        P.counters[kCtrBonus] = 0;               // and the bonus rows it queues from the back
        *unit_counter<kModeResid>(P) = 0ull;     // unit counters of the passes that follow this one in the call
        *unit_counter<kModeHist>(P) = 0ull;
        reinterpret_cast<unsigned long long*>(P.counters)[kCellRetryUnits] = 0ull;
        P.counters[kCtrRetry] = 0;               // rows of the threshold search's second look
        *unit_counter<kMode>(P) = 0ull;          // and this pass's own, published by the tag
        __threadfence();
        atomicExch(unit_tag(P), P.launch_tag);
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int n_streams = stream_count<kMode>(P, n_rows);
    const int nblk = (kMode == kModeResid) ? P.nblk_r : P.nblk;
    const int ppr = (nblk + kConsumerWarps - 1) / kConsumerWarps;
    // the second pass also streams the bonus rows queued from the back of the task array, in 32 KB pieces
    const int ppr_b = (P.nblk + kConsumerWarps - 1) / kConsumerWarps;
    int n_bonus = 0;
    if (kMode == kModeResid && P.skip_bonus) {
        n_bonus = __ldcg(&P.counters[kCtrBonus]);
        n_bonus = n_bonus < 0 ? 0 : (n_bonus > P.resid_cap - n_streams ? P.resid_cap - n_streams : n_bonus);
    }
    const long long total_first = (long long)n_streams * ppr;
    const long long total = total_first + (long long)n_bonus * ppr_b;
    volatile int* abort_flag = &s_abort;
    // Statistics pass without the bonus rows: the target rows that are not bonus rows are, in order, the draft
    // positions of the batch, so stream s' of them is target row s' + r for the request r it falls into.  Every CTA
    // keeps row_offsets[r] - r behind its stages (one coalesced read) and finds r by a search in shared memory.
    int* pref = reinterpret_cast<int*>(stage_mem + kStages * kStageBytes);
    const bool skip_bonus = kMode == kModeStats && P.skip_bonus;
    const int nd = n_rows > P.R ? n_rows - P.R : 0;
    // Where it fits behind that array: the request of every draft position, so that a unit costs its producer one
    // look-up instead of a search (and a draft unit no search through global memory for its physical row).
    unsigned short* req_of = reinterpret_cast<unsigned short*>(pref + ((P.R + 4) & ~3));
    const bool have_req_of = skip_bonus && P.req_table;
    // and, with one temperature per request, every request's exponent scale log2(e)/T behind that table (no kernel
    // that expands the temperatures to rows is needed then: the producer knows each unit's request)
    float* scale_of = reinterpret_cast<float*>(req_of + ((P.req_table + 7) & ~7));
    const bool have_scale_of = kReqScale && have_req_of;
    if (skip_bonus) {
#pragma unroll
        for (int k = 0; k < kPrefPer; ++k) {
            const int r = tid + k * kStreamThreads;
            if (r <= P.R) pref[r] = pref_reg[k];
            if (have_scale_of && r < P.R) {
                const float T = temp_reg[k];
                scale_of[r] = (T > 0.0f && T < INFINITY) ? (float)(1.4426950408889634 / (double)T) : 1.0f;
            }
        }
        __syncthreads();
        if (have_req_of) {
            for (int r = tid; r < P.R; r += kStreamThreads) {
                int a = pref[r], b = pref[r + 1];
                a = a < 0 ? 0 : a; b = b > P.req_table ? P.req_table : b;
                for (int i = a; i < b; ++i) req_of[i] = (unsigned short)r;
            }
            __syncthreads();
        }
    }

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
                if (live && kMode == kModeResid && u >= total_first) {
                    // a bonus row: task from the back of the queue, one 32 KB piece of the target row
                    const long long v = u - total_first;
                    const int tb = (int)(v / ppr_b);
                    slot.s = P.resid_cap - 1 - tb;
                    slot.piece = (int)(v - (long long)tb * ppr_b);
                    slot.task = P.resid[slot.s];
                    slot.scale = slot.task.scale;
                    const long long off = (long long)slot.piece * kStageBytes;
                    const long long rem = (long long)P.row_bytes - off;
                    bytes = (int)(rem < kStageBytes ? rem : kStageBytes);
                    src0 = P.target + (long long)slot.task.row_t * P.tstride_bytes + off;
                } else if (live) {
                    slot.s = total <= 0x7fffffffll ? (int)((unsigned)u / (unsigned)ppr) : (int)(u / ppr);
                    slot.piece = (int)(u - (long long)slot.s * ppr);
                    long long draft_row = -2;                // physical draft row, where it is found here
                    float own_scale = 0.f;                   // exponent scale of the unit's request, where it is known here
                    if (skip_bonus) {
                        // draft position ds of the batch (target stream s' = ds, draft stream s' = nd + ds) belongs to
                        // the largest r with row_offsets[r] - r <= ds
                        const int ds = slot.s < nd ? slot.s : slot.s - nd;
                        int lo = 0;
                        if (have_req_of && ds < P.req_table) {
                            lo = req_of[ds];
                            if (lo >= P.R) lo = P.R - 1;                    // only with inconsistent offsets
                            if (have_scale_of) own_scale = scale_of[lo];
                        } else if (slot.s < nd) {
                            int hi = P.R;
                            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (pref[mid] <= ds) lo = mid; else hi = mid; }
                        }
                        if (slot.s < nd) {
                            slot.s = ds + lo;
                            if (slot.s >= n_rows) slot.s = n_rows - 1;      // only with inconsistent offsets
                        } else {
                            slot.s = n_rows + ds;
                            if (have_req_of && ds < P.req_table) {
                                const int j = ds - pref[lo], len = pref[lo + 1] - pref[lo];
                                draft_row = !P.draft_row_start ? (long long)ds
                                                               : ((j >= 0 && j < len) ? P.draft_row_start[lo] + j : -1);
                            }
                        }
                    }
                    if (kMode == kModeResid) slot.task = P.resid[slot.s];
                    if (kMode == kModeHist) {
                        if (P.hist_retry) {                  // second look: the rows the first one listed
                            const int row = __ldcg(&P.retry_rows[slot.s]);
                            slot.s = row < 0 ? 0 : (row >= n_rows ? n_rows - 1 : row);
                        }
                        slot.trunc = P.trunc_rows[slot.s];
                    }
                    unit_sources<kMode>(P, slot.s, slot.piece, n_rows, src0, src1, bytes, kMode == kModeResid ? &slot.task : nullptr,
                                        draft_row);
                    slot.scale = have_scale_of ? (own_scale != 0.f ? own_scale : 1.0f)     // (no per-row scales exist then)
                                               : stream_scale<kMode>(P, slot.s, n_rows, n_streams + (skip_bonus ? P.R : 0));
                } else {
                    slot.s = -1; slot.piece = 0; slot.scale = 0.f;
                }
            }
            if (*abort_flag) return false;
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&empty_bar[st], ph ^ 1u, entry_limit))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                return false;
            }
            if (lane == 0) {
                // read by the consumers after the barrier below completes
                s_unit[st].s = slot.s; s_unit[st].piece = slot.piece; s_unit[st].scale = slot.scale;
                if (kMode == kModeResid) s_unit[st].task = slot.task;
                if (kMode == kModeHist) s_unit[st].trunc = slot.trunc;
                if (live) {
                    unsigned char* dst = stage_mem + st * kStageBytes;
                    const bool two = M::kSrc == 2 && src1 != nullptr;
                    mbar_arrive_expect_tx(&full_bar[st], (uint32_t)(two ? 2 * bytes : bytes));
                    bulk_g2s_hint(dst, src0, (uint32_t)bytes, &full_bar[st], pol_first);
                    if (two) bulk_g2s_hint(dst + M::kPieceBytes, src1, (uint32_t)bytes, &full_bar[st], pol_first);
                    if (!counter_ready && !(counter_ready = wait_for_tag(unit_tag(P), P.launch_tag, entry_limit))) {
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
            if (!__all_sync(0xffffffffu, mbar_wait_bounded(&full_bar[st], ph, entry_limit))) {
                if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                break;
            }
            const int unit_s = s_unit[st].s, unit_piece = s_unit[st].piece;
            const float unit_scale = s_unit[st].scale;
            if (unit_s < 0) break;
            unsigned char* sp = stage_mem + st * kStageBytes + warp * M::kBlockBytes;
            SmemFetch f0{sp}, f1{sp + M::kPieceBytes};
            if constexpr (kMode == kModeHist) {
                // The eight blocks of the unit are counted into one histogram in shared memory; when all consumer
                // warps have added theirs (a barrier of their own, bounded like every wait), each thread moves
                // its share of the non-empty bins to the row's counts and leaves them zero for the unit after next.
                const uint32_t window = s_unit[st].trunc.size & ~kWindowDense;
                unsigned int* h = unit_bins + (it & 1) * kHistBins;
                consume_block<kElem, kMode>(P, unit_s, unit_piece, n_rows, warp, lane, f0, f1, unit_scale, nullptr,
                                            &s_unit[st].trunc, h);
                __syncwarp();
                if (lane == 0) { mbar_arrive(&empty_bar[st]); mbar_arrive(&hist_bar[it & 1]); }
                if (!__all_sync(0xffffffffu, mbar_wait_bounded(&hist_bar[it & 1], (uint32_t)(it >> 1) & 1u, entry_limit))) {
                    if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_TIMEOUT); *abort_flag = 1; }
                    break;
                }
                unsigned int* bins = P.trunc_bins + (long long)unit_s * kHistBins;
#pragma unroll
                for (int j = 0; j < kHistBins / (kConsumerWarps * 32); ++j) {
                    const uint32_t d = (uint32_t)(j * kConsumerWarps * 32 + warp * 32 + lane);
                    const unsigned int c = d < window ? h[d] : 0u;
                    if (c) { atomicAdd(&bins[d], c); h[d] = 0u; }
                }
            } else {
                consume_block<kElem, kMode>(P, unit_s, unit_piece, n_rows, warp, lane, f0, f1, unit_scale,
                                            kMode == kModeResid ? &s_unit[st].task : nullptr, nullptr);
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[st]);
            }
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
        P.counters[kCtrRetry] = 0;
        if (bad_rows) atomicOr(P.dev_status, DSPARK_DEV_BAD_OFFSETS);
    }
    const int n_streams = stream_count<kMode>(P, n_rows);
    const int nblk = (kMode == kModeResid) ? P.nblk_r : P.nblk;
    UnitCursor cur;
    cur.init((nblk + kConsumerWarps - 1) / kConsumerWarps);
    for (; cur.s < n_streams; cur.next()) {
        const unsigned char *src0, *src1;
        int bytes;
        int row = cur.s;
        if (kMode == kModeHist && P.hist_retry) {            // second look of the threshold search: the listed rows
            row = __ldcg(&P.retry_rows[cur.s]);
            row = row < 0 ? 0 : (row >= n_rows ? n_rows - 1 : row);
        }
        unit_sources<kMode>(P, row, cur.piece, n_rows, src0, src1, bytes);
        GlobalFetch<kElem> f0{src0 + warp * M::kBlockBytes};
        GlobalFetch<kElem> f1{(kMode == kModeResid ? src1 : src0) + warp * M::kBlockBytes};
        consume_block<kElem, kMode>(P, row, cur.piece, n_rows, warp, lane, f0, f1,
                                    stream_scale<kMode>(P, row, n_rows, n_streams));
    }
}

// ---------------------------------------------------------------------------------------
// top-k / top-p truncation of the target distribution inside the verifier (bf16 rows).
// The kept set of a row is {v : x_v >= tau}; tau is found exactly on the 16-bit keys:
//   trunc_prep    per target row: row maximum m (recovered exactly from the statistics: the reference
//                 c = m * scale determines the bf16 value m), the window of keys below m (down to the k-th largest
//                 block maximum for top-k of at most one token per block; to m - 8 T or the bound on the nucleus for
//                 top-p alone; else kHistBins keys), zeroed counters;
//   stream<Hist>  one more streamed pass over the target rows counts the keys inside the window (per 32 KB unit in
//                 shared memory, non-empty bins added to the row's counts);
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

// The window of keys from the row maximum down to lo_val (at most kHistBins keys, and no key below the lowest).
__device__ __forceinline__ void key_window(float lo_val, uint32_t kmax, uint32_t& size, uint32_t& cut2)
{
    const uint32_t klo = bf16_key((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rd(lo_val)));
    size = kHistBins;
    if (klo <= kmax && kmax - klo + 1u < (uint32_t)kHistBins) size = kmax - klo + 1u;
    if (size > kmax + 1u) size = kmax + 1u;                          // keys 0 .. kmax exist
    const uint32_t cb = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(bf16_key_value(kmax - (size - 1u))));
    cut2 = cb | (cb << 16);
    // a wide window of positive values only: counted by the distance of the bit patterns (consume_block)
    if (size >= 256u && kmax - (size - 1u) > 0x8000u) size |= kWindowDense;
}

// Top-p: the tokens below a value v weigh at most V 2^(v scale - C) together, so the nucleus ends above the v at
// which that is (1 - p) Z.
__device__ __forceinline__ float nucleus_floor(float C, float Z, float p, float scale, int V)
{
    return (C + log2f((1.f - p) * Z / (float)V)) / scale - 0.07f / scale;
}

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
        // The window's lower end.  Top-k of at most one token per block: the k-th largest block maximum (tau is at
        // least tau_k, which cannot lie below it; the smallest block maximum would do and needs no ranking, but the
        // short last block of a row pulls it down, and every token more in the window costs a divergent branch).  Top-k of more tokens: every key the histogram has (for a maximum
        // of 13 the kHistBins keys below it reach down to 0.05).  Top-p alone: m - 8 T, where a peaked row's nucleus
        // ends, unless the bound on the nucleus is nearer; a row it does not resolve gets a second look down to
        // that bound (trunc_scan_kernel).
        float lo_val = m;
        if (use_p) lo_val = fmaxf(nucleus_floor(A.C, (float)A.S, pf, scale, P.V), m - 8.f * temp);
        if (use_k && k > P.nblk) lo_val = -INFINITY;
        if (use_k && k <= P.nblk) {
            // every block maximum is an element of the row, so the k-th largest logit is at least the k-th
            // largest block maximum: the window reaches down to it (rank by counting, 64-128 blocks)
            const float2* st = P.stats_t + (long long)row * P.nblk;
            float kth = kNegInf;
            if (P.nblk <= 64) {                              // two block references per lane, compared through shuffles
                float c[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) c[q] = (q * 32 + lane < P.nblk) ? __ldcg(&st[q * 32 + lane]).x : kNegInf;
                int rank[2] = {0, 0};                        // blocks that come before mine in descending order
#pragma unroll
                for (int q2 = 0; q2 < 2; ++q2) {
                    if (q2 * 32 >= P.nblk) break;
#pragma unroll 8
                    for (int l2 = 0; l2 < 32; ++l2) {
                        const float cj = __shfl_sync(0xffffffffu, c[q2], l2);
                        const int j = q2 * 32 + l2;
#pragma unroll
                        for (int q = 0; q < 2; ++q) rank[q] += (cj > c[q]) || (cj == c[q] && j < q * 32 + lane);
                    }
                }
#pragma unroll
                for (int q = 0; q < 2; ++q)
                    if (q * 32 + lane < P.nblk && rank[q] == k - 1) kth = c[q];
            } else if (P.nblk <= 128) {                      // four per lane
                float c[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) c[q] = (q * 32 + lane < P.nblk) ? __ldcg(&st[q * 32 + lane]).x : kNegInf;
                int rank[4] = {0, 0, 0, 0};
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
            if (kth > kNegInf) lo_val = __bfloat162float(__float2bfloat16_rn(kth / scale));
            else if (!use_p) lo_val = -INFINITY;
        }
        if (!(lo_val <= m)) lo_val = m;
        uint32_t size, cut2;
        key_window(lo_val, kmax, size, cut2);
        tr.kmax = kmax; tr.size = size; tr.cut2 = cut2; tr.scale = scale;
        tr.k = use_k ? k : 0; tr.p = use_p ? pf : 1.f;
        unsigned int* bins = P.trunc_bins + (long long)row * kHistBins;
        for (uint32_t i = lane; i < (size & ~kWindowDense); i += 32) bins[i] = 0u;
    }
    if (lane == 0) { P.trunc_rows[row] = tr; T.tau[row] = kNegInf; P.trunc_flag[row] = 0; P.trunc_z[row] = -1.0; }
    if (row == 0 && lane == 0) {                                         // the per-row fallback's work counter and the
        P.trunc_flag[P.n_rows_cap] = 0;                                  // number of rows left to it
        P.trunc_flag[P.n_rows_cap + 1] = 0;
    }
}

constexpr int kScanThreads = 256;
// A row its window did not resolve: after the first look it is listed for a second one with the window the bound on
// its nucleus gives (counts zeroed here), if that is deeper; else (and after the second look) it goes to the per-row
// search.  Called by all threads of the row's CTA.
__device__ __forceinline__ void leave_unresolved(const VerifyParams& P, int row, const TruncRow& tr, int retry, int tid)
{
    uint32_t size = 0u, cut2 = 0u;
    if (!retry && tr.k == 0 && tr.p < 1.f && tr.p > 0.f)
        key_window(nucleus_floor(tr.C, tr.Z, tr.p, tr.scale, P.V), tr.kmax, size, cut2);
    if ((size & ~kWindowDense) > tr.size) {
        unsigned int* bins = P.trunc_bins + (long long)row * kHistBins;
        for (uint32_t i = tid; i < (size & ~kWindowDense); i += kScanThreads) bins[i] = 0u;
        if (tid == 0) {
            P.trunc_rows[row].size = size;
            P.trunc_rows[row].cut2 = cut2;
            P.trunc_flag[row] = 2;
            const int slot = atomicAdd(&P.counters[kCtrRetry], 1);
            if (slot < P.n_rows_cap) P.retry_rows[slot] = row;
        }
    } else if (tid == 0) {
        P.trunc_flag[row] = 1;
        atomicAdd(&P.trunc_flag[P.n_rows_cap + 1], 1);
    }
}

__global__ void __launch_bounds__(kScanThreads) trunc_scan_kernel(VerifyParams P, TruncArgs T, int retry)
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
    if (retry && P.trunc_flag[row] != 2) return;            // the second look is for the rows listed by the first
    TruncRow tr = P.trunc_rows[row];
    tr.size &= ~kWindowDense;
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
        leave_unresolved(P, row, tr, retry, tid);
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
                leave_unresolved(P, row, tr, retry, tid);
                return;
            }
            if (dp < dist) dist = dp;
        }
    }
    if (tid == 0 && dist != 0x7fffffff) T.tau[row] = bf16_key_value(tr.kmax - (uint32_t)dist);
    if (tid == 0 && retry) P.trunc_flag[row] = 0;           // resolved by the second look
    if (dist != 0x7fffffff && dist / kPer == tid) {         // mass of the kept set: what the accept test divides by
        double q = m_excl;
        for (int j = 0; j <= dist % kPer; ++j) q += mass[j];
        P.trunc_z[row] = q;
    }
}

// One warp per (bonus row, statistics block): s = sum over x >= tau of 2^(x * scale - c).  Only a bonus token is drawn
// from a target row's block sums; the accept tests take the mass of the kept set from the key counts (trunc_z) and
// the residual pass sums its own blocks.
__global__ void __launch_bounds__(256) trunc_sums_kernel(VerifyParams P, TruncArgs T)
{
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = P.row_offsets[blockIdx.x + 1] - 1;      // the last row of request blockIdx.x
    const int b = blockIdx.y * 8 + (threadIdx.x >> 5);
    bool bad_rows;
    if (row < 0 || row >= device_rows(P, &bad_rows) || b >= P.nblk) return;
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
// Row statistics on their own (dspark_row_stats): what the statistics pass and the accept kernel compute for a row,
// (reference, sum) = (max * scale, sum 2^(x * scale - reference)), for a caller that produces logits and wants to hand
// their statistics to dspark_verify_draft_stats.  One CTA per row; same blocks, same block arithmetic and same order
// of combination as the verifier, so the result is bit-identical to what the verifier would have computed.
// ---------------------------------------------------------------------------------------
constexpr int kRowStatsThreads = 256;
constexpr int kRowStatsMaxBlocks = 2048;
template <int kElem>
__global__ void __launch_bounds__(kRowStatsThreads) row_stats_kernel(const unsigned char* logits, long long stride_bytes, int V,
                                                                      int n_rows, float temperature, const float* row_temperatures,
                                                                      float2* out)
{
    __shared__ float2 s_e[kRowStatsMaxBlocks];
    pdl_wait();
    const int row = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (row >= n_rows) return;
    const float T = row_temperatures ? row_temperatures[row] : temperature;
    if (!(T > 0.f) || !(T < INFINITY)) {
        if (threadIdx.x == 0) out[row] = make_float2(NAN, NAN);
        return;
    }
    const float scale = (float)(1.4426950408889634 / (double)T);
    const int row_bytes = V * kElem;
    const int nblk = blocks_per_row(V, kElem, kStatBlockBytes);
    const unsigned char* base = logits + (long long)row * stride_bytes;
    for (int b = warp; b < nblk; b += kRowStatsThreads / 32) {
        const int rem = row_bytes - b * kStatBlockBytes;
        uint4 v[kStatVec];
        load_block<kElem, kStatVec>(GlobalFetch<kElem>{base + (long long)b * kStatBlockBytes}, rem < kStatBlockBytes ? rem : kStatBlockBytes, lane, v);
        const float2 e = block_stats<kElem, kStatVec>(v, scale);
        if (lane == 0) s_e[b] = e;
    }
    __syncthreads();
    if (warp != 0) return;
    RowAcc A;
    A.init();
    for (int b0 = 0; b0 < nblk; b0 += 128) {
        float2 e[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) { const int i = b0 + k * 32 + lane; e[k] = i < nblk ? s_e[i] : make_float2(kNegInf, 0.f); }
#pragma unroll
        for (int k = 0; k < 4; ++k) A.add(e[k]);
    }
    A.finish();
    if (lane == 0) out[row] = make_float2(A.C, (float)A.S);
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
// kDraftStats: the draft rows' (reference, sum) come from the drafter (P.draft_stats) instead of the statistics pass.
template <bool kDraftStats>
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
    // no barrier here: the token check is looked at after the first round of positions, whose barrier covers it
    const bool want_all = (P.out_p != nullptr) || (P.out_q != nullptr);
    float scale_f = P.scale;
    if (P.req_temp) {
        const float T = P.req_temp[r];
        if (!(T > 0.0f) || !(T < INFINITY)) {
            __syncthreads();                     // a request reports everything that is wrong with it
            if (tid == 0) { atomicOr(P.dev_status, s_bad | DSPARK_DEV_BAD_TEMPERATURE); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone; }
            return;
        }
        scale_f = (float)(1.4426950408889634 / (double)T);
    }
    const double scale_d = (double)scale_f;

    // (P.skip_bonus: the bonus row has not been streamed; it is looked at by the draw kernel if the request gets there)
    const int last_pos = P.skip_bonus ? len - 1 : len;
    for (int j0 = 0; j0 <= last_pos; j0 += kWarps) {
        const int j = j0 + warp;
        if (j <= last_pos) {
            const bool is_draft_pos = j < len;
            // the two logits at the draft token do not depend on the statistics: fetch them first
            float xt = 0.f, xd = 0.f;
            bool tok_ok = true;
            if (is_draft_pos && lane == 0) {
                const int d = P.draft_tokens[lo + j];
                tok_ok = d >= 0 && d < P.V;          // a token out of range voids the request (flagged by the scan above)
                if (tok_ok) {
                    xt = load_logit(P.target, lo + j, P.tstride_bytes, P.elem, d);
                    xd = load_logit(P.draft, drow0 + j, P.dstride_bytes, P.elem, d);
                }
            }
            RowAcc A, D;
            if (kDraftStats) {
                // the drafter kept the statistics of the rows it wrote: nothing of the draft row was streamed
                float2 ds = make_float2(kNegInf, 0.f);
                if (is_draft_pos) ds = __ldg(&P.draft_stats[drow0 + j]);
                combine_rows(P.stats_t + (long long)(lo + j) * P.nblk, nullptr, P.nblk, lane, A, D);
                D.C = ds.x; D.S = (double)ds.y;
            } else {
                combine_rows(P.stats_t + (long long)(lo + j) * P.nblk,
                             is_draft_pos ? P.stats_d + (long long)(lo - r + j) * P.nblk : nullptr, P.nblk, lane, A, D);
            }
            if (P.trunc_z && is_draft_pos) {
                // truncated target (top-k / top-p) by the streamed search: the mass of the kept set comes from the key
                // counts (a bonus row, and a row left to the per-row search, carry it in their block sums instead)
                const double zs = __ldcg(&P.trunc_z[lo + j]);
                if (zs > 0.0) A.S = zs;
            }
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
                if (is_draft_pos && tok_ok) {
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
        const bool stop = void_req || (!want_all && first < len) || s_bad != 0;
        __syncthreads();                         // everyone has read the flags before the next round updates them
        if (stop) break;
    }

    if (tid != 0) return;
    if (s_bad) {                                 // a draft token outside the vocabulary
        atomicOr(P.dev_status, s_bad); P.accepted_len[r] = 0; P.req[r].kind = kTaskNone;
        return;
    }
    const int n = s_first;
    RequestRec rec;
    rec.kind = kTaskNone; rec.row_t = lo + n; rec.row_d = drow0 + n;
    rec.cp = rec.cq = 0.f; rec.inv_zp = rec.inv_zq = 1.f; rec.u = 0.f; rec.scale = scale_f; rec.pad = 0;
    rec.tau = kNegInf;
    const bool void_req = want_all ? s_first_bad != 0x7fffffff : s_first_bad < n;
    const bool bonus_later = P.skip_bonus && n == len;         // every draft token accepted, its bonus row not seen yet
    if (bonus_later) {
        if (void_req) {
            atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW);
            P.accepted_len[r] = 0;
        } else {
            // queue the bonus row for the second pass (one source: row_d < 0); the draw kernel combines its statistics
            for (int i = 0; i < n; ++i) P.out_tokens[lo + i] = P.draft_tokens[lo + i];
            float ua, ur;
            philox_uniforms(P.seed, (uint32_t)r, (uint32_t)n, ua, ur);
            P.accepted_len[r] = n;
            rec.u = ur;
            rec.kind = kTaskBonus;
            const int slot = P.resid_cap - 1 - atomicAdd(&P.counters[kCtrBonus], 1);
            ResidTask q;
            q.request = r; q.row_t = rec.row_t; q.row_d = -1;
            q.cp = q.cq = 0.f; q.inv_zp = q.inv_zq = 1.f;
            q.u = ur; q.scale = scale_f; q.wslot = r; q.tau = kNegInf;
            P.resid[slot] = q;
        }
    } else if (void_req || !s_have_fin || !row_usable(s_fin_C[0], s_fin_S[0]) ||
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
    // and, where the second pass streams the bonus rows, the block statistics it left for this request (up to 256
    // blocks in registers; whether the request drew a bonus token at all is in the record)
    const float2* sb = P.stats_b + (long long)r * P.nblk;
    float2 eb[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int i = k * 32 + lane;
        eb[k] = (P.skip_bonus && i < P.nblk) ? __ldcg(&sb[i]) : make_float2(kNegInf, 0.f);
    }
    if (rec.kind == kTaskNone) return;
    Level2Scratch<kElem>& S = s_scr[warp];
    const double u = (double)rec.u;
    const unsigned char* trow = P.target + (long long)rec.row_t * P.tstride_bytes;
    int token = -1;
    // A bonus row that the second pass has streamed (P.skip_bonus): its row statistics are combined here, and here
    // it turns out whether the row can be normalised at all; its block masses then come from the saved statistics
    // exactly as on the second attempt of a rejected row below.
    const bool late_bonus = P.skip_bonus && rec.kind == kTaskBonus;
    float cp = rec.cp;
    if (late_bonus) {
        RowAcc A, D;
        if (P.nblk <= 256) {                   // the entries in the order combine_rows takes them
            A.init();
#pragma unroll
            for (int k = 0; k < 8; ++k) A.add(eb[k]);
            A.finish();
        } else {
            combine_rows(sb, nullptr, P.nblk, lane, A, D);
        }
        if (!row_usable(A.C, A.S)) {
            const int lo = P.row_offsets[r], hi = P.row_offsets[r + 1];
            for (int i = lo + lane; i < hi; i += 32) P.out_tokens[i] = -1;
            if (lane == 0) { atomicOr(P.dev_status, DSPARK_DEV_BAD_ROW); P.accepted_len[r] = 0; }
            return;
        }
        cp = A.C;
    }
    for (int attempt = late_bonus ? 1 : 0; attempt < 2 && token < 0; ++attempt) {
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
                if (i < P.nblk && P.nblk <= 256) {
                    const float2 e = late_bonus ? eb[k] : __ldcg(&st[i]);
                    m = e.x > kNegInf ? e.y * ex2_approx(e.x - cp) : 0.f;
                }
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
            const float2* st = late_bonus ? sb : P.stats_t + (long long)rec.row_t * P.nblk;
            auto mass = [&](int i) { const float2 e = __ldcg(&st[i]); return e.x > kNegInf ? e.y * ex2_approx(e.x - cp) : 0.f; };
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
            const float nc = -cp, scale = rec.scale, tau = rec.tau;
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
static std::atomic<int> g_skip_bonus{1};      // diagnostic switch: 0 streams every bonus row in the statistics pass
static std::atomic<int> g_stream_path{0};     // 0 automatic, 1 direct loads, 2 bulk copies in separate passes

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

template <int kElem, int kMode, bool kReqScale = false>
static cudaError_t set_smem_attr()
{
    return cudaFuncSetAttribute(stream_bulk_kernel<kElem, kMode, kReqScale>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                kStages * kStageBytes + (kMode == kModeStats ? kSkipBonusSmemBytes : 0) +
                                    (kMode == kModeHist ? 2 * kHistBins * (int)sizeof(unsigned int) : 0));
}

static bool ensure_attrs()
{
    DeviceInfo& d = device_info();
    if (d.attrs_set) return true;
    bool ok = set_smem_attr<2, kModeStats>() == cudaSuccess && set_smem_attr<4, kModeStats>() == cudaSuccess &&
              set_smem_attr<2, kModeGreedy>() == cudaSuccess && set_smem_attr<4, kModeGreedy>() == cudaSuccess &&
              set_smem_attr<2, kModeResid>() == cudaSuccess && set_smem_attr<4, kModeResid>() == cudaSuccess &&
              set_smem_attr<2, kModeHist>() == cudaSuccess &&
              set_smem_attr<2, kModeStats, true>() == cudaSuccess && set_smem_attr<4, kModeStats, true>() == cudaSuccess;
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
        size_t smem = (size_t)kStages * kStageBytes;
        if (kMode == kModeStats && P.skip_bonus)
            smem += (size_t)((P.R + 4) / 4) * 16 + (size_t)((P.req_table + 7) / 8) * 16 + (P.req_scale_smem ? (size_t)((P.R + 3) / 4) * 16 : 0);
        if (kMode == kModeHist) smem += 2 * kHistBins * sizeof(unsigned int);
        if (kMode == kModeStats && P.req_scale_smem)
            launch_pdl(stream_bulk_kernel<kElem, kMode, kMode == kModeStats>, dim3((unsigned)g), dim3(kStreamThreads), smem, s, P);
        else
            launch_pdl(stream_bulk_kernel<kElem, kMode>, dim3((unsigned)g), dim3(kStreamThreads), smem, s, P);
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

static bool aligned16(const void* p, long long stride_bytes, long long row_bytes)
{
    return (((uintptr_t)p) & 15u) == 0 && (stride_bytes & 15) == 0 && (row_bytes & 15) == 0;
}

// Argument checks and everything of the parameter block that does not live in the workspace.
static int fill_common(VerifyParams& P, const void* target, const void* draft, int dtype,
                       int64_t tstride, int64_t dstride, int V, const int32_t* row_offsets,
                       const int64_t* draft_row_start, const int32_t* draft_tokens, int R, int n_rows,
                       int32_t* accepted_len, int32_t* out_tokens)
{
    if (!target || !row_offsets || !draft_tokens || !accepted_len || !out_tokens) return DSPARK_ERR_INVALID_ARG;
    if (dtype != DSPARK_F32 && dtype != DSPARK_BF16) return DSPARK_ERR_INVALID_ARG;
    if (R < 1 || V < 1 || n_rows < R) return DSPARK_ERR_INVALID_ARG;
    const int elem = dtype == DSPARK_BF16 ? 2 : 4;
    if ((long long)V * elem >= (1ll << 31) || tstride < V) return DSPARK_ERR_SHAPE;
    P = VerifyParams{};
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
    P.launch_tag = next_launch_tag();
    P.resid_cap = R;
    P.req_temp = nullptr;
    P.tau = nullptr;
    P.draft_stats = nullptr;
    P.skip_bonus = 0;
    return DSPARK_OK;
}

static int fill_params(VerifyParams& P, const void* target, const void* draft, int dtype,
                       int64_t tstride, int64_t dstride, int V, const int32_t* row_offsets,
                       const int64_t* draft_row_start, const int32_t* draft_tokens, int R, int n_rows,
                       int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                       void* workspace, size_t workspace_bytes)
{
    int rc = fill_common(P, target, draft, dtype, tstride, dstride, V, row_offsets, draft_row_start, draft_tokens, R, n_rows,
                         accepted_len, out_tokens);
    if (rc != DSPARK_OK) return rc;
    const Workspace w = workspace_layout(R, n_rows, V);
    if (!workspace || workspace_bytes < w.total) return DSPARK_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255u) != 0) return DSPARK_ERR_ALIGNMENT;
    unsigned char* ws = (unsigned char*)workspace;
    P.counters = (int*)(ws + w.counters);
    P.dev_status = dev_status ? dev_status : P.counters + 1;
    P.stats_t = (float2*)(ws + w.stats_t);
    P.stats_d = (float2*)(ws + w.stats_d);
    P.stats_b = (float2*)(ws + w.stats_b);
    P.resid = (ResidTask*)(ws + w.resid);
    P.req = (RequestRec*)(ws + w.req);
    P.wblk = (float*)(ws + w.wblk);
    P.trunc_rows = (TruncRow*)(ws + w.trunc_rows);
    P.trunc_bins = (unsigned int*)(ws + w.trunc_bins);
    P.trunc_flag = (int32_t*)(ws + w.trunc_flag);
    P.retry_rows = (int32_t*)(ws + w.retry_rows);
    P.trunc_z = nullptr;
    P.hist_retry = 0;
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

int dspark_set_wait_poll_limit(unsigned int polls)
{
    const uint32_t v = polls ? polls - 1u : kWaitPollLimit;     // 1: no poll at all, the wait gives up at once
    return cudaMemcpyToSymbol(g_entry_poll_limit, &v, sizeof(v)) == cudaSuccess ? DSPARK_OK : launch_status();
}

int dspark_set_stream_path(int path)
{
    // 0 automatic, 1 direct loads, 2 bulk copies; + 16: every bonus row in the statistics pass (the earlier order)
    const int base = path & 15;
    if (path < 0 || path > 31 || base > 2) return DSPARK_ERR_INVALID_ARG;
    g_stream_path.store(base, std::memory_order_relaxed);
    g_skip_bonus.store((path & 16) ? 0 : 1, std::memory_order_relaxed);
    return DSPARK_OK;
}

// Greedy verification on a scratch region laid out by greedy_workspace_layout (the front of a caller workspace,
// or the built-in array of dspark_verify_greedy_static).
static int greedy_launch(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                         const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                         int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                         void* scratch, size_t scratch_bytes, void* stream)
{
    VerifyParams P;
    int rc = fill_common(P, target_logits, nullptr, dtype, target_row_stride, 0, V, row_offsets, nullptr, draft_tokens, R, n_rows,
                         accepted_len, out_tokens);
    if (rc != DSPARK_OK) return rc;
    const GreedyWorkspace w = greedy_workspace_layout(n_rows, V, P.elem);
    if (!scratch || scratch_bytes < w.total) return DSPARK_ERR_WORKSPACE;
    if (((uintptr_t)scratch & 255u) != 0) return DSPARK_ERR_ALIGNMENT;
    P.counters = (int*)((unsigned char*)scratch + w.counters);
    P.dev_status = dev_status ? dev_status : P.counters + 1;
    P.stats_t = (float2*)((unsigned char*)scratch + w.stats);
    if (!ensure_attrs()) return launch_status();
    cudaStream_t s = (cudaStream_t)stream;
    const bool bulk = g_stream_path.load(std::memory_order_relaxed) != 1 && aligned16(P.target, P.tstride_bytes, P.row_bytes);
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

int dspark_verify_greedy(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                         const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                         int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    // the documented workspace size is that of the sampling verifier; greedy uses the front of it
    if (R >= 1 && n_rows >= R && V >= 1 && workspace && workspace_bytes < workspace_layout(R, n_rows, V).total)
        return DSPARK_ERR_WORKSPACE;
    return greedy_launch(target_logits, dtype, target_row_stride, V, row_offsets, draft_tokens, R, n_rows,
                         accepted_len, out_tokens, dev_status, workspace, workspace_bytes, stream);
}

static int verify_launch(const void* target_logits, const void* draft_logits, int dtype,
                         int64_t target_row_stride, int64_t draft_row_stride, int V,
                         const int32_t* row_offsets, const int64_t* draft_row_start,
                         const int32_t* draft_tokens, int R, int n_rows,
                         float temperature, const float* req_temp, uint64_t seed,
                         int32_t* accepted_len, int32_t* out_tokens,
                         float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream,
                         const int32_t* top_k = nullptr, const float* top_p = nullptr, const float* draft_row_stats = nullptr)
{
    if (!draft_logits) return DSPARK_ERR_INVALID_ARG;
    const bool truncate = top_k || top_p;
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
    P.draft_stats = (const float2*)draft_row_stats;
    cudaStream_t s = (cudaStream_t)stream;
    const int path = g_stream_path.load(std::memory_order_relaxed);
    const bool bulk = path != 1 && aligned16(P.target, P.tstride_bytes, P.row_bytes) &&
                      aligned16(P.draft, P.dstride_bytes, P.row_bytes);
    if (!ensure_attrs()) return launch_status();
    // A rejected request never needs its bonus row: the statistics pass leaves the bonus rows out and the second pass
    // streams them for the requests that accepted every draft token.  (Not with a truncated target, whose threshold
    // search wants the statistics of every target row first, nor on the direct-load path.)
    P.skip_bonus = (bulk && !truncate && g_skip_bonus.load(std::memory_order_relaxed) && R <= kSkipBonusMaxRequests) ? 1 : 0;
    // the request of every draft position rides along in shared memory when it fits beside the offsets (16-bit entries)
    P.req_table = 0;
    if (P.skip_bonus && R <= 65535 && (size_t)((R + 4) / 4) * 16 + (size_t)((n_rows - R + 7) / 8) * 16 <= (size_t)kSkipBonusSmemBytes)
        P.req_table = n_rows - R;
    // with one temperature per request and that table in place, the requests' exponent scales ride along as well, and
    // the kernel that expands the temperatures to rows is not needed
    P.req_scale_smem = 0;
    if (req_temp && P.req_table > 0 &&
        (size_t)((R + 4) / 4) * 16 + (size_t)((P.req_table + 7) / 8) * 16 + (size_t)((R + 3) / 4) * 16 <= (size_t)kSkipBonusSmemBytes)
        P.req_scale_smem = 1;
    if (req_temp && !P.req_scale_smem) {
        KernelTimerScope timer(DSPARK_K_ROW_SCALE, s);
        launch_pdl(row_scale_kernel, dim3((R + 255) / 256), dim3(256), 0, s, P);
    }
    {
        KernelTimerScope timer(DSPARK_K_STREAM, s);
        launch_stream_dtype<kModeStats>(P, bulk, (draft_row_stats ? (long long)n_rows : 2ll * n_rows - R) * pieces(P.nblk), s);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    if (truncate && dtype == DSPARK_F32) {
        // fp32 rows: the threshold of every target row by a descent over its 32-bit patterns (one CTA per row),
        // which also replaces the row's block sums by the sums over the kept set
        float* tau = (float*)((unsigned char*)workspace + workspace_layout(R, n_rows, V).tau);
        KernelTimerScope timer(DSPARK_K_TRUNCATE, s);
        rc = truncate_f32_virtual_launch(P.target, (long long)target_row_stride, V, row_offsets, R, n_rows, top_k, top_p,
                                         temperature, req_temp, tau, P.stats_t, P.nblk, P.epb, s);
        if (rc != DSPARK_OK) return rc;
        P.tau = tau;
    } else if (truncate) {
        // top-k / top-p of the target distribution without touching the rows: one kernel finds the threshold of
        // every target row and replaces the row's block sums by the sums over the kept set; from here on a
        // target logit below the threshold counts as -inf
        float* tau = (float*)((unsigned char*)workspace + workspace_layout(R, n_rows, V).tau);
        KernelTimerScope timer(DSPARK_K_TRUNCATE, s);
        TruncArgs T;
        T.top_k = top_k; T.top_p = top_p; T.temperatures = req_temp; T.temperature = temperature; T.tau = tau;
        P.trunc_z = (double*)((unsigned char*)workspace + workspace_layout(R, n_rows, V).trunc_z);
        launch_pdl(trunc_prep_kernel, dim3((n_rows + 7) / 8), dim3(256), 0, s, P, T);
        launch_stream<2, kModeHist>(P, bulk, (long long)n_rows * pieces(P.nblk), s);
        launch_pdl(trunc_scan_kernel, dim3(n_rows), dim3(kScanThreads), 0, s, P, T, 0);
        // second look at the rows whose nucleus reaches below the first window (flat rows), down to the bound
        P.hist_retry = 1;
        launch_stream<2, kModeHist>(P, bulk, (long long)n_rows * pieces(P.nblk), s);
        P.hist_retry = 0;
        launch_pdl(trunc_scan_kernel, dim3(n_rows), dim3(kScanThreads), 0, s, P, T, 1);
        launch_pdl(trunc_sums_kernel, dim3(R, (P.nblk + 7) / 8), dim3(256), 0, s, P, T);
        // rows whose threshold lies beyond the window (flat rows): the per-row search
        rc = truncate_virtual_launch(P.target, P.tstride_bytes, V, row_offsets, R, n_rows, top_k, top_p, temperature,
                                     req_temp, tau, P.stats_t, P.nblk, P.epb, P.trunc_flag, s);
        if (rc != DSPARK_OK) return rc;
        P.tau = tau;
    }
    {
        KernelTimerScope timer(DSPARK_K_DECIDE, s);
        if (P.draft_stats) launch_pdl(decide_kernel<true>, dim3(R), dim3(kDecideThreads), 0, s, P);
        else launch_pdl(decide_kernel<false>, dim3(R), dim3(kDecideThreads), 0, s, P);
    }
    if ((rc = launch_status()) != DSPARK_OK) return rc;
    {
        KernelTimerScope timer(DSPARK_K_RESIDUAL, s);
        const long long per_task = pieces(P.nblk_r) > pieces(P.nblk) ? pieces(P.nblk_r) : pieces(P.nblk);
        launch_stream_dtype<kModeResid>(P, bulk, (long long)R * per_task, s);
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
static std::atomic<void*> g_static_scratch_ptr[64];

static int static_scratch_address(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return DSPARK_ERR_CUDA; }
    void* ptr = g_static_scratch_ptr[dev].load(std::memory_order_acquire);
    if (!ptr) {
        // two threads making their first call together both look the address up and store the same value
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) {
            fprintf(stderr, "dspark: cudaGetSymbolAddress(static scratch) failed: %s\n", cudaGetErrorString(e));
            cudaGetLastError();
            return DSPARK_ERR_CUDA;
        }
        g_static_scratch_ptr[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return DSPARK_OK;
}

}  // namespace dspark

extern "C" {

size_t dspark_verify_greedy_static_capacity(void) { return kStaticScratchBytes; }

size_t dspark_verify_greedy_static_bytes(int R, int n_rows, int V, int dtype)
{
    if (R < 1 || n_rows < R || V < 1 || (dtype != DSPARK_F32 && dtype != DSPARK_BF16)) return 0;
    return greedy_workspace_layout(n_rows, V, dtype == DSPARK_BF16 ? 2 : 4).total;
}

int dspark_verify_greedy_static(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                                const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                                int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status, void* stream)
{
    if (R < 1 || n_rows < R || V < 1 || (dtype != DSPARK_F32 && dtype != DSPARK_BF16)) return DSPARK_ERR_INVALID_ARG;
    const size_t need = dspark_verify_greedy_static_bytes(R, n_rows, V, dtype);
    if (need > kStaticScratchBytes) {
        fprintf(stderr, "dspark_verify_greedy_static: this batch needs %zu bytes of scratch, the built-in array "
                        "holds %zu; use dspark_verify_greedy with a caller workspace\n", need, kStaticScratchBytes);
        return DSPARK_ERR_STATIC_LIMIT;
    }
    void* scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != DSPARK_OK) return rc;
    // every ticket, counter and statistic the call reads is cleared or rewritten by the call itself, so nothing
    // left in the array by an earlier call matters
    return greedy_launch(target_logits, dtype, target_row_stride, V, row_offsets, draft_tokens, R, n_rows,
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

int dspark_row_stats(const void* logits, int dtype, int64_t row_stride, int V, int n_rows,
                     float temperature, const float* row_temperatures, float* out_row_stats, void* stream)
{
    if (!logits || !out_row_stats || n_rows < 1 || V < 1 || row_stride < V) return DSPARK_ERR_INVALID_ARG;
    if (dtype != DSPARK_F32 && dtype != DSPARK_BF16) return DSPARK_ERR_INVALID_ARG;
    if (!row_temperatures && (!(temperature > 0.0f) || !isfinite(temperature))) return DSPARK_ERR_INVALID_ARG;
    const int elem = dtype == DSPARK_BF16 ? 2 : 4;
    if ((long long)V * elem >= (1ll << 31) || blocks_per_row(V, elem, kStatBlockBytes) > kRowStatsMaxBlocks) return DSPARK_ERR_SHAPE;
    if (((uintptr_t)out_row_stats & 7u) != 0 || ((uintptr_t)logits & (uintptr_t)(elem - 1)) != 0) return DSPARK_ERR_ALIGNMENT;
    cudaStream_t s = (cudaStream_t)stream;
    if (elem == 2)
        launch_pdl(row_stats_kernel<2>, dim3(n_rows), dim3(kRowStatsThreads), 0, s, (const unsigned char*)logits,
                   (long long)row_stride * elem, V, n_rows, temperature, row_temperatures, (float2*)out_row_stats);
    else
        launch_pdl(row_stats_kernel<4>, dim3(n_rows), dim3(kRowStatsThreads), 0, s, (const unsigned char*)logits,
                   (long long)row_stride * elem, V, n_rows, temperature, row_temperatures, (float2*)out_row_stats);
    return launch_status();
}

int dspark_verify_draft_stats(const void* target_logits, const void* draft_logits, int dtype,
                              int64_t target_row_stride, int64_t draft_row_stride, int V,
                              const int32_t* row_offsets, const int64_t* draft_row_start,
                              const int32_t* draft_tokens, const float* draft_row_stats, int R, int n_rows,
                              float temperature, const float* temperatures, uint64_t seed,
                              int32_t* accepted_len, int32_t* out_tokens,
                              float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                              void* workspace, size_t workspace_bytes, void* stream)
{
    if (!draft_row_stats) return DSPARK_ERR_INVALID_ARG;
    if (((uintptr_t)draft_row_stats & 7u) != 0) return DSPARK_ERR_ALIGNMENT;
    return verify_launch(target_logits, draft_logits, dtype, target_row_stride, draft_row_stride, V, row_offsets,
                         draft_row_start, draft_tokens, R, n_rows, temperatures ? 1.0f : temperature, temperatures, seed,
                         accepted_len, out_tokens, out_p_tok, out_q_tok, dev_status, workspace, workspace_bytes, stream,
                         nullptr, nullptr, draft_row_stats);
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
    const bool bulk = g_stream_path.load(std::memory_order_relaxed) != 1 && aligned16(P.target, P.tstride_bytes, P.row_bytes) &&
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
