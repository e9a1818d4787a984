/*
 * dspark.h -- C ABI of the B200 (sm_100a) hot path of DSpark's serving step:
 * the confidence-scheduled verification-length scheduler and the fused
 * ragged-batch speculative verifier.
 *
 * Conventions for every entry point
 *  - "device" pointers are CUDA global-memory addresses on the current device,
 *    "host" pointers are ordinary process memory.  The caller owns every buffer;
 *    the library allocates only inside dspark_profile_create / dspark_ktimer_create.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *    Calls enqueue kernels on it and return; they never synchronise and never read
 *    device data on the host.
 *  - Return value: DSPARK_OK (0) or one of the positive error codes below.  Host-detectable
 *    problems (NULL pointers, non-positive sizes, workspace too small, bad
 *    temperature) return an error and launch nothing.  Problems only visible on the
 *    device (bad offsets, token id outside [0,V), NaN rows, ...) set bits in the
 *    int32 that `dev_status` points to (bits are OR-ed in; the caller zeroes it),
 *    the affected request gets accepted_len = 0 and tokens -1; kernels never trap
 *    and every device-side wait is bounded.
 *  - Logit rows are row-major with unit inner stride; `*_row_stride` is in elements.
 *    The bulk-copy fast path needs 16-byte aligned base pointers, row strides that
 *    are multiples of 16 bytes and V*sizeof(elem) a multiple of 16; anything else
 *    takes a slower element-wise path with identical results.
 */
#ifndef DSPARK_H
#define DSPARK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DSPARK_OK = 0,
    DSPARK_ERR_INVALID_ARG = 1,
    DSPARK_ERR_SHAPE = 2,
    DSPARK_ERR_ALIGNMENT = 3,
    DSPARK_ERR_WORKSPACE = 4,
    DSPARK_ERR_CUDA = 5,
    /* 6 is not used: no call waits for the device, so a device-side wait that runs out can only be
     * reported through DSPARK_DEV_TIMEOUT in *dev_status */
    DSPARK_ERR_STATIC_LIMIT = 7
} dspark_status_t;

typedef enum { DSPARK_F32 = 0, DSPARK_BF16 = 1 } dspark_dtype_t;

typedef enum {
    DSPARK_SCHED_EARLY_STOP = 0, /* Algorithm 1 as printed: stop at the first non-improving admission */
    DSPARK_SCHED_GLOBAL = 1,     /* Section 5.2, scheduler in practice: same path without the break, first maximiser wins */
    DSPARK_SCHED_TOPK = 2        /* Section 5.2: admit the K most confident candidates (K from the caller) */
} dspark_sched_mode_t;

/* Bits OR-ed into *dev_status (verifier) and into dspark_sched_info_t.status (scheduler). */
#define DSPARK_DEV_BAD_OFFSETS 1   /* row_offsets not increasing by >= 1, or beyond the n_rows capacity */
#define DSPARK_DEV_BAD_TOKEN 2     /* a draft token id outside [0, V) */
#define DSPARK_DEV_BAD_ROW 4       /* a logit row with NaN, +inf, or no finite element */
#define DSPARK_DEV_TIMEOUT 8       /* a bounded device-side wait ran out */
#define DSPARK_DEV_CONF_CLAMPED 16 /* a confidence was NaN, negative or above 1 (read as 0, 0, 1) */
#define DSPARK_DEV_BUDGET_LT_R 32  /* token budget below the number of requests: every l*_r = 0 */
#define DSPARK_DEV_ALL_NEG_INF 64  /* greedy: a row without any element above -inf (index 0 reported) */
#define DSPARK_DEV_BAD_TEMPERATURE 128 /* a per-request temperature that is not a positive finite number */

/* ------------------------------------------------------------------------------------
 * Engine throughput profile SPS(B), steps per second at B batch tokens: a table the engine measures
 * once when it starts up and only looks up afterwards (Section 3.2.2).
 *
 * bp_tokens / bp_sps: host arrays of n_bp breakpoints, bp_tokens strictly increasing.
 * The library builds a dense fp64 device table SPS[0..max_tokens]: piecewise linear
 * between breakpoints, constant outside them (a step-wise curve is expressed by passing
 * every B as a breakpoint).  Lookups beyond max_tokens use the last entry.
 * Allocates device memory (cudaMalloc) and synchronises; call it at start-up.
 * Errors: INVALID_ARG (NULL, n_bp < 1, max_tokens < 1, non-increasing tokens), CUDA.
 */
typedef struct dspark_profile dspark_profile_t;
int dspark_profile_create(const int32_t* bp_tokens, const double* bp_sps, int n_bp,
                          int max_tokens, dspark_profile_t** out);
int dspark_profile_destroy(dspark_profile_t* prof);
/* Device pointer to the fp64 table (max_tokens + 1 entries); owned by the profile. */
const double* dspark_profile_table(const dspark_profile_t* prof, int* max_tokens);

/* What the scheduler reports besides the lengths (device struct, 32 bytes). */
typedef struct {
    int32_t B;            /* batch tokens R + sum_r l*_r                         */
    int32_t n_admitted;   /* admitted candidates i*                               */
    int32_t status;       /* DSPARK_DEV_* warning bits                            */
    int32_t n_candidates; /* |E|, candidates with positive survival probability   */
    double tau;           /* expected accepted tokens R + sum of admitted a_{r,j} */
    double theta;         /* tau * SPS(B), the objective reached                  */
} dspark_sched_info_t;

/* ------------------------------------------------------------------------------------
 * dspark_schedule -- hardware-aware prefix scheduler (Algorithm 1; a, B, tau, Theta as
 * defined in Section 3.2.2; no-break and top-K variants and the capacity limit from
 * Section 5.2, "Hardware-Aware Prefix Scheduler in Practice").
 *
 * Computes survival products a_{r,j} = prod_{i<=j} c_{r,i} (fp32, left to right), orders
 * all candidates with a > 0 by (a descending, position ascending, request ascending),
 * walks the admission path i = 1..min(|E|, budget_tokens - R) with
 *     tau_i = R + sum of the first i survival values (exact, in units of 2^-40),
 *     Theta_i = tau_i * SPS(R + i)   (one fp64 multiply),
 * and stops per `mode`.  l*_r = number of admitted candidates of request r.
 *
 *  conf            device [R, gamma] fp32, row-major, c in [0,1] (NaN/<0 -> 0, >1 -> 1 with a warning bit)
 *  draft_len       device [R] int32 or NULL: positions >= draft_len[r] are not candidates (NULL: gamma)
 *  budget_tokens   cap on batch tokens B = R + sum l_r
 *  topk_K          only for DSPARK_SCHED_TOPK
 *  out_len         device [R] int32: l*_r
 *  out_row_offsets device [R+1] int32 or NULL: exclusive scan of (l*_r + 1), the verifier's row_offsets
 *  out_survival    device [R, gamma] fp32 or NULL: a_{r,j} (0 where not a candidate)
 *  out_expected_len device [R] fp32 or NULL: 1 + sum_{j < l*_r} a_{r,j}
 *  out_info        device dspark_sched_info_t or NULL
 *  workspace       device scratch of at least dspark_schedule_workspace_bytes(R, gamma) bytes, 16-byte aligned
 *
 * Limits: 1 <= R <= 2^20, 0 <= gamma <= 4096, R*gamma <= 2^20.
 * Errors: INVALID_ARG, SHAPE (limits), WORKSPACE, CUDA (launch failure).
 */
size_t dspark_schedule_workspace_bytes(int R, int gamma);
int dspark_schedule(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                    int R, int gamma, int budget_tokens, int mode, int topk_K,
                    int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                    float* out_expected_len, dspark_sched_info_t* out_info,
                    void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * dspark_schedule_async -- the scheduler as deployed (Section 5.2): the engine must know the
 * batch size of the next step before the current one ends, so the capacity K (how many draft
 * tokens are admitted in total) is taken from the unconstrained, no-break search over the
 * confidences of TWO STEPS EARLIER, while the candidates themselves are ranked by their current
 * survival products (a dynamic top-K, still under the token budget).
 *
 * state: device int32[4], owned by the caller and kept between steps: {step t, K slot 0,
 * K slot 1, reserved}.  Each call reads the K stored by step t-2 (slot t mod 2), admits that many
 * of the most confident current candidates, overwrites the slot with the admission count of the
 * global search on the CURRENT confidences (to be used at step t+2) and increments t -- all on the
 * device, so a captured CUDA graph of schedule -> verify can simply be replayed step after step.
 * dspark_async_state_init sets t = 0 and both slots to initial_K (used by the first two steps).
 * All other arguments, outputs, limits and errors are those of dspark_schedule.
 */
int dspark_async_state_init(int32_t* state, int initial_K, void* stream);
int dspark_schedule_async(const dspark_profile_t* prof, const float* conf, const int32_t* draft_len,
                          int R, int gamma, int budget_tokens, int32_t* state,
                          int32_t* out_len, int32_t* out_row_offsets, float* out_survival,
                          float* out_expected_len, dspark_sched_info_t* out_info,
                          void* workspace, size_t workspace_bytes, void* stream);

/* row_offsets[0..R] = exclusive scan of (lengths[r] + 1): the flat ragged layout of
 * Section 5.3, "High-Throughput and Low-Latency Inference" (all verified tokens of all requests flattened).
 * Device in, device out. */
int dspark_build_offsets(const int32_t* lengths, int R, int32_t* row_offsets, void* stream);

/* ------------------------------------------------------------------------------------
 * Ragged verification batch (both verifiers).
 *  R requests; request r owns target rows [row_offsets[r], row_offsets[r+1]): l_r draft
 *  positions followed by one bonus row, so row_offsets[r+1] - row_offsets[r] = l_r + 1 >= 1.
 *  n_rows is the host-known CAPACITY of the flat arrays (target rows, draft_tokens,
 *  out_tokens, out_p_tok, out_q_tok); the true row count is row_offsets[R] on the device
 *  and must not exceed it.  draft_tokens[row_offsets[r] + j] is the token proposed at
 *  position j < l_r (the bonus-row entry is ignored).
 * Outputs: accepted_len[r] = n_r, the number of accepted draft tokens;
 *  out_tokens[row_offsets[r] + i] = draft token for i < n_r, the corrected / bonus token
 *  at i = n_r, -1 for i > n_r.  The request emits n_r + 1 tokens.
 */
size_t dspark_verify_workspace_bytes(int R, int n_rows, int V);

/* dspark_verify_greedy -- a draft token is accepted iff it equals the argmax of its
 * target row (lowest index on ties; NaN never wins; -0.0 ties +0.0); the first mismatch
 * ends the prefix (Section 2.1: the first rejection discards all later tokens) and the
 * argmax of that row is emitted; if every token matched, the argmax of the bonus row.
 * target_logits: device [n_rows, V] of `dtype`.  One pass over the rows, no exponentials.
 */
int dspark_verify_greedy(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                         const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                         int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream);

/* dspark_verify_greedy_static -- the same greedy verification for callers that are not
 * allowed to allocate device memory.  (The paper has no counterpart; this is a packaging
 * variant of dspark_verify_greedy.)
 *
 * Who needs it: a serving engine once it has entered its steady-state loop usually cannot call
 * cudaMalloc any more -- every byte of HBM is already promised to weights and KV cache, an
 * allocation would synchronise the whole device in the middle of a step, and code that runs as
 * a plug-in of another runtime may simply be forbidden to allocate after start-up.  Such a
 * caller has nowhere to get a workspace from, so this entry point takes none: the per-block
 * (max, argmax) statistics go into a fixed array of DSPARK_STATIC_SCRATCH_BYTES that is part
 * of the library image.  Every GPU that loads the library carries that array until the
 * process exits, whether or not this function is ever called.
 *
 * Arguments, outputs and device-side error reporting are those of dspark_verify_greedy, minus
 * the workspace.  Differences a caller has to know:
 *  - Size limit.  The array has to hold what greedy verification itself uses: 256 bytes plus 8 bytes per
 *    4 KB block of every target row (dspark_verify_greedy_static_bytes(R, n_rows, V, dtype) gives the exact
 *    figure).  A batch that needs more than dspark_verify_greedy_static_capacity() is refused with
 *    DSPARK_ERR_STATIC_LIMIT and a message on stderr; nothing is launched.  8 MiB covers 8 256 fp32 rows
 *    or 16 383 bf16 rows at V = 129 280.
 *  - First call on a device.  It looks up the device address of the array
 *    (cudaGetSymbolAddress) with that device current and caches it; later calls on that
 *    device do no set-up.  Make that first call during initialisation, before any stream
 *    capture begins.  On every call the device that owns `stream` must be the current device:
 *    the array that is used is the current device's copy.
 *  - One array for everybody.  All calls in the process, on every stream, share it, and it keeps
 *    whatever the previous call left.  That is harmless for results (each call rewrites every
 *    entry it later reads), but two calls that overlap in time on the GPU race on it: run them
 *    on one stream, or order them yourself.
 *  - It calls no cudaMalloc, cudaFree or other allocating routine.
 */
#define DSPARK_STATIC_SCRATCH_BYTES (8u << 20)
size_t dspark_verify_greedy_static_capacity(void);
size_t dspark_verify_greedy_static_bytes(int R, int n_rows, int V, int dtype);
int dspark_verify_greedy_static(const void* target_logits, int dtype, int64_t target_row_stride, int V,
                                const int32_t* row_offsets, const int32_t* draft_tokens, int R, int n_rows,
                                int32_t* accepted_len, int32_t* out_tokens, int32_t* dev_status,
                                void* stream);

/* dspark_verify -- lossless sampling verification (Section 2.1): with p = softmax(target/T)
 * and q = softmax(draft/T) at each position, token x is accepted with probability
 * min(1, p(x)/q(x)), tested as  u * q(x) < p(x)  with u in [0,1) from Philox4x32-10 keyed by
 * `seed` at counter (position, 0, request, 0), word 0.  Left to right; at the first rejection
 * the emitted token is drawn from norm(max(0, p - q)) of that position, otherwise the bonus
 * token is drawn from p of the last row (Section 1: longest accepted prefix plus one bonus
 * token); both draws invert the CDF in vocabulary order with u' = word 1 of the same counter
 * (position n_r): the smallest v whose running sum exceeds u' times the total.
 *
 *  draft_logits     device rows of `dtype`, same V.  draft_row_start == NULL: compact layout,
 *                   the draft row of (r, j) is row_offsets[r] - r + j (needs n_rows - R rows of
 *                   capacity).  Otherwise device [R] int64: the row of (r, j) is
 *                   draft_row_start[r] + j (e.g. r * gamma for the drafter's full blocks).
 *  temperature      T > 0, applied to both distributions.
 *  out_p_tok/out_q_tok  device [n_rows] fp32 or NULL: p(x), q(x) at every draft position
 *                   (bonus-row entries are not written).  When NULL, positions after the first
 *                   rejection are not evaluated.
 * Device-side errors void one request (accepted_len 0, its tokens -1) and set a bit of *dev_status; the
 * others are unaffected.  DSPARK_DEV_BAD_TOKEN: any draft token of the request outside [0, V).
 * DSPARK_DEV_BAD_ROW: an unusable row (NaN, +inf, no finite element) among the rows that decide the output,
 * i.e. the target and draft rows of the positions up to the first rejection and the row the emitted token is
 * drawn from; with out_p_tok / out_q_tok every draft position is evaluated and an unusable row at any of them
 * voids the request.  A request reports every bit that applies to it.  Logits must be small enough for
 * x * log2(e) / T to stay finite in fp32 (|x| / T below about 2e38); larger finite values count as infinite.
 * Streams the target and draft row of every draft position once (online softmax statistics per 4 KB block),
 * then in a second pass re-reads the rejected position's row pair of each rejected request and reads the bonus row
 * of each request that accepted every draft token (the bonus row of a rejected request is never needed and never
 * read; with a truncated target, direct loads or more than 2 048 requests all bonus rows go through the first pass).
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, CUDA.
 */
int dspark_verify(const void* target_logits, const void* draft_logits, int dtype,
                  int64_t target_row_stride, int64_t draft_row_stride, int V,
                  const int32_t* row_offsets, const int64_t* draft_row_start,
                  const int32_t* draft_tokens, int R, int n_rows,
                  float temperature, uint64_t seed,
                  int32_t* accepted_len, int32_t* out_tokens,
                  float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                  void* workspace, size_t workspace_bytes, void* stream);

/* dspark_verify_per_request -- dspark_verify with one temperature per request (a serving batch
 * mixes requests with different sampling settings): temperatures is a device array [R], request
 * r uses p = softmax(target / T_r), q = softmax(draft / T_r).  A temperature that is not a
 * positive finite number sets DSPARK_DEV_BAD_TEMPERATURE and voids that request only.
 * The statistics pass takes each unit's exponent scale from its request (on very large batches, and with a truncated
 * target, one extra tiny kernel expands T_r to the rows first); everything else is dspark_verify.
 */
int dspark_verify_per_request(const void* target_logits, const void* draft_logits, int dtype,
                              int64_t target_row_stride, int64_t draft_row_stride, int V,
                              const int32_t* row_offsets, const int64_t* draft_row_start,
                              const int32_t* draft_tokens, int R, int n_rows,
                              const float* temperatures, uint64_t seed,
                              int32_t* accepted_len, int32_t* out_tokens,
                              float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                              void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * dspark_accept_rate -- the analytical per-step acceptance rate of every draft position,
 *     c*_{r,j} = 1 - 1/2 * || p^d_{r,j} - p^t_{r,j} ||_1          (Section 3.2.1, Eq. accept_rate),
 * which the paper uses as the training label of the confidence head; with it an engine can also
 * watch the calibration of its confidences on live batches.  p = softmax(target/T),
 * q = softmax(draft/T); same ragged batch layout as the verifiers.
 *  out_cstar  device [n_rows] fp32: entry row_offsets[r] + j for j < l_r; bonus-row entries and
 *             positions with an unusable row (NaN, +inf, no finite element; BAD_ROW is set) are NaN.
 * Reads every target and draft row once for the softmax statistics and the row pairs of all
 * draft positions a second time (2 x the bytes of dspark_verify's first pass).
 * workspace: dspark_accept_rate_workspace_bytes(R, n_rows, V), 256-byte aligned.
 * Errors: INVALID_ARG, SHAPE, WORKSPACE, CUDA.
 */
size_t dspark_accept_rate_workspace_bytes(int R, int n_rows, int V);
int dspark_accept_rate(const void* target_logits, const void* draft_logits, int dtype,
                       int64_t target_row_stride, int64_t draft_row_stride, int V,
                       const int32_t* row_offsets, const int64_t* draft_row_start, int R, int n_rows,
                       float temperature, float* out_cstar, int32_t* dev_status,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * The Markov-head sequential draft step (Section 3.1, Eq. sequential-factorization and Eq. markov;
 * confidence head: Section 3.2.1, Eq. confidence).  For block position k and every request r,
 *     logits[r, :] = U[r, :] + W1[x_prev[r]] W2,   W1 in R^{V x 256}, W2 in R^{256 x V}  (rank 256),
 *     x[r] ~ softmax(logits[r, :] / T),
 *     conf[r] = sigmoid(w^T [ H[r, :] ; W1[x_prev[r]] ]).
 * The bias product runs on the tensor cores (bf16 operands, fp32 accumulation over the 256 terms);
 * base logits are added in fp32 and the sum is rounded once to bf16 (round to nearest even): the
 * stored logits are what the draw uses and what a verifier later reads as the draft distribution.
 *
 * dspark_markov_pack_w2: one-time re-layout of W2 (device, bf16, row-major [256, V]) into the
 *   tile order the contraction reads (device, dspark_markov_w2_packed_bytes(V), 16-byte aligned;
 *   columns past V are zero).  The caller owns both buffers.  Done once when the weights are loaded:
 *   the call synchronises `stream` and returns after the re-layout has completed (the contraction
 *   prefetches the packed weights ahead of its stream dependencies, so they must never be in flight
 *   while a draft step is enqueued; not capturable in a CUDA graph).
 * dspark_markov_logits:
 *   U            device bf16 [R, >= V], row stride u_row_stride elements: base logits of position k
 *   W1           device bf16 [V, 256] row-major, 32-byte aligned
 *   W2_packed    output of dspark_markov_pack_w2
 *   x_prev       device int32 [R]: previous token of each request (anchor token at k = 1); a value
 *                outside [0, V) sets DSPARK_DEV_BAD_TOKEN and contributes a zero embedding
 *   H, w_conf    device bf16 [R, >= d] (stride h_row_stride) and device fp32 [d + 256]; read only
 *                when out_conf is non-NULL.  The d + 256 products are accumulated in fp32 (error far
 *                below 1e-6 on the confidence).
 *   out_logits   device bf16 [R, >= V], row stride out_row_stride elements
 *   out_conf     device fp32 [R] or NULL
 *   workspace    dspark_markov_workspace_bytes(R, V), 256-byte aligned
 * dspark_markov_draft_step: dspark_markov_logits, then one draw per request with the rule of the
 *   verifier's bonus draw for a request with no draft position: temperature > 0 inverts the CDF of
 *   softmax(stored logits / T) in vocabulary order with the second uniform of (seed, request r,
 *   position 0); temperature == 0 takes the argmax (lowest index on ties, NaN never wins; a row with
 *   nothing above -inf sets DSPARK_DEV_ALL_NEG_INF and yields 0).  The softmax statistics are taken
 *   per 128-column tile inside the contraction's epilogue, so the logits are not read a second time.
 *   A row with NaN, +inf or no finite element sets DSPARK_DEV_BAD_ROW and yields -1.
 *   out_tokens device int32 [R].
 * Resources: the contraction runs one CTA per SM with 225 KB of shared memory and allocates all 512
 * tensor-memory columns of the SM for its lifetime; a concurrent kernel that needs tensor memory waits.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, CUDA; SHAPE from dspark_markov_draft_step when V exceeds
 * 524 288 (the draw keeps one statistics entry per 128 columns in registers); a device wait that ran out
 * sets DSPARK_DEV_TIMEOUT in *dev_status and the affected logits are unspecified.
 */
/* Diagnostic switch for the epilogue of dspark_markov_logits: 0 = automatic (base logits and draft
 * logits move through 2-D tensor-map copies when both base addresses are 16-byte aligned and both
 * row pitches are multiples of 16 bytes, direct loads and stores otherwise), 1 = always direct.
 * Same results either way.  Process-wide; the paper has no counterpart. */
int dspark_markov_set_epilogue_path(int path);
size_t dspark_markov_w2_packed_bytes(int V);
int dspark_markov_pack_w2(const void* W2, int V, void* W2_packed, void* stream);
size_t dspark_markov_workspace_bytes(int R, int V);
int dspark_markov_logits(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                         const int32_t* x_prev, int R, int V,
                         const void* H, int64_t h_row_stride, int d, const float* w_conf,
                         void* out_logits, int64_t out_row_stride, float* out_conf, int32_t* dev_status,
                         void* workspace, size_t workspace_bytes, void* stream);
int dspark_markov_draft_step(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                             const int32_t* x_prev, int R, int V,
                             const void* H, int64_t h_row_stride, int d, const float* w_conf,
                             float temperature, uint64_t seed,
                             void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                             int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream);

/* dspark_verify_draft_stats -- dspark_verify / dspark_verify_per_request for a caller whose drafter kept the softmax
 * statistics of the draft rows it wrote (Section 2.1: the accept test needs q(x) = 2^(x_d * s - c_q) / Z_q, i.e. of a
 * draft row only its logit at the draft token and the row's reference and sum).  The statistics pass then streams the
 * target rows alone: on a batch with as many draft rows as cfg3 a third fewer bytes.  The draft rows themselves are
 * still read where they are needed: one logit per position, and the whole row of a rejected position.
 *   draft_row_stats   device fp32 [n_draft_rows_physical][2], 8-byte aligned, indexed like the rows of draft_logits
 *                     (draft_row_start[r] + j, or the compact index): (c, Z) with s = log2(e) / T of the row's request,
 *                     c = max(x) * s and Z = sum 2^(x * s - c) -- what dspark_markov_draft_step_stats and
 *                     dspark_row_stats write.  A row whose entry is not a usable pair (NaN, Z <= 0) counts as a row
 *                     that cannot be normalised (DSPARK_DEV_BAD_ROW for a request that looks at it).
 *   temperature / temperatures   one T > 0, or device fp32 [R] (then `temperature` is ignored); the statistics must have
 *                     been computed with the same temperatures
 * Everything else as dspark_verify.  Losslessness rests on the statistics being those of the stored draft logits.
 */
int dspark_verify_draft_stats(const void* target_logits, const void* draft_logits, int dtype,
                              int64_t target_row_stride, int64_t draft_row_stride, int V,
                              const int32_t* row_offsets, const int64_t* draft_row_start,
                              const int32_t* draft_tokens, const float* draft_row_stats, int R, int n_rows,
                              float temperature, const float* temperatures, uint64_t seed,
                              int32_t* accepted_len, int32_t* out_tokens,
                              float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                              void* workspace, size_t workspace_bytes, void* stream);

/* dspark_row_stats -- the (c, Z) pair of dspark_verify_draft_stats for every row of a logit matrix, for a producer
 * that has no statistics of its own: same blocks, block arithmetic and order of combination as the verifier, so the
 * pair is what the verifier would have computed (Z rounded to fp32).  One read of the rows.
 *   logits            device fp32 / bf16 [n_rows, >= V], row stride in elements
 *   temperature / row_temperatures   one T > 0, or device fp32 [n_rows] (one per ROW; a value that is not positive and
 *                     finite gives (NaN, NaN))
 *   out_row_stats     device fp32 [n_rows][2], 8-byte aligned
 * Errors: INVALID_ARG, SHAPE (more than 2 048 blocks of 4 KB per row), ALIGNMENT, CUDA.
 */
int dspark_row_stats(const void* logits, int dtype, int64_t row_stride, int V, int n_rows,
                     float temperature, const float* row_temperatures, float* out_row_stats, void* stream);

/* dspark_markov_draft_step_stats -- dspark_markov_draft_step that also hands out, per request, the statistics of the
 * draft logits it has just written and drawn from (temperature > 0 only): out_row_stats[r * row_stats_stride] = (c, Z)
 * as dspark_verify_draft_stats reads them (device fp32 pairs, 8-byte aligned; the stride, in pairs, lets position k of
 * a block layout [R, block, V] write entry r * block + k).  They are by-products of the draw: nothing is read again.
 */
int dspark_markov_draft_step_stats(const void* U, int64_t u_row_stride, const void* W1, const void* W2_packed,
                                   const int32_t* x_prev, int R, int V,
                                   const void* H, int64_t h_row_stride, int d, const float* w_conf,
                                   float temperature, uint64_t seed,
                                   void* out_logits, int64_t out_row_stride, int32_t* out_tokens, float* out_conf,
                                   float* out_row_stats, int64_t row_stats_stride,
                                   int32_t* dev_status, void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * dspark_truncate_target -- top-k / top-p truncation of the target distribution, per request (Section 4.1
 * evaluates every model with its own suggested sampling settings; the paper states no rule of its own).
 * The logits of the excluded tokens of every target row are set to -inf IN PLACE, so that softmax
 * renormalises over the kept set and dspark_verify / dspark_verify_per_request, run afterwards on the same
 * rows, are lossless with respect to the truncated target distribution.
 *   kept set S = { v : x_v >= tau } (a value cut: every token tied with the threshold value is kept);
 *   top-k first: tau_k = k-th largest logit of the row (top_k[r] <= 0 or >= V: off); then top-p on the
 *   distribution renormalised over the top-k set: walking the distinct values downwards, tau_p is the first
 *   value at which the cumulative mass reaches top_p[r] * Z_k (top_p >= 1: off; <= 0: only the maximum);
 *   tau = max(tau_k, tau_p).  p = softmax(row / T_r).
 *  target_logits   device bf16 or fp32 [n_rows, >= V], modified in place.  bf16: the threshold is found exactly on
 *                  a histogram of the 16-bit keys.  fp32: by a descent over the 32-bit patterns (a histogram
 *                  linear in the distance to the row maximum, then 11 bits of the key at a time), masses summed
 *                  as integers so that the result does not change from run to run; several times slower per row
 *  row_offsets, R, n_rows   the ragged batch of the verifiers; every row of request r uses r's parameters
 *  top_k           device int32 [R] or NULL;  top_p  device fp32 [R] or NULL (both NULL: nothing to do)
 *  temperature / temperatures   one T > 0, or device fp32 [R] (a T that is not positive and finite leaves
 *                  that request's rows alone)
 *  out_tau         device fp32 [n_rows] or NULL: threshold value of each row (-inf: untouched)
 *  out_kept        device int32 [n_rows] or NULL: size of the kept set (V: untouched)
 * A row with NaN, +inf or no finite element is left as it is (the verifier reports it).  Costs one read of
 * the row from HBM, two from L2 and one write (fp32: four to six reads).  No workspace.  Errors: INVALID_ARG, CUDA.
 */
int dspark_truncate_target(void* target_logits, int dtype, int64_t target_row_stride, int V,
                           const int32_t* row_offsets, int R, int n_rows,
                           const int32_t* top_k, const float* top_p, float temperature, const float* temperatures,
                           float* out_tau, int32_t* out_kept, int32_t* dev_status, void* stream);

/* dspark_verify_truncated -- dspark_verify / dspark_verify_per_request on the top-k / top-p truncated target
 * distribution of dspark_truncate_target, without modifying the target rows: after the statistics pass the
 * threshold tau of every target row is found (same rule, exact on the 16-bit keys: one more streamed pass counts the
 * keys next to the row maximum, a row that this does not resolve is counted once more over a deeper window, and what
 * is left goes through the per-row search of dspark_truncate_target) together with the mass of the kept set; the
 * accept test, the residual pass and the final draws then treat a target logit below tau as -inf.  The draft
 * distribution q is used as given.  Costs one extra read of the target rows instead of the read + write of
 * dspark_truncate_target.  temperatures / top_k / top_p: device [R] or NULL (temperatures NULL: the scalar
 * `temperature`; top_k and top_p both NULL: plain dspark_verify).  out_p_tok reports the truncated p(x).
 * fp32 rows: the threshold of every target row comes from the per-row descent of dspark_truncate_target (no
 * streamed search), the rest is the same.  Same workspace as dspark_verify.
 */
int dspark_verify_truncated(const void* target_logits, const void* draft_logits, int dtype,
                            int64_t target_row_stride, int64_t draft_row_stride, int V,
                            const int32_t* row_offsets, const int64_t* draft_row_start,
                            const int32_t* draft_tokens, int R, int n_rows,
                            float temperature, const float* temperatures, const int32_t* top_k, const float* top_p,
                            uint64_t seed, int32_t* accepted_len, int32_t* out_tokens,
                            float* out_p_tok, float* out_q_tok, int32_t* dev_status,
                            void* workspace, size_t workspace_bytes, void* stream);

/* ------------------------------------------------------------------------------------
 * Sequential Temperature Scaling of the confidence head (Section 3.2.1, "Post-hoc Calibration").
 * From left to right, position k receives the temperature T_k of a caller-given grid that minimises
 * the Expected Calibration Error of the cumulative product a_{n,k} = prod_{i<=k} sigmoid(logit(c_{n,i}) / T_i)
 * over N held-out draft blocks, T_1..T_{k-1} already fixed:
 *     ECE_k = (1/N_k) sum_b | sum_{n in b} y_{n,k} - sum_{n in b} a_{n,k} |,  b = min(n_bins-1, floor(a n_bins)),
 * y_{n,k} = 1 iff accepted_len[n] > k; block n counts at position k iff k < verified_len[n].
 *  conf          device fp32 [N, gamma]: raw confidences of the head; a value outside (0,1) is clamped to
 *                [0,1] (NaN -> 0) and never rescaled
 *  accepted_len  device int32 [N]: accepted draft tokens of the block (what the verifier returned)
 *  verified_len  device int32 [N] or NULL (= gamma): how many positions of the block were verified
 *  grid          device fp32 [G]: candidate temperatures; a point that is not a positive finite number is
 *                never chosen and gets NaN in out_ece_grid (if none is usable the position keeps T = 1);
 *                ties take the first grid point
 *  n_bins        1..64 equal-width bins
 *  out_T         device fp32 [gamma]; a position nobody verified gets 1
 *  out_ece_before / out_ece_after  device fp64 [gamma] or NULL: ECE of the raw and of the calibrated chain
 *  out_ece_grid  device fp64 [gamma, G] or NULL: ECE of every candidate
 * The products are fp32, per-bin sums of a are exact integers (a * 2^32 truncated), the ECE is fp64.
 * dspark_sts_apply writes sigmoid(logit(c) / T_k) for every entry: the confidences to hand to
 * dspark_schedule.  Temperature scaling keeps the order of the confidences of a position.
 * workspace: dspark_sts_workspace_bytes(N, gamma, G, n_bins), 256-byte aligned.
 * Errors: INVALID_ARG, SHAPE (n_bins > 64), WORKSPACE, ALIGNMENT, CUDA.
 */
size_t dspark_sts_workspace_bytes(int N, int gamma, int G, int n_bins);
int dspark_sts_calibrate(const float* conf, int N, int gamma, const int32_t* accepted_len, const int32_t* verified_len,
                         const float* grid, int G, int n_bins, float* out_T, double* out_ece_before,
                         double* out_ece_after, double* out_ece_grid, void* workspace, size_t workspace_bytes, void* stream);
int dspark_sts_apply(const float* conf, int N, int gamma, const float* T, float* out, void* stream);

/* The two uniforms of (seed, request, position) exactly as the verifier draws them
 * (host computation; for tests and for replaying a step). */
void dspark_uniforms(uint64_t seed, uint32_t request, uint32_t position,
                     float* u_accept, float* u_resample);

/* ------------------------------------------------------------------------------------
 * Per-kernel device timing (measurement aid; the paper has no counterpart).
 * While a timer is attached, every kernel the library launches is bracketed by a pair
 * of CUDA events on the caller's stream; dspark_ktimer_read synchronises on them and
 * returns, for one kernel id, the summed milliseconds and the number of launches.
 * Not thread-safe; attach NULL to detach.  Launches beyond `capacity` are not recorded.
 */
typedef struct dspark_ktimer dspark_ktimer_t;
enum {
    DSPARK_K_SCHEDULE = 0, DSPARK_K_OFFSETS = 1, DSPARK_K_STREAM = 2, DSPARK_K_DECIDE = 3,
    DSPARK_K_RESIDUAL = 4, DSPARK_K_FINALIZE = 5, DSPARK_K_GREEDY_STREAM = 6, DSPARK_K_GREEDY_DECIDE = 7,
    DSPARK_K_ROW_SCALE = 8, DSPARK_K_MARKOV_GEMM = 9, DSPARK_K_MARKOV_DRAW = 10, DSPARK_K_TRUNCATE = 11,
    DSPARK_K_COUNT = 12
};
int dspark_ktimer_create(int capacity, dspark_ktimer_t** out);
int dspark_ktimer_destroy(dspark_ktimer_t* t);
int dspark_ktimer_attach(dspark_ktimer_t* t);
int dspark_ktimer_reset(dspark_ktimer_t* t);
int dspark_ktimer_read(dspark_ktimer_t* t, int kernel_id, float* total_ms, int* launches);

/* Diagnostic switch for the verifiers: 0 = automatic (the bulk-copy pipeline when the 16-byte rules hold,
 * direct loads otherwise), 1 = always direct loads, 2 = bulk copies; add 16 to stream every bonus row in the
 * statistics pass instead of only the needed ones in the second pass (the earlier order).  Results are the same
 * (direct loads: up to fp32 summation order).  Process-wide (atomics); the paper has no counterpart. */
int dspark_set_stream_path(int path);

/* Diagnostic: how many polls the streamed passes of the verifiers spend on an entry wait (a consumer warp
 * waiting for its data, the producer waiting for a free stage or for the launch tag) before they give up,
 * set DSPARK_DEV_TIMEOUT in *dev_status and leave.  0 restores the default (about 4 million polls, on the
 * order of a second); a wait gives up after polls - 1 unsuccessful polls, so 1 makes every such wait run
 * out at once.  That is how the tests reach the give-up path without hanging anything: a kernel that gives
 * up still waits, with the long default bound, for the bulk copies it has already issued before it leaves,
 * and its outputs are unspecified.  Per device (the current one), synchronous; the paper has no counterpart. */
int dspark_set_wait_poll_limit(unsigned int polls);

const char* dspark_status_string(int status);
const char* dspark_kernel_name(int kernel_id);
int dspark_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DSPARK_H */
