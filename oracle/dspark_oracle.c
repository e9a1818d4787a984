/*
 * DSpark CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, sequential restatement of what the scheduler and the
 * speculative verifier compute, in fp64 (except where noted), written from
 * the paper's definitions.  Only tests, the smoke check and the benchmark's
 * cpu_baseline / reference legs may call it.  It shares no code, header,
 * table or constant generator with the CUDA library; the handful of enum
 * values it repeats (dtype, mode, status bits) are the public API contract.
 *
 * Every function names the passage of the paper it follows.  Where the paper
 * is silent the reading taken is stated next to the code.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC -pthread
 * (no contraction: products and sums round exactly as written).
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORC_F32 0
#define ORC_BF16 1

#define ORC_MODE_EARLY_STOP 0
#define ORC_MODE_GLOBAL 1
#define ORC_MODE_TOPK 2

/* status bits (per request in the verifier, global in the scheduler) */
#define ORC_ST_BAD_OFFSETS 1
#define ORC_ST_BAD_TOKEN 2
#define ORC_ST_BAD_ROW 4
#define ORC_ST_CONF_CLAMPED 16
#define ORC_ST_BUDGET_LT_R 32
#define ORC_ST_ALL_NEG_INF 64
#define ORC_ST_BAD_TEMPERATURE 128

/* ------------------------------------------------------------------------ */
/* Counter-based RNG.  The paper never names a generator; the reading taken  */
/* is Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of       */
/*   (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)) */
/* with the key bumped by the Weyl constants between rounds.                 */
/* ------------------------------------------------------------------------ */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * The two uniforms of (seed, request r, position j): counter (j, 0, r, 0),
 * key (seed low word, seed high word); word 0 drives the accept test, word 1
 * the residual / bonus draw.  u = (word >> 8) * 2^-24 lies in [0,1) and is
 * exact in fp32.
 */
void orc_uniforms(uint64_t seed, uint32_t r, uint32_t j, float* u_accept, float* u_resample)
{
    uint32_t ctr[4] = { j, 0u, r, 0u };
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    uint32_t w[4];
    orc_philox4x32_10(ctr, key, w);
    *u_accept = (float)(w[0] >> 8) * (1.0f / 16777216.0f);
    *u_resample = (float)(w[1] >> 8) * (1.0f / 16777216.0f);
}

/* ------------------------------------------------------------------------ */
/* Engine throughput profile SPS(B) (Section 3.2.2: profiled once, stored as */
/* a cost table).  Reading: dense fp64 table B = 0..max_tokens, piecewise    */
/* linear between the given breakpoints, constant outside them.              */
/* ------------------------------------------------------------------------ */
int orc_sps_table(const int32_t* bp_tokens, const double* bp_sps, int n_bp,
                  int max_tokens, double* table)
{
    if (n_bp < 1 || max_tokens < 0) return -1;
    for (int k = 1; k < n_bp; ++k)
        if (bp_tokens[k] <= bp_tokens[k - 1]) return -1;
    for (int B = 0; B <= max_tokens; ++B) {
        double y;
        if (B <= bp_tokens[0]) {
            y = bp_sps[0];
        } else if (B >= bp_tokens[n_bp - 1]) {
            y = bp_sps[n_bp - 1];
        } else {
            int k = 0;
            while (!(bp_tokens[k] <= B && B < bp_tokens[k + 1])) ++k;
            double frac = (double)(B - bp_tokens[k]) / (double)(bp_tokens[k + 1] - bp_tokens[k]);
            double dy = bp_sps[k + 1] - bp_sps[k];
            double t = dy * frac;
            y = bp_sps[k] + t;
        }
        table[B] = y;
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Scheduler (Algorithm 1; definitions of a, B, tau, Theta in Section 3.2.2; */
/* no-break variant and capacity limit in Section 5.2).                      */
/* ------------------------------------------------------------------------ */
typedef struct {
    float a;
    int32_t j;
    int32_t r;
} orc_cand_t;

static int cand_cmp(const void* pa, const void* pb)
{
    const orc_cand_t* x = (const orc_cand_t*)pa;
    const orc_cand_t* y = (const orc_cand_t*)pb;
    if (x->a > y->a) return -1;       /* survival probability, descending */
    if (x->a < y->a) return 1;
    if (x->j != y->j) return x->j < y->j ? -1 : 1;   /* then position ascending */
    if (x->r != y->r) return x->r < y->r ? -1 : 1;   /* then request ascending  */
    return 0;
}

/* Confidence as the scheduler reads it: c in [0,1]; NaN or negative ends the
 * block (0), above 1 is 1.  Sets *clamped when it changed anything. */
static float sanitize_conf(float c, int* clamped)
{
    if (!(c >= 0.0f)) { *clamped = 1; return 0.0f; }
    if (c > 1.0f) { *clamped = 1; return 1.0f; }
    return c;
}

/* Survival products a_{r,j} = prod_{i<=j} c_{r,i} (Algorithm 1, line 2), as a
 * left-to-right fp32 product.  Positions at or beyond draft_len[r], and all
 * positions after the product reaches 0, hold 0 and are not candidates. */
static void survival_products(const float* conf, const int32_t* draft_len, int R, int gamma,
                              float* surv, int* clamped)
{
    for (int r = 0; r < R; ++r) {
        int lim = gamma;
        if (draft_len) { lim = draft_len[r]; if (lim < 0) lim = 0; if (lim > gamma) lim = gamma; }
        float a = 1.0f;
        int dead = 0;
        for (int j = 0; j < gamma; ++j) {
            if (j >= lim) dead = 1;
            if (!dead) {
                a = a * sanitize_conf(conf[(size_t)r * gamma + j], clamped);
                if (!(a > 0.0f)) dead = 1;
            }
            surv[(size_t)r * gamma + j] = dead ? 0.0f : a;
        }
    }
}

/* Expected-accept mass of one candidate in units of 2^-40 (an exact integer
 * sum keeps tau independent of summation order). */
static uint64_t fix40(float a)
{
    return (uint64_t)((double)a * 1099511627776.0);
}

typedef struct {
    int32_t B;           /* batch tokens R + sum l*_r        */
    int32_t n_admitted;  /* i*                               */
    int32_t status;      /* warning bits                     */
    int32_t n_candidates;/* |E|                              */
    double tau;          /* expected accepted tokens         */
    double theta;        /* tau * SPS(B)                     */
} orc_sched_info_t;

/*
 * table[0..max_tokens] is SPS; lookups beyond max_tokens use the last entry.
 * theta_path (optional, length >= min(|E|, cap)+1) receives Theta_i * 2^40.
 */
int orc_schedule(const float* conf, const int32_t* draft_len, int R, int gamma,
                 int budget_tokens, int mode, int topk_K,
                 const double* table, int max_tokens,
                 int32_t* out_len, float* out_survival, float* out_expected_len,
                 orc_sched_info_t* info, double* theta_path)
{
    if (R <= 0 || gamma < 0 || max_tokens < 0) return -1;
    size_t n = (size_t)R * (size_t)(gamma > 0 ? gamma : 1);
    float* surv = (float*)calloc(n, sizeof(float));
    orc_cand_t* cand = (orc_cand_t*)malloc(n * sizeof(orc_cand_t));
    if (!surv || !cand) { free(surv); free(cand); return -2; }
    int clamped = 0;
    survival_products(conf, draft_len, R, gamma, surv, &clamped);

    /* candidate space E = {(r,j) : a_{r,j} > 0}, sorted descending by a */
    size_t nE = 0;
    for (int r = 0; r < R; ++r)
        for (int j = 0; j < gamma; ++j) {
            float a = surv[(size_t)r * gamma + j];
            if (a > 0.0f) { cand[nE].a = a; cand[nE].j = j; cand[nE].r = r; ++nE; }
        }
    qsort(cand, nE, sizeof(orc_cand_t), cand_cmp);

    int status = 0;
    if (clamped) status |= ORC_ST_CONF_CLAMPED;
    long cap = (long)budget_tokens - (long)R;
    if (cap < 0) { cap = 0; status |= ORC_ST_BUDGET_LT_R; }
    size_t N = nE < (size_t)cap ? nE : (size_t)cap;

    /* initial state: l = 0, B = R, tau = R, Theta_best = R * SPS(R) */
    uint64_t T = (uint64_t)R << 40;
    int B = R;
    double theta_best = (double)T * table[B < max_tokens ? B : max_tokens];
    uint64_t T_best = T;
    size_t i_star = 0;
    if (theta_path) theta_path[0] = theta_best;

    for (size_t i = 1; i <= N; ++i) {
        T += fix40(cand[i - 1].a);
        B = R + (int)i;
        double theta = (double)T * table[B < max_tokens ? B : max_tokens];
        if (theta_path) theta_path[i] = theta;
        if (mode == ORC_MODE_TOPK) {
            if ((long)i <= (long)topk_K) { theta_best = theta; T_best = T; i_star = i; }
            continue;
        }
        if (theta > theta_best) {
            theta_best = theta; T_best = T; i_star = i;
        } else if (mode == ORC_MODE_EARLY_STOP) {
            break;                                  /* Algorithm 1: else break */
        }
    }

    for (int r = 0; r < R; ++r) out_len[r] = 0;
    for (size_t k = 0; k < i_star; ++k) out_len[cand[k].r] += 1;

    if (out_survival) memcpy(out_survival, surv, (size_t)R * gamma * sizeof(float));
    if (out_expected_len)
        for (int r = 0; r < R; ++r) {
            double e = 1.0;
            for (int j = 0; j < out_len[r]; ++j) e += (double)surv[(size_t)r * gamma + j];
            out_expected_len[r] = (float)e;
        }
    if (info) {
        info->B = R + (int)i_star;
        info->n_admitted = (int32_t)i_star;
        info->status = status;
        info->n_candidates = (int32_t)nE;
        info->tau = (double)T_best / 1099511627776.0;
        info->theta = theta_best / 1099511627776.0;
    }
    free(surv); free(cand);
    return 0;
}

/*
 * Asynchronous scheduling (Section 5.2, "Hardware-Aware Prefix Scheduler in Practice").
 * The capacity K used at step t is the admission count found by the unconstrained (no break)
 * search on the confidences of step t-2; the candidates admitted at step t are the K most
 * confident ones by the CURRENT survival products (dynamic top-K), still under the token cap.
 * state = {t, K slot 0, K slot 1}: slot t mod 2 holds the K of step t-2 until this call
 * overwrites it with the K found on the current confidences (used at step t+2).
 * Reading: the first two steps use the K values the caller put into the slots.
 */
int orc_schedule_async(const float* conf, const int32_t* draft_len, int R, int gamma,
                       int budget_tokens, const double* table, int max_tokens, int32_t* state,
                       int32_t* out_len, float* out_survival, float* out_expected_len,
                       orc_sched_info_t* info)
{
    int32_t* scratch = (int32_t*)malloc((size_t)R * sizeof(int32_t));
    if (!scratch) return -2;
    orc_sched_info_t ginfo;
    /* capacity for step t+2: unconstrained global search on the current confidences */
    int rc = orc_schedule(conf, draft_len, R, gamma, budget_tokens, ORC_MODE_GLOBAL, 0, table, max_tokens,
                          scratch, NULL, NULL, &ginfo, NULL);
    free(scratch);
    if (rc != 0) return rc;
    const int slot = 1 + (state[0] & 1);
    const int K_use = state[slot];
    /* admission at step t: top-K by current scores with the capacity decided two steps ago */
    rc = orc_schedule(conf, draft_len, R, gamma, budget_tokens, ORC_MODE_TOPK, K_use < 0 ? 0 : K_use, table,
                      max_tokens, out_len, out_survival, out_expected_len, info, NULL);
    if (rc != 0) return rc;
    state[slot] = ginfo.n_admitted;
    state[0] += 1;
    return 0;
}

/*
 * Exhaustive companion for tiny batches: every schedule l in {0..gamma}^R whose
 * positions are all candidates (a > 0, j < draft_len) and whose admitted count
 * is within the cap; Theta(l) from the same integer tau and the same table.
 * Returns the maximum Theta*2^40 and, among maximisers, the smallest batch size.
 */
int orc_schedule_bruteforce(const float* conf, const int32_t* draft_len, int R, int gamma,
                            int budget_tokens, const double* table, int max_tokens,
                            double* best_theta_scaled, int32_t* best_B, int32_t* best_len)
{
    if (R <= 0 || R > 8 || gamma < 0 || gamma > 8) return -1;
    float surv[64];
    int clamped = 0;
    survival_products(conf, draft_len, R, gamma, surv, &clamped);
    long cap = (long)budget_tokens - (long)R;
    if (cap < 0) cap = 0;
    int len[8] = {0};
    double best = -1.0; int bestB = -1;
    for (;;) {
        int ok = 1; long tot = 0;
        uint64_t T = (uint64_t)R << 40;
        for (int r = 0; r < R && ok; ++r) {
            for (int j = 0; j < len[r]; ++j) {
                float a = surv[r * gamma + j];
                if (!(a > 0.0f)) { ok = 0; break; }
                T += fix40(a);
            }
            tot += len[r];
        }
        if (ok && tot <= cap) {
            int B = R + (int)tot;
            double theta = (double)T * table[B < max_tokens ? B : max_tokens];
            if (theta > best || (theta == best && B < bestB)) {
                best = theta; bestB = B;
                if (best_len) for (int r = 0; r < R; ++r) best_len[r] = len[r];
            }
        }
        int r = 0;
        while (r < R) { if (++len[r] <= gamma) break; len[r] = 0; ++r; }
        if (r == R) break;
    }
    *best_theta_scaled = best; *best_B = bestB;
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Logit access: bf16 is storage only; its 16 bits are the high half of the  */
/* fp32 pattern.                                                             */
/* ------------------------------------------------------------------------ */
static inline double logit_at(const void* base, int dtype, int64_t row, int64_t stride, int64_t v)
{
    if (dtype == ORC_BF16) {
        uint16_t h = ((const uint16_t*)base)[row * stride + v];
        uint32_t bits = (uint32_t)h << 16;
        float f;
        memcpy(&f, &bits, 4);
        return (double)f;
    }
    return (double)((const float*)base)[row * stride + v];
}

/* Lowest-index argmax; NaN never wins a comparison.  Returns 1 when no element
 * exceeds -inf (index 0 is reported then). */
static int row_argmax(const void* base, int dtype, int64_t row, int64_t stride, int V, int32_t* idx)
{
    double best = -INFINITY;
    int32_t bi = 0;
    for (int v = 0; v < V; ++v) {
        double x = logit_at(base, dtype, row, stride, v);
        if (x > best) { best = x; bi = v; }
    }
    *idx = bi;
    return best == -INFINITY;
}

/* ------------------------------------------------------------------------ */
/* Greedy verification: a draft token is accepted iff it equals the target   */
/* row's argmax (lowest index on ties); the first mismatch ends the prefix   */
/* (Section 2.1: the first rejection discards the rest) and the emitted      */
/* token is the argmax of that row, or of the bonus row when all matched.    */
/* ------------------------------------------------------------------------ */
int orc_verify_greedy(const void* target, int dtype, int64_t target_row_stride, int V,
                      const int32_t* row_offsets, const int32_t* draft_tokens, int R,
                      int32_t* accepted_len, int32_t* out_tokens, int32_t* row_argmax_out,
                      int32_t* status /* [R] */)
{
    if (R <= 0 || V <= 0) return -1;
    for (int r = 0; r < R; ++r) {
        int32_t lo = row_offsets[r], hi = row_offsets[r + 1];
        int32_t st = 0;
        if (lo < 0 || hi - lo < 1) { status[r] = ORC_ST_BAD_OFFSETS; accepted_len[r] = 0; continue; }
        int32_t len = hi - lo - 1;
        for (int32_t i = lo; i < hi; ++i) out_tokens[i] = -1;
        int32_t n = len;
        int32_t emitted = -1;
        for (int32_t j = 0; j < len; ++j) {
            int32_t d = draft_tokens[lo + j];
            if (d < 0 || d >= V) st |= ORC_ST_BAD_TOKEN;
        }
        if (st) {                          /* invalid draft token: nothing is emitted */
            accepted_len[r] = 0; status[r] = st; continue;
        }
        for (int32_t j = 0; j <= len; ++j) {
            int32_t am;
            if (row_argmax(target, dtype, lo + j, target_row_stride, V, &am)) st |= ORC_ST_ALL_NEG_INF;
            if (row_argmax_out) row_argmax_out[lo + j] = am;
            if (j == len) { emitted = am; break; }
            if (draft_tokens[lo + j] != am) { n = j; emitted = am; break; }
        }
        for (int32_t j = 0; j < n; ++j) out_tokens[lo + j] = draft_tokens[lo + j];
        out_tokens[lo + n] = emitted;
        accepted_len[r] = n;
        status[r] = st;
    }
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Sampling verification (Section 2.1): accept x_k with probability          */
/* min(1, p_k^t(x_k)/p_k^d(x_k)), left to right, first rejection discards    */
/* the suffix; on rejection draw from norm(max(0, p - q)) at that position,  */
/* otherwise draw the bonus token from p of the last row (Section 1).        */
/* p = softmax(target/T), q = softmax(draft/T), one temperature for both.    */
/* ------------------------------------------------------------------------ */

/* m = max_v x_v and Z = sum_v exp(x_v - m) in vocabulary order, x = logit/T.
 * Returns 1 when the row is unusable (contains NaN, or its max is -inf). */
static int row_softmax_stats(const void* base, int dtype, int64_t row, int64_t stride, int V,
                             double T, double* m_out, double* Z_out)
{
    double m = -INFINITY;
    int bad = 0;
    for (int v = 0; v < V; ++v) {
        double x = logit_at(base, dtype, row, stride, v) / T;
        if (x != x) bad = 1;
        if (x > m) m = x;
    }
    double Z = 0.0;
    for (int v = 0; v < V; ++v) {
        double x = logit_at(base, dtype, row, stride, v) / T;
        Z += exp(x - m);
    }
    *m_out = m; *Z_out = Z;
    if (m == -INFINITY || !(Z > 0.0) || Z != Z) bad = 1;
    return bad;
}

static inline double prob_at(const void* base, int dtype, int64_t row, int64_t stride, int v,
                             double T, double m, double Z)
{
    return exp(logit_at(base, dtype, row, stride, v) / T - m) / Z;
}

/* Full probability row (used by the pins and by small-case parity checks). */
int orc_softmax_row(const void* base, int dtype, int64_t row, int64_t stride, int V,
                    double temperature, double* probs, double* m_out, double* Z_out)
{
    double m, Z;
    int bad = row_softmax_stats(base, dtype, row, stride, V, temperature, &m, &Z);
    for (int v = 0; v < V; ++v) probs[v] = prob_at(base, dtype, row, stride, v, temperature, m, Z);
    if (m_out) *m_out = m;
    if (Z_out) *Z_out = Z;
    return bad;
}

/* Inverse CDF over p in vocabulary order: smallest v with sum_{i<=v} p_i > thr.
 * If rounding leaves the running sum at or below thr, the last v with p_v > 0. */
static int32_t sample_from_p(const void* base, int dtype, int64_t row, int64_t stride, int V,
                             double T, double m, double Z, double thr, double* margin)
{
    double cum = 0.0;
    int32_t last_pos = -1;
    for (int v = 0; v < V; ++v) {
        double pv = prob_at(base, dtype, row, stride, v, T, m, Z);
        double prev = cum;
        cum += pv;
        if (pv > 0.0) last_pos = v;
        if (cum > thr) {
            double d0 = thr - prev, d1 = cum - thr;
            *margin = d0 < d1 ? d0 : d1;
            return v;
        }
    }
    *margin = 0.0;
    return last_pos;
}

typedef struct {
    const void* target; const void* draft; int dtype;
    int64_t tstride, dstride; int V;
    const int32_t* row_offsets; const int64_t* draft_row_start; const int32_t* draft_tokens;
    int R; double T; const float* temps; uint64_t seed; int eval_all;
    int32_t* accepted_len; int32_t* out_tokens;
    double* p_tok; double* q_tok; double* accept_margin; double* token_margin;
    double* token_margin_abs; double* resid_mass;
    int32_t* status;
    int r_begin, r_end;
} verify_job_t;

static void verify_request(const verify_job_t* J, int r)
{
    int32_t lo = J->row_offsets[r], hi = J->row_offsets[r + 1];
    J->token_margin[r] = NAN;
    if (J->token_margin_abs) J->token_margin_abs[r] = NAN;
    if (J->resid_mass) J->resid_mass[r] = NAN;
    if (lo < 0 || hi - lo < 1) { J->status[r] = ORC_ST_BAD_OFFSETS; J->accepted_len[r] = 0; return; }
    int32_t len = hi - lo - 1;
    int64_t drow0 = J->draft_row_start ? J->draft_row_start[r] : (int64_t)lo - (int64_t)r;
    /* compact layout (Section 5.3, flat ragged rows): the draft rows of request r follow those of the requests
       before it, at lo - r; an earlier request without a row of its own would put them before the array */
    if (drow0 < 0) { J->status[r] = ORC_ST_BAD_OFFSETS; J->accepted_len[r] = 0; return; }
    int32_t st = 0;
    /* per-request temperature (requests of one batch may use different sampling settings) */
    const double T = J->temps ? (double)J->temps[r] : J->T;
    for (int32_t i = lo; i < hi; ++i) {
        J->out_tokens[i] = -1;
        if (J->p_tok) J->p_tok[i] = NAN;
        if (J->q_tok) J->q_tok[i] = NAN;
        if (J->accept_margin) J->accept_margin[i] = NAN;
    }
    for (int32_t j = 0; j < len; ++j) {
        int32_t d = J->draft_tokens[lo + j];
        if (d < 0 || d >= J->V) st |= ORC_ST_BAD_TOKEN;
    }
    if (!(T > 0.0) || !isfinite(T)) st |= ORC_ST_BAD_TEMPERATURE;
    if (st) { J->status[r] = st; J->accepted_len[r] = 0; return; }

    int32_t n = len;           /* first rejected position, or len */
    for (int32_t j = 0; j < len; ++j) {
        if (n < len && !J->eval_all) break;   /* verification stops at the first rejection */
        double mp, Zp, mq, Zq;
        int bad = row_softmax_stats(J->target, J->dtype, lo + j, J->tstride, J->V, T, &mp, &Zp);
        bad |= row_softmax_stats(J->draft, J->dtype, drow0 + j, J->dstride, J->V, T, &mq, &Zq);
        if (bad) { st |= ORC_ST_BAD_ROW; break; }
        int32_t d = J->draft_tokens[lo + j];
        double p = prob_at(J->target, J->dtype, lo + j, J->tstride, d, T, mp, Zp);
        double q = prob_at(J->draft, J->dtype, drow0 + j, J->dstride, d, T, mq, Zq);
        if (J->p_tok) J->p_tok[lo + j] = p;
        if (J->q_tok) J->q_tok[lo + j] = q;
        float ua, ur;
        orc_uniforms(J->seed, (uint32_t)r, (uint32_t)j, &ua, &ur);
        double lhs = (double)ua * q;
        if (J->accept_margin) {
            double big = p > q ? p : q;
            J->accept_margin[lo + j] = big > 0.0 ? fabs(lhs - p) / big : 0.0;
        }
        int accept = lhs < p;      /* u < p/q without the division; u in [0,1) */
        if (!accept && j < n) n = j;
    }
    if (st) { J->status[r] = st; J->accepted_len[r] = 0; return; }

    float ua, ur;
    orc_uniforms(J->seed, (uint32_t)r, (uint32_t)n, &ua, &ur);
    int32_t tok = -1;
    double margin = 0.0, margin_abs = 0.0, resid_W = NAN;
    double mp, Zp;
    if (row_softmax_stats(J->target, J->dtype, lo + n, J->tstride, J->V, T, &mp, &Zp)) {
        J->status[r] = ORC_ST_BAD_ROW; J->accepted_len[r] = 0; return;
    }
    int resampled = 0;
    if (n < len) {
        /* residual norm(max(0, p - q)) at the rejected position */
        double mq, Zq;
        row_softmax_stats(J->draft, J->dtype, drow0 + n, J->dstride, J->V, T, &mq, &Zq);
        double W = 0.0;
        for (int v = 0; v < J->V; ++v) {
            double pv = prob_at(J->target, J->dtype, lo + n, J->tstride, v, T, mp, Zp);
            double qv = prob_at(J->draft, J->dtype, drow0 + n, J->dstride, v, T, mq, Zq);
            double w = pv - qv;
            if (w > 0.0) W += w;
        }
        if (W > 0.0) {
            double thr = (double)ur * W;
            double cum = 0.0;
            int32_t last_pos = -1;
            for (int v = 0; v < J->V; ++v) {
                double pv = prob_at(J->target, J->dtype, lo + n, J->tstride, v, T, mp, Zp);
                double qv = prob_at(J->draft, J->dtype, drow0 + n, J->dstride, v, T, mq, Zq);
                double w = pv - qv;
                if (!(w > 0.0)) continue;
                double prev = cum;
                cum += w;
                last_pos = v;
                if (cum > thr) {
                    double d0 = thr - prev, d1 = cum - thr;
                    /* distance of u' W to the nearer end of the token's interval of the running sum: kept both in
                     * probability units and as a fraction of the residual mass W (the distance on the CDF of the
                     * distribution the token is drawn from) */
                    margin_abs = d0 < d1 ? d0 : d1;
                    margin = margin_abs / W;
                    tok = v;
                    break;
                }
            }
            if (tok < 0) { tok = last_pos; margin = 0.0; margin_abs = 0.0; }
            resampled = 1;
            resid_W = W;
        }
    }
    if (!resampled) {
        /* bonus token from p of row n (also the fallback when the residual is empty) */
        tok = sample_from_p(J->target, J->dtype, lo + n, J->tstride, J->V, T, mp, Zp, (double)ur, &margin);
        margin_abs = margin;       /* p sums to one */
    }
    for (int32_t j = 0; j < n; ++j) J->out_tokens[lo + j] = J->draft_tokens[lo + j];
    J->out_tokens[lo + n] = tok;
    J->accepted_len[r] = n;
    J->token_margin[r] = margin;
    if (J->token_margin_abs) J->token_margin_abs[r] = margin_abs;
    if (J->resid_mass) J->resid_mass[r] = resid_W;
    J->status[r] = st;
}

static void* verify_worker(void* arg)
{
    const verify_job_t* J = (const verify_job_t*)arg;
    for (int r = J->r_begin; r < J->r_end; ++r) verify_request(J, r);
    return NULL;
}

/*
 * eval_all != 0 evaluates p(d), q(d) and the accept margin at every draft
 * position (for parity checks); otherwise evaluation stops at the first
 * rejection, as verification itself does.  n_threads splits requests over
 * pthreads (requests are independent); results do not depend on it.
 */
int orc_verify(const void* target, const void* draft, int dtype,
               int64_t target_row_stride, int64_t draft_row_stride, int V,
               const int32_t* row_offsets, const int64_t* draft_row_start,
               const int32_t* draft_tokens, int R, double temperature, const float* temperatures,
               uint64_t seed, int eval_all, int n_threads,
               int32_t* accepted_len, int32_t* out_tokens,
               double* p_tok, double* q_tok, double* accept_margin, double* token_margin,
               double* token_margin_abs, double* resid_mass, int32_t* status)
{
    if (R <= 0 || V <= 0) return -1;
    if (!temperatures && (!(temperature > 0.0) || !isfinite(temperature))) return -1;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > R) n_threads = R;
    if (n_threads > 256) n_threads = 256;
    verify_job_t base = { target, draft, dtype, target_row_stride, draft_row_stride, V,
                          row_offsets, draft_row_start, draft_tokens, R, temperature, temperatures, seed, eval_all,
                          accepted_len, out_tokens, p_tok, q_tok, accept_margin, token_margin,
                          token_margin_abs, resid_mass, status, 0, R };
    if (n_threads == 1) { verify_worker(&base); return 0; }
    pthread_t th[256];
    verify_job_t jobs[256];
    for (int t = 0; t < n_threads; ++t) {
        jobs[t] = base;
        jobs[t].r_begin = (int)((long)R * t / n_threads);
        jobs[t].r_end = (int)((long)R * (t + 1) / n_threads);
        pthread_create(&th[t], NULL, verify_worker, &jobs[t]);
    }
    for (int t = 0; t < n_threads; ++t) pthread_join(th[t], NULL);
    return 0;
}

/*
 * Analytical per-step acceptance rate (Section 3.2.1, Eq. "accept_rate"):
 *   c*_k = 1 - 1/2 * || p_k^d - p_k^t ||_1
 * for every draft position of the ragged batch, p = softmax(target/T), q = softmax(draft/T).
 * cstar has one entry per target row; bonus-row entries are set to NaN.
 */
int orc_accept_rate(const void* target, const void* draft, int dtype,
                    int64_t target_row_stride, int64_t draft_row_stride, int V,
                    const int32_t* row_offsets, const int64_t* draft_row_start, int R,
                    double temperature, double* cstar, int32_t* status)
{
    if (R <= 0 || V <= 0 || !(temperature > 0.0) || !isfinite(temperature)) return -1;
    for (int r = 0; r < R; ++r) {
        int32_t lo = row_offsets[r], hi = row_offsets[r + 1];
        status[r] = 0;
        if (lo < 0 || hi - lo < 1) { status[r] = ORC_ST_BAD_OFFSETS; continue; }
        int32_t len = hi - lo - 1;
        int64_t drow0 = draft_row_start ? draft_row_start[r] : (int64_t)lo - (int64_t)r;
        if (drow0 < 0) { status[r] = ORC_ST_BAD_OFFSETS; continue; }   /* see verify_request */
        cstar[hi - 1] = NAN;
        for (int32_t j = 0; j < len; ++j) {
            double mp, Zp, mq, Zq;
            int bad = row_softmax_stats(target, dtype, lo + j, target_row_stride, V, temperature, &mp, &Zp);
            bad |= row_softmax_stats(draft, dtype, drow0 + j, draft_row_stride, V, temperature, &mq, &Zq);
            if (bad) { status[r] |= ORC_ST_BAD_ROW; cstar[lo + j] = NAN; continue; }
            double l1 = 0.0;
            for (int v = 0; v < V; ++v) {
                double pv = prob_at(target, dtype, lo + j, target_row_stride, v, temperature, mp, Zp);
                double qv = prob_at(draft, dtype, drow0 + j, draft_row_stride, v, temperature, mq, Zq);
                l1 += fabs(qv - pv);
            }
            cstar[lo + j] = 1.0 - 0.5 * l1;
        }
    }
    return 0;
}

/*
 * Markov-head draft step (Section 3.1, Eq. "sequential-factorization" and Eq. "markov"):
 * the draft logits of position k are the backbone's base logits plus a first-order transition
 * bias from the previously sampled token,
 *     logits[r, v] = U_k[r, v] + sum_i W1[x_prev[r], i] * W2[i, v],
 * with W1 in R^{V x rank} (embedding lookup) and W2 in R^{rank x V} (logit projection).
 * All inputs are bf16 bit patterns; the sum is taken in fp64 in index order.  The result is
 * returned in fp64 and, rounded to nearest-even, as the bf16 pattern a drafter would store
 * (the verifier later reads exactly those stored logits as the draft distribution).
 */
static inline double bf16_to_f64(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}
static inline uint16_t f64_to_bf16_rne(double x)
{
    float f = (float)x;                 /* fp64 -> fp32 (double rounding is far below a bf16 ulp) */
    uint32_t bits;
    memcpy(&bits, &f, 4);
    if ((bits & 0x7F800000u) == 0x7F800000u) return (uint16_t)(bits >> 16);   /* inf / nan */
    uint32_t lsb = (bits >> 16) & 1u;
    bits += 0x7FFFu + lsb;
    return (uint16_t)(bits >> 16);
}

int orc_markov_logits(const uint16_t* U, int64_t u_stride, const uint16_t* W1, const uint16_t* W2,
                      const int32_t* x_prev, int R, int V, int rank, double* out_f64, uint16_t* out_bf16)
{
    if (R <= 0 || V <= 0 || rank <= 0) return -1;
    for (int r = 0; r < R; ++r) {
        int32_t x = x_prev[r];
        if (x < 0 || x >= V) return -2;
        for (int v = 0; v < V; ++v) {
            double b = 0.0;
            for (int i = 0; i < rank; ++i)
                b += bf16_to_f64(W1[(size_t)x * rank + i]) * bf16_to_f64(W2[(size_t)i * V + v]);
            double l = bf16_to_f64(U[(size_t)r * u_stride + v]) + b;
            if (out_f64) out_f64[(size_t)r * V + v] = l;
            if (out_bf16) out_bf16[(size_t)r * V + v] = f64_to_bf16_rne(l);
        }
    }
    return 0;
}

/* Confidence head (Section 3.2.1, Eq. "confidence"): c = sigmoid(w^T [h ; W1[x_prev]]),
 * h in R^d (bf16), w in R^{d + rank} (fp32). */
int orc_confidence(const uint16_t* H, int64_t h_stride, int d, const uint16_t* W1, int rank, int V,
                   const float* w, const int32_t* x_prev, int R, double* conf)
{
    for (int r = 0; r < R; ++r) {
        int32_t x = x_prev[r];
        if (x < 0 || x >= V) return -2;
        double z = 0.0;
        for (int i = 0; i < d; ++i) z += (double)w[i] * bf16_to_f64(H[(size_t)r * h_stride + i]);
        for (int i = 0; i < rank; ++i) z += (double)w[d + i] * bf16_to_f64(W1[(size_t)x * rank + i]);
        conf[r] = 1.0 / (1.0 + exp(-z));
    }
    return 0;
}

/* Threaded wrapper for the greedy verifier's timing leg (same results). */
typedef struct {
    const void* target; int dtype; int64_t stride; int V;
    const int32_t* row_offsets; const int32_t* draft_tokens;
    int32_t* accepted_len; int32_t* out_tokens; int32_t* status; int r_begin, r_end;
} greedy_job_t;

static void* greedy_worker(void* arg)
{
    greedy_job_t* G = (greedy_job_t*)arg;
    /* each slice is an independent batch over a window of the offsets array */
    orc_verify_greedy(G->target, G->dtype, G->stride, G->V, G->row_offsets + G->r_begin,
                      G->draft_tokens, G->r_end - G->r_begin,
                      G->accepted_len + G->r_begin, G->out_tokens, NULL, G->status + G->r_begin);
    return NULL;
}

int orc_verify_greedy_mt(const void* target, int dtype, int64_t target_row_stride, int V,
                         const int32_t* row_offsets, const int32_t* draft_tokens, int R,
                         int n_threads, int32_t* accepted_len, int32_t* out_tokens, int32_t* status)
{
    if (R <= 0 || V <= 0) return -1;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > R) n_threads = R;
    if (n_threads > 256) n_threads = 256;
    pthread_t th[256];
    greedy_job_t jobs[256];
    for (int t = 0; t < n_threads; ++t) {
        greedy_job_t g = { target, dtype, target_row_stride, V, row_offsets, draft_tokens,
                           accepted_len, out_tokens, status,
                           (int)((long)R * t / n_threads), (int)((long)R * (t + 1) / n_threads) };
        jobs[t] = g;
        if (g.r_end > g.r_begin) pthread_create(&th[t], NULL, greedy_worker, &jobs[t]);
    }
    for (int t = 0; t < n_threads; ++t)
        if (jobs[t].r_end > jobs[t].r_begin) pthread_join(th[t], NULL);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Sequential Temperature Scaling (Section 3.2.1, "Post-hoc Calibration").   */
/* From left to right, position k gets the temperature of a 1-D grid that     */
/* minimises the Expected Calibration Error of the cumulative product         */
/*   a_{n,k} = prod_{i<=k} sigmoid(logit(c_{n,i}) / T_i)                      */
/* over held-out blocks n, with T_1..T_{k-1} already fixed.  The label of     */
/* (n, k) is 1 when the block's draft prefix through k was accepted           */
/* (accepted_len[n] > k, positions 0-based); a block counts at position k     */
/* only if that position was verified (k < verified_len[n]; NULL = all).      */
/* Readings where the paper is silent: temperature scaling acts on the logit  */
/* of the sigmoid output; a confidence outside (0,1) is clamped to [0,1]       */
/* (NaN -> 0) and not rescaled; ECE uses n_bins equal-width bins on [0,1],     */
/*   ECE = (1/N_k) * sum_b | sum_{n in b} y_n - sum_{n in b} a_n |,            */
/* bin(a) = min(n_bins-1, floor(a*n_bins)); ties take the first grid point;    */
/* a position nobody verified keeps T = 1.                                     */
/* ------------------------------------------------------------------------ */
static double sts_scaled(double c, double T)
{
    if (c != c || c <= 0.0) return 0.0;
    if (c >= 1.0) return 1.0;
    double z = log(c) - log1p(-c);
    return 1.0 / (1.0 + exp(-z / T));
}

static double sts_ece(const double* a, const uint8_t* y, const uint8_t* used, int N, int n_bins)
{
    double* sum_a = (double*)calloc((size_t)n_bins, sizeof(double));
    double* sum_y = (double*)calloc((size_t)n_bins, sizeof(double));
    long cnt = 0;
    for (int n = 0; n < N; ++n) {
        if (!used[n]) continue;
        int b = (int)floor(a[n] * n_bins);
        if (b > n_bins - 1) b = n_bins - 1;
        if (b < 0) b = 0;
        sum_a[b] += a[n];
        sum_y[b] += y[n];
        ++cnt;
    }
    double e = 0.0;
    for (int b = 0; b < n_bins; ++b) e += fabs(sum_y[b] - sum_a[b]);
    free(sum_a); free(sum_y);
    return cnt ? e / (double)cnt : 0.0;
}

int orc_sts_calibrate(const float* conf, int N, int gamma, const int32_t* accepted_len,
                      const int32_t* verified_len, const float* grid, int G, int n_bins,
                      float* out_T, double* ece_before, double* ece_after, double* ece_grid)
{
    if (N <= 0 || gamma <= 0 || G <= 0 || n_bins <= 0) return -1;
    for (int g = 0; g < G; ++g) if (!(grid[g] > 0.f) || isinf(grid[g])) return -2;
    double* a_raw = (double*)malloc(sizeof(double) * (size_t)N);   /* product of raw confidences   */
    double* a_cal = (double*)malloc(sizeof(double) * (size_t)N);   /* product of calibrated ones   */
    double* a_try = (double*)malloc(sizeof(double) * (size_t)N);
    uint8_t* y = (uint8_t*)malloc((size_t)N);
    uint8_t* used = (uint8_t*)malloc((size_t)N);
    for (int n = 0; n < N; ++n) a_raw[n] = a_cal[n] = 1.0;
    for (int k = 0; k < gamma; ++k) {
        long cnt = 0;
        for (int n = 0; n < N; ++n) {
            used[n] = (uint8_t)(!verified_len || k < verified_len[n]);
            y[n] = (uint8_t)(accepted_len[n] > k);
            cnt += used[n];
            a_raw[n] *= sts_scaled((double)conf[(size_t)n * gamma + k], 1.0);
        }
        if (ece_before) ece_before[k] = sts_ece(a_raw, y, used, N, n_bins);
        int best = -1;
        double best_e = 0.0;
        for (int g = 0; g < G && cnt > 0; ++g) {
            for (int n = 0; n < N; ++n)
                a_try[n] = a_cal[n] * sts_scaled((double)conf[(size_t)n * gamma + k], (double)grid[g]);
            double e = sts_ece(a_try, y, used, N, n_bins);
            if (ece_grid) ece_grid[(size_t)k * G + g] = e;
            if (best < 0 || e < best_e) { best = g; best_e = e; }
        }
        if (cnt == 0 && ece_grid) for (int g = 0; g < G; ++g) ece_grid[(size_t)k * G + g] = 0.0;
        double T = best >= 0 ? (double)grid[best] : 1.0;
        out_T[k] = (float)T;
        for (int n = 0; n < N; ++n) a_cal[n] *= sts_scaled((double)conf[(size_t)n * gamma + k], T);
        if (ece_after) ece_after[k] = sts_ece(a_cal, y, used, N, n_bins);
    }
    free(a_raw); free(a_cal); free(a_try); free(y); free(used);
    return 0;
}

/* Calibrated confidences for the scheduler: c~ = sigmoid(logit(c) / T_k). */
int orc_sts_apply(const float* conf, int N, int gamma, const float* T, double* out)
{
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < gamma; ++k)
            out[(size_t)n * gamma + k] = sts_scaled((double)conf[(size_t)n * gamma + k], (double)T[k]);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Top-k / top-p truncation of the target distribution (per-request sampling */
/* parameters; the evaluation of Section 4.1 takes each model's suggested     */
/* sampling settings and the paper gives no rule of its own).  Readings:     */
/*  - the truncated distribution is obtained by setting the logits of the     */
/*    excluded tokens to -inf, so that softmax renormalises over the kept set  */
/*    S and the lossless verifier runs unchanged on the masked rows;           */
/*  - S is a value cut, S = { v : x_v >= tau }: every token tied with the      */
/*    threshold value is kept (no dependence on token order);                  */
/*  - top-k first: tau_k = k-th largest logit (0 or >= V: off); then top-p on  */
/*    the distribution renormalised over the top-k set: walking the distinct   */
/*    values downwards, tau_p is the first value at which the cumulative mass  */
/*    reaches top_p * Z_k (top_p >= 1: off; top_p <= 0: only the maximum);     */
/*    tau = max(tau_k, tau_p);                                                 */
/*  - a row with NaN, +inf or no finite element is left as it is (the          */
/*    verifier reports it).                                                    */
/* Every target row of request r uses top_k[r], top_p[r] and its temperature.  */
/* margin[row]: relative distance of top_p * Z_k from the nearest cumulative   */
/* mass at a value boundary (how close the top-p decision was); +inf if none.  */
/* ------------------------------------------------------------------------ */
static int cmp_desc_double(const void* a, const void* b)
{
    double x = *(const double*)a, y = *(const double*)b;
    return x > y ? -1 : (x < y ? 1 : 0);
}

int orc_warp_target(void* target, int dtype, int64_t stride, int V, const int32_t* row_offsets, int R,
                    const int32_t* top_k, const float* top_p, double temperature, const float* temperatures,
                    double* tau_out, int32_t* kept_out, double* margin_out)
{
    if (R <= 0 || V <= 0) return -1;
    double* v = (double*)malloc(sizeof(double) * (size_t)V);
    for (int r = 0; r < R; ++r) {
        const double T = temperatures ? (double)temperatures[r] : temperature;
        const int k = top_k ? top_k[r] : 0;
        const double pr = top_p ? (double)top_p[r] : 1.0;
        for (int row = row_offsets[r]; row < row_offsets[r + 1]; ++row) {
            if (tau_out) tau_out[row] = -INFINITY;
            if (kept_out) kept_out[row] = V;
            if (margin_out) margin_out[row] = INFINITY;
            const int use_k = k > 0 && k < V, use_p = pr < 1.0;
            if (!use_k && !use_p) continue;
            if (!(T > 0.0) || isinf(T)) continue;
            int bad = 0;
            for (int i = 0; i < V; ++i) { v[i] = logit_at(target, dtype, row, stride, i); if (v[i] != v[i]) bad = 1; }
            qsort(v, (size_t)V, sizeof(double), cmp_desc_double);
            const double m = v[0];
            if (bad || m == INFINITY || m == -INFINITY) continue;
            double tau_k = -INFINITY;
            int n_k = V;                                   /* size of the top-k set, ties included */
            if (use_k) {
                tau_k = v[k - 1];
                n_k = k;
                while (n_k < V && v[n_k] == tau_k) ++n_k;
            }
            double tau = tau_k;
            if (use_p) {
                double Zk = 0.0;
                for (int i = 0; i < n_k; ++i) Zk += exp((v[i] - m) / T);
                const double thr = pr * Zk;
                double cum = 0.0, margin = INFINITY, tau_p = m;
                int i = 0;
                if (pr > 0.0) {
                    while (i < n_k) {                       /* one group of equal values at a time */
                        const double val = v[i];
                        const double before = cum;
                        while (i < n_k && v[i] == val) { cum += exp((val - m) / T); ++i; }
                        tau_p = val;
                        double d0 = fabs(thr - before) / Zk, d1 = fabs(cum - thr) / Zk;
                        if (d0 < margin) margin = d0;
                        if (d1 < margin) margin = d1;
                        if (cum >= thr) break;
                    }
                }
                if (tau_p > tau) tau = tau_p;
                if (margin_out) margin_out[row] = margin;
            }
            int kept = 0;
            for (int i = 0; i < V; ++i) {
                double x = logit_at(target, dtype, row, stride, i);
                if (x >= tau) { ++kept; continue; }
                if (dtype == ORC_BF16) ((uint16_t*)target)[(size_t)row * stride + i] = 0xFF80u;   /* -inf */
                else ((float*)target)[(size_t)row * stride + i] = -INFINITY;
            }
            if (tau_out) tau_out[row] = tau;
            if (kept_out) kept_out[row] = kept;
        }
    }
    free(v);
    return 0;
}
