/*
 * rapid_oracle.c -- float64 CPU oracle for the importance-weighted group-advantage
 * policy-gradient loss of RAPID (arXiv 2510.03515) and its gradient w.r.t. the logits.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, single-definition restatement of the
 * paper's equations, used only by the test-suite, by the smoke check and by the CPU-baseline
 * leg of the benchmark.  The CUDA library never calls it and shares no code with it.
 *
 * The steps, in the paper's order and notation (Algorithm 1, procedure IW-GRPG, the two
 * "Compute ..." lines):
 *
 *   step 1  log pi_theta(y_t | .) = z[y_t] - log sum_v exp z[v]         (softmax policy, Sec. 3.1)
 *   step 2  s_n = sum_t m_t (log pi_theta(y_t) - log mu(y_t))           (Sec. 4.3, "Importance-
 *           S_n = sum_t m_t  log pi_theta(y_t)                           weight clipping": token
 *                                                                        weights are accumulated
 *                                                                        per generation)
 *   step 3  w_n = exp(s_n),  c_n = min(w_n, eta)                        (Eq. 5, read as a cap)
 *   step 4  A_n = R_n - (1/N_k) sum_{n' in group k} c_n' R_n'           (Eq. 5; Eq. 2 if c == 1;
 *                                                                        Eq. 4 if eta = +inf)
 *   step 5  g_n = chat_n A_n / Z,  loss = - sum_n g_n S_n                (Eq. 3 with
 *                                                                        grad pi / mu = w grad log pi)
 *   step 6  dz[r,v] = g_n m_r (softmax(z[r,.])_v - 1[v = y_r])          (chain rule through step 1)
 *
 * Every sum runs in index order, in double, with no blocking or reordering.  The only
 * parallelism is an OpenMP "parallel for" over rows in steps 1 and 6 (rows are independent, so
 * the result does not depend on the thread count); it exists so that the oracle can be timed on
 * all host cores.  Compile with -ffp-contract=off so that no multiply-add is fused.
 *
 * Pins (tests/test_oracle_pins.py): closed forms (all-equal logits), brute force on tiny rows,
 * agreement with a library logsumexp, zero-sum identities of Eq. 2 and Eq. 5, the on-policy
 * reduction to Eq. 1 + Eq. 2, hand-worked rational examples under tests/golden/, row sums of
 * dlogits, and two independent central finite-difference checks.
 * What the paper leaves open (min-vs-max in Eq. 5, whether the outer weight of Eq. 3 is also
 * clipped, the 1/N normaliser) is "parity unpinned" by the paper itself: both readings of the
 * outer weight are implemented here and selected by a flag.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* flag bits -- same numeric values as the library's public flags so that a test can pass one
 * integer to both sides; the meaning is restated here, nothing is included from the library. */
#define ORACLE_FLAG_OUTER_UNCLIPPED 1u     /* step 5 uses w_n (Eq. 3 as printed), not c_n        */
#define ORACLE_FLAG_NORM_TOKENS 2u         /* Z = number of unmasked tokens instead of N         */
#define ORACLE_FLAG_ADV_INPUT_IS_WEIGHT 4u /* step 3 input is w_n itself, not s_n = log w_n      */
#define ORACLE_FLAG_LEAVE_ONE_OUT 8u       /* baseline over the group without n, / (N_k - 1)     */
#define ORACLE_FLAG_LOO_LITERAL_DIVISOR 16u /* with LEAVE_ONE_OUT: divide by N_k as printed      */

void rapid_oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int rapid_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Exact widening of one stored logit to double.  bf16 is the upper half of an IEEE float. */
static inline double load_elem(const void* base, int dtype, int64_t idx) {
    if (dtype == ORACLE_BF16) {
        uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float*)base)[idx];
}

/* ---------------------------------------------------------------------------------------------
 * step 1: per-row log-sum-exp and the sampled token's log-probability.
 *   logits  [n_rows, ld] (first `vocab` entries of each row are used)
 *   row_ok  out, 1 where the row takes part (mask != 0 and 0 <= target < vocab), else 0
 *   lse, token_logp   out, 0 for rows that do not take part
 * returns the number of rows whose mask is set but whose target id is outside [0, vocab).
 * ------------------------------------------------------------------------------------------- */
int64_t rapid_oracle_token_logp(const void* logits, int dtype, int64_t ld, int64_t n_rows,
                                int32_t vocab, const int32_t* targets, const uint8_t* mask,
                                double* lse, double* token_logp, uint8_t* row_ok) {
    int64_t n_bad = 0;
#pragma omp parallel for schedule(dynamic, 16) reduction(+ : n_bad)
    for (int64_t r = 0; r < n_rows; ++r) {
        lse[r] = 0.0;
        token_logp[r] = 0.0;
        row_ok[r] = 0;
        if (mask && !mask[r]) continue;
        int32_t y = targets[r];
        if (y < 0 || y >= vocab) {
            n_bad += 1;
            continue;
        }
        const int64_t off = r * ld;
        double big = load_elem(logits, dtype, off);
        for (int32_t v = 1; v < vocab; ++v) {
            double z = load_elem(logits, dtype, off + v);
            if (z > big) big = z;
        }
        double sum = 0.0;
        for (int32_t v = 0; v < vocab; ++v) sum += exp(load_elem(logits, dtype, off + v) - big);
        lse[r] = big + log(sum);
        token_logp[r] = load_elem(logits, dtype, off + y) - lse[r];
        row_ok[r] = 1;
    }
    return n_bad;
}

/* ---------------------------------------------------------------------------------------------
 * step 2: per-generation sums over the unmasked tokens, in token order.
 *   seq_log_ratio[n] = s_n,  seq_logp[n] = S_n,  seq_tokens[n] = number of tokens that count
 * ------------------------------------------------------------------------------------------- */
void rapid_oracle_seq_reduce(int32_t n_seq, int32_t seq_len, const double* token_logp,
                             const float* behav_logp, const uint8_t* row_ok, double* seq_log_ratio,
                             double* seq_logp, int32_t* seq_tokens) {
    for (int32_t n = 0; n < n_seq; ++n) {
        double s = 0.0, S = 0.0;
        int32_t cnt = 0;
        for (int32_t t = 0; t < seq_len; ++t) {
            int64_t r = (int64_t)n * seq_len + t;
            if (!row_ok[r]) continue;
            s += token_logp[r] - (double)behav_logp[r];
            S += token_logp[r];
            cnt += 1;
        }
        seq_log_ratio[n] = s;
        seq_logp[n] = S;
        seq_tokens[n] = cnt;
    }
}

/* step 3 for one generation: w_n (1 when on-policy) and its clipped value c_n = min(w_n, eta) */
static double clipped_weight(const double* seq_log_ratio, int32_t n, double eta, uint32_t flags,
                             double* w_out) {
    double w = 1.0;
    if (seq_log_ratio)
        w = (flags & ORACLE_FLAG_ADV_INPUT_IS_WEIGHT) ? seq_log_ratio[n] : exp(seq_log_ratio[n]);
    *w_out = w;
    return (w < eta) ? w : eta; /* a tie gives eta */
}

/* ---------------------------------------------------------------------------------------------
 * steps 3 and 4: clipped generation-level weights and the group advantage.
 *   seq_log_ratio  s_n (or w_n with ADV_INPUT_IS_WEIGHT); NULL means on-policy, w == 1 (Eq. 2)
 *   group_offsets  [n_groups + 1]; group k is the index range [off[k], off[k+1])
 *   weight, clipped_w, adv64, adv32   outputs (any may be NULL)
 * returns 0, or -1 if the offsets are not a monotone cover of [0, n_seq) (nothing is written).
 * A group of size zero is allowed and simply contributes nothing.
 * ------------------------------------------------------------------------------------------- */
int rapid_oracle_group_advantage(int32_t n_seq, int32_t n_groups, const float* rewards,
                                 const double* seq_log_ratio, const int32_t* group_offsets,
                                 double eta, uint32_t flags, double* weight, double* clipped_w,
                                 double* adv64, float* adv32) {
    if (group_offsets[0] != 0 || group_offsets[n_groups] != n_seq) return -1;
    for (int32_t k = 0; k < n_groups; ++k)
        if (group_offsets[k + 1] < group_offsets[k]) return -1;

    for (int32_t k = 0; k < n_groups; ++k) {
        const int32_t lo = group_offsets[k], hi = group_offsets[k + 1];
        const int32_t Nk = hi - lo;
        if (Nk == 0) continue;
        /* step 3 for the members of this group, and sum_{n'} c_n' R_n' in index order */
        double csum = 0.0;
        for (int32_t n = lo; n < hi; ++n) {
            double w;
            const double c = clipped_weight(seq_log_ratio, n, eta, flags, &w);
            if (weight) weight[n] = w;
            if (clipped_w) clipped_w[n] = c;
            csum += c * (double)rewards[n];
        }
        /* step 4 */
        for (int32_t n = lo; n < hi; ++n) {
            double a;
            if (flags & ORACLE_FLAG_LEAVE_ONE_OUT) {
                /* baseline over the other members of the group (display after Eq. 4) */
                double others = 0.0, w;
                for (int32_t q = lo; q < hi; ++q)
                    if (q != n) others += clipped_weight(seq_log_ratio, q, eta, flags, &w) *
                                          (double)rewards[q];
                if (flags & ORACLE_FLAG_LOO_LITERAL_DIVISOR)
                    a = (double)rewards[n] - others / (double)Nk;
                else if (Nk > 1)
                    a = (double)rewards[n] - others / (double)(Nk - 1);
                else
                    a = (double)rewards[n]; /* nobody else to form a baseline from */
            } else {
                a = (double)rewards[n] - csum / (double)Nk;
            }
            if (adv64) adv64[n] = a;
            if (adv32) adv32[n] = (float)a;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * step 5: per-generation coefficient g_n, the scalar loss, and the side statistics.
 *   stats_out[0] = number of generations with w_n > eta (strictly)
 *   stats_out[1] = mean_n log c_n        (log c_n taken as min(s_n, log eta), which equals
 *   stats_out[2] = mean_n |log c_n|       log(min(exp s_n, eta)) but cannot underflow)
 *   stats_out[3] = total number of tokens that count
 * ------------------------------------------------------------------------------------------- */
double rapid_oracle_coef_loss(int32_t n_seq, const double* seq_log_ratio, const double* seq_logp,
                              const int32_t* seq_tokens, const double* weight,
                              const double* clipped_w, const double* adv64, double eta,
                              uint32_t flags, double* coef, double* stats_out) {
    double total_tokens = 0.0;
    for (int32_t n = 0; n < n_seq; ++n) total_tokens += (double)seq_tokens[n];
    const double Z = (flags & ORACLE_FLAG_NORM_TOKENS) ? total_tokens : (double)n_seq;

    double loss = 0.0, sum_log = 0.0, sum_abs = 0.0, n_clip = 0.0;
    const double log_eta = log(eta);
    for (int32_t n = 0; n < n_seq; ++n) {
        double chat = (flags & ORACLE_FLAG_OUTER_UNCLIPPED) ? weight[n] : clipped_w[n];
        double g = (Z > 0.0) ? chat * adv64[n] / Z : 0.0;
        coef[n] = g;
        loss -= g * seq_logp[n];
        if (weight[n] > eta) n_clip += 1.0;
        double lc = (seq_log_ratio[n] < log_eta) ? seq_log_ratio[n] : log_eta;
        sum_log += lc;
        sum_abs += fabs(lc);
    }
    if (stats_out) {
        stats_out[0] = n_clip;
        stats_out[1] = sum_log / (double)n_seq;
        stats_out[2] = sum_abs / (double)n_seq;
        stats_out[3] = total_tokens;
    }
    return loss;
}

/* ---------------------------------------------------------------------------------------------
 * step 6 for a list of rows: out[i, v] = g_{n(r)} m_r (exp(z[r,v] - lse[r]) - 1[v = y_r]),
 * r = rows[i].  `logits` points at global row `row_base` (so that a caller can hand over a
 * chunk of a larger grid); lse, row_ok, targets are indexed by global row.  out is [n_list, vocab].
 * ------------------------------------------------------------------------------------------- */
void rapid_oracle_dlogits_rows(const void* logits, int dtype, int64_t ld, int64_t row_base,
                               int32_t vocab, int32_t seq_len, const int32_t* targets,
                               const uint8_t* row_ok, const double* lse, const double* coef,
                               const int64_t* rows, int64_t n_list, double* out) {
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < n_list; ++i) {
        const int64_t r = rows[i];
        const int32_t n = (int32_t)(r / seq_len);
        double* o = out + i * (int64_t)vocab;
        if (!row_ok[r]) {
            for (int32_t v = 0; v < vocab; ++v) o[v] = 0.0;
            continue;
        }
        const double g = coef[n];
        const int64_t off = (r - row_base) * ld;
        for (int32_t v = 0; v < vocab; ++v) {
            double p = exp(load_elem(logits, dtype, off + v) - lse[r]);
            o[v] = g * (p - (v == targets[r] ? 1.0 : 0.0));
        }
    }
}

/* ---------------------------------------------------------------------------------------------
 * steps 1-6 in one call over a whole mini-batch (n_seq x seq_len rows).
 * Optional outputs may be NULL.  dlogits, if given, is [n_rows, vocab] doubles (dense).
 * returns 0, or -1 for bad group offsets.
 * ------------------------------------------------------------------------------------------- */
int rapid_oracle_pg_loss(const void* logits, int dtype, int64_t ld, int32_t n_seq, int32_t seq_len,
                         int32_t vocab, int32_t n_groups, const int32_t* targets,
                         const uint8_t* mask, const float* behav_logp, const float* rewards,
                         const int32_t* group_offsets, double eta, uint32_t flags,
                         /* outputs */
                         double* loss, double* lse, double* token_logp, uint8_t* row_ok,
                         double* seq_log_ratio, double* seq_logp, int32_t* seq_tokens,
                         double* weight, double* clipped_w, double* adv64, float* adv32,
                         double* coef, double* stats_out, int64_t* n_bad_token, double* dlogits) {
    const int64_t n_rows = (int64_t)n_seq * seq_len;
    int64_t bad = rapid_oracle_token_logp(logits, dtype, ld, n_rows, vocab, targets, mask, lse,
                                          token_logp, row_ok);
    if (n_bad_token) *n_bad_token = bad;
    rapid_oracle_seq_reduce(n_seq, seq_len, token_logp, behav_logp, row_ok, seq_log_ratio,
                            seq_logp, seq_tokens);
    int rc = rapid_oracle_group_advantage(n_seq, n_groups, rewards, seq_log_ratio, group_offsets,
                                          eta, flags & ~ORACLE_FLAG_ADV_INPUT_IS_WEIGHT, weight,
                                          clipped_w, adv64, adv32);
    if (rc) return rc;
    *loss = rapid_oracle_coef_loss(n_seq, seq_log_ratio, seq_logp, seq_tokens, weight, clipped_w,
                                   adv64, eta, flags, coef, stats_out);
    if (dlogits) {
        for (int64_t r0 = 0; r0 < n_rows; r0 += 1024) {
            int64_t list[1024];
            int64_t cnt = (n_rows - r0 < 1024) ? n_rows - r0 : 1024;
            for (int64_t i = 0; i < cnt; ++i) list[i] = r0 + i;
            rapid_oracle_dlogits_rows(logits, dtype, ld, 0, vocab, seq_len, targets, row_ok, lse,
                                      coef, list, cnt, dlogits + r0 * (int64_t)vocab);
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Fused-head form: the logits are z = h W with h [n_rows, hidden] and W [hidden, vocab], both
 * bf16, and are never stored by the method.  The oracle simply forms them in double.
 *   rows      list of global rows to produce (NULL = rows 0..n_list-1)
 *   out       [n_list, vocab] doubles
 * ------------------------------------------------------------------------------------------- */
void rapid_oracle_head_logits(const uint16_t* hidden, const uint16_t* w_vocab, int32_t hidden_dim,
                              int32_t vocab, const int64_t* rows, int64_t n_list, double* out) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_list; ++i) {
        const int64_t r = rows ? rows[i] : i;
        double* o = out + i * (int64_t)vocab;
        for (int32_t v = 0; v < vocab; ++v) o[v] = 0.0;
        for (int32_t d = 0; d < hidden_dim; ++d) {
            const double hv = load_elem(hidden, ORACLE_BF16, r * (int64_t)hidden_dim + d);
            const int64_t woff = (int64_t)d * vocab;
            for (int32_t v = 0; v < vocab; ++v)
                o[v] += hv * load_elem(w_vocab, ORACLE_BF16, woff + v);
        }
    }
}

/* step 1 on double logits held in memory (used after rapid_oracle_head_logits) */
void rapid_oracle_token_logp_f64(const double* z, int64_t n_list, int32_t vocab,
                                 const int32_t* targets_of_list, double* lse, double* token_logp) {
    for (int64_t i = 0; i < n_list; ++i) {
        const double* row = z + i * (int64_t)vocab;
        double big = row[0];
        for (int32_t v = 1; v < vocab; ++v)
            if (row[v] > big) big = row[v];
        double sum = 0.0;
        for (int32_t v = 0; v < vocab; ++v) sum += exp(row[v] - big);
        lse[i] = big + log(sum);
        token_logp[i] = row[targets_of_list[i]] - lse[i];
    }
}

/* dz rows from double logits: dz[i,v] = g_i (exp(z[i,v] - lse_i) - 1[v = y_i]) (in place) */
void rapid_oracle_dlogits_f64(double* z, int64_t n_list, int32_t vocab,
                              const int32_t* targets_of_list, const double* lse,
                              const double* coef_of_list) {
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < n_list; ++i) {
        double* row = z + i * (int64_t)vocab;
        for (int32_t v = 0; v < vocab; ++v)
            row[v] = coef_of_list[i] * (exp(row[v] - lse[i]) - (v == targets_of_list[i] ? 1.0 : 0.0));
    }
}

/* dh[r, d] = sum_v dz[r, v] W[d, v]  for the rows held in dz ([n_list, vocab]) */
void rapid_oracle_head_dhidden(const double* dz, const uint16_t* w_vocab, int32_t hidden_dim,
                               int32_t vocab, int64_t n_list, double* dh) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < n_list; ++i) {
        const double* row = dz + i * (int64_t)vocab;
        for (int32_t d = 0; d < hidden_dim; ++d) {
            double acc = 0.0;
            const int64_t woff = (int64_t)d * vocab;
            for (int32_t v = 0; v < vocab; ++v)
                acc += row[v] * load_elem(w_vocab, ORACLE_BF16, woff + v);
            dh[i * (int64_t)hidden_dim + d] = acc;
        }
    }
}

/* dW[d, v] += sum_i h[rows[i], d] dz[i, v]; the caller zeroes dW and may call this once per
 * block of rows (the sum over rows is then taken block by block, rows in order). */
void rapid_oracle_head_dweight_accum(const double* dz, const uint16_t* hidden, int32_t hidden_dim,
                                     int32_t vocab, const int64_t* rows, int64_t n_list,
                                     double* dW) {
#pragma omp parallel for schedule(static)
    for (int32_t d = 0; d < hidden_dim; ++d) {
        double* o = dW + (int64_t)d * vocab;
        for (int64_t i = 0; i < n_list; ++i) {
            const int64_t r = rows ? rows[i] : i;
            const double hv = load_elem(hidden, ORACLE_BF16, r * (int64_t)hidden_dim + d);
            const double* row = dz + i * (int64_t)vocab;
            for (int32_t v = 0; v < vocab; ++v) o[v] += hv * row[v];
        }
    }
}
