/*
 * CPU oracle for the prune-and-rebatch path of online rollout pruning.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what each
 * step of the path computes, in fp64, written from the paper's definitions.  It
 * shares no code with the CUDA library and is never used by it: only the tests,
 * the smoke check and the bench's CPU-baseline leg call it.
 *
 * Every function takes host pointers.  Floating inputs carry a dtype code:
 *   0 = IEEE binary32, 1 = bfloat16 stored as its 16-bit pattern, 2 = binary64.
 * Values are widened to double exactly and all arithmetic is double, one IEEE
 * operation per source operation (compile with -ffp-contract=off).
 *
 * Parity pins: every function below is pinned by the CPU test-suite against
 * closed forms, exact rational arithmetic, brute force or a library routine;
 * none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORA_F32 = 0, ORA_BF16 = 1, ORA_F64 = 2 };

static double load_as_double(const void* base, int dtype, int64_t i) {
    if (dtype == ORA_F32) return (double)((const float*)base)[i];
    if (dtype == ORA_F64) return ((const double*)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16; /* bf16 = top half of a binary32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---------------------------------------------------------------------------------------------
 * Quality head (Section 4.2, "Quality Score Prediction"): a small head on the policy's hidden
 * representation of the partial rollout gives one scalar score s_i.
 *   h == 0 : s = sum_k w[k] x[k] + b                                   (linear head)
 *   h  > 0 : u_j = sum_k W1[j,k] x[k] + b1[j];  g_j = u_j/2 (1 + erf(u_j / sqrt 2));
 *            s = sum_j w2[j] g_j + b2                                   (2-layer MLP, exact GELU)
 * x is row row_index[i] (or row i when row_index is NULL) of `hidden`, rows row_stride apart.
 * Sums run in index order.  Null bias pointers mean zero.
 * --------------------------------------------------------------------------------------------- */
int oracle_head_score(const void* hidden, int dtype, int64_t row_stride, const int64_t* row_index,
                      int N, int d, int h, const void* W1, const void* b1, const void* w2,
                      const void* b2, double* score) {
    if (N < 0 || d <= 0 || h < 0) return -1;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) {
        int64_t row = row_index ? row_index[i] : (int64_t)i;
        int64_t x0 = row * row_stride;
        if (h == 0) {
            double s = 0.0;
            for (int k = 0; k < d; ++k)
                s = s + load_as_double(W1, dtype, k) * load_as_double(hidden, dtype, x0 + k);
            if (b1) s = s + load_as_double(b1, dtype, 0);
            score[i] = s;
        } else {
            double s = 0.0;
            for (int j = 0; j < h; ++j) {
                double u = 0.0;
                for (int k = 0; k < d; ++k)
                    u = u + load_as_double(W1, dtype, (int64_t)j * d + k) *
                                load_as_double(hidden, dtype, x0 + k);
                if (b1) u = u + load_as_double(b1, dtype, j);
                double g = 0.5 * u * (1.0 + erf(u / sqrt(2.0)));
                s = s + load_as_double(w2, dtype, j) * g;
            }
            if (b2) s = s + load_as_double(b2, dtype, 0);
            score[i] = s;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Score normalisation and binned posterior lookup (Appendix A.4):
 *   s' = sigmoid(s) in [0,1];  b(s') = min(B-1, floor(B s'));  q = q_lut[b]  (q = s' if no table).
 * --------------------------------------------------------------------------------------------- */
int oracle_bin_index(double sprime, int B) {
    int b = (int)floor((double)B * sprime);
    if (b > B - 1) b = B - 1;
    if (b < 0) b = 0;
    return b;
}

void oracle_prob_map(const double* score, int N, int B, const float* q_lut, double* prob,
                     int32_t* bin, double* q) {
    for (int i = 0; i < N; ++i) {
        double sp = 1.0 / (1.0 + exp(-score[i]));
        prob[i] = sp;
        int b = oracle_bin_index(sp, B > 0 ? B : 1);
        if (bin) bin[i] = b;
        q[i] = (q_lut && B > 0) ? (double)q_lut[b] : sp;
    }
}

/* Histogram counts of the positive / negative buffers (Appendix A.4, Eq. "count"):
 *   c_b^+ = #{k : b(s_k^+) = b},  c_b^- = #{k : b(s_k^-) = b}. */
void oracle_calib_counts(const double* sprime, const uint8_t* y, int64_t n, int B, int64_t* cpos,
                         int64_t* cneg) {
    for (int b = 0; b < B; ++b) cpos[b] = cneg[b] = 0;
    for (int64_t k = 0; k < n; ++k) {
        int b = oracle_bin_index(sprime[k], B);
        if (y[k]) cpos[b] += 1; else cneg[b] += 1;
    }
}

/* Laplace-smoothed class-conditional likelihoods and Bayes posterior per bin (Appendix A.4):
 *   P(b|1) = (c_b^+ + alpha) / (n^+ + alpha B),  P(b|0) = (c_b^- + alpha) / (n^- + alpha B),
 *   q_b = pi P(b|1) / (pi P(b|1) + (1-pi) P(b|0)),  pi = n^+ / (n^+ + n^-)  (0.5 if both empty).
 * q64 receives the double values, q32 the same rounded once to binary32 (either may be NULL). */
void oracle_build_q_lut(const int64_t* cpos, const int64_t* cneg, int B, double alpha, double* q64,
                        float* q32) {
    double npos = 0.0, nneg = 0.0;
    for (int b = 0; b < B; ++b) { npos += (double)cpos[b]; nneg += (double)cneg[b]; }
    double pi = (npos + nneg > 0.0) ? npos / (npos + nneg) : 0.5;
    for (int b = 0; b < B; ++b) {
        double p1 = ((double)cpos[b] + alpha) / (npos + alpha * (double)B);
        double p0 = ((double)cneg[b] + alpha) / (nneg + alpha * (double)B);
        double qb = pi * p1 / (pi * p1 + (1.0 - pi) * p0);
        if (q64) q64[b] = qb;
        if (q32) q32[b] = (float)qb;
    }
}

/* ---------------------------------------------------------------------------------------------
 * Per-group correctness-balancing selection (Section 4.1, Theorem 1's pruning rule
 *   j^ = argmin_j | mu_{-j} - rho |,  mu_{-j} = mean of q over the group without j),
 * applied repeatedly until exactly K rollouts of each group of G remain.
 * With n = |S| members left and Sigma their sum, |mu_{S\j} - rho| = |q_j - tau| / (n-1) with
 * tau = Sigma - rho (n-1): the same argmin without a division.  Among equal keys the rollout
 * with the HIGHEST index is removed, so of two tied rollouts the lower index survives.
 * Sigma starts as the index-order sum and is updated by subtracting the removed q.
 * removal_order (optional) receives, per group, the G-K removed in-group indices in order.
 * --------------------------------------------------------------------------------------------- */
int oracle_select(const float* q, int P, int G, int K, double rho, uint8_t* keep,
                  int32_t* removal_order) {
    if (P < 0 || G < 1 || K < 1 || K > G) return -1;
    for (int p = 0; p < P; ++p) {
        const float* qg = q + (int64_t)p * G;
        uint8_t* kg = keep + (int64_t)p * G;
        double sigma = 0.0;
        for (int j = 0; j < G; ++j) { kg[j] = 1; sigma = sigma + (double)qg[j]; }
        int n = G;
        while (n > K) {
            double prod = rho * (double)(n - 1);
            double tau = sigma - prod;
            int best = -1;
            double best_key = 0.0;
            for (int j = 0; j < G; ++j) {
                if (!kg[j]) continue;
                double key = fabs((double)qg[j] - tau);
                if (best < 0 || key <= best_key) { best = j; best_key = key; } /* <= : the last tied index wins */
            }
            kg[best] = 0;
            sigma = sigma - (double)qg[best];
            if (removal_order) removal_order[(int64_t)p * (G - K) + (G - n)] = best;
            n -= 1;
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------------------------------
 * Filter + re-batch (Section 4.3 (ii); Algorithm 1, frontend "Filter pruned rollouts, rebatch").
 * Survivors keep their original order.  cu_seqlens is the exclusive prefix sum of the survivors'
 * lengths; num = {S, T}.
 * --------------------------------------------------------------------------------------------- */
void oracle_survivor_scan(const uint8_t* keep, const int32_t* lengths, int N, int32_t* survivor_idx,
                          int64_t* cu_seqlens, int64_t* num) {
    int64_t S = 0, T = 0;
    cu_seqlens[0] = 0;
    for (int i = 0; i < N; ++i) {
        if (!keep[i]) continue;
        survivor_idx[S] = i;
        T += (int64_t)lengths[i];
        S += 1;
        cu_seqlens[S] = T;
    }
    num[0] = S;
    num[1] = T;
}

/* dst row cu[s]+t  <-  src row src_tok_off[idx[s]]+t, for token ids and (optionally) row payloads. */
void oracle_gather(const int32_t* survivor_idx, const int64_t* cu_seqlens, int64_t S,
                   const int64_t* src_tok_off, const int32_t* src_tokens, const uint8_t* src_rows,
                   int64_t row_bytes, int32_t* dst_tokens, uint8_t* dst_rows, int32_t* tok_seq) {
    for (int64_t s = 0; s < S; ++s) {
        int64_t len = cu_seqlens[s + 1] - cu_seqlens[s];
        int64_t src0 = src_tok_off[survivor_idx[s]];
        for (int64_t t = 0; t < len; ++t) {
            int64_t dr = cu_seqlens[s] + t;
            if (dst_tokens) dst_tokens[dr] = src_tokens[src0 + t];
            if (tok_seq) tok_seq[dr] = (int32_t)s;
            if (dst_rows)
                for (int64_t b = 0; b < row_bytes; ++b)
                    dst_rows[dr * row_bytes + b] = src_rows[(src0 + t) * row_bytes + b];
        }
    }
}

/* ---------------------------------------------------------------------------------------------
 * Group-relative advantage (Section 3) evaluated on the survivors of each group:
 *   A_i = (R_i - mean) / (std + eps),  mean and std over the kept rollouts of i's group,
 *   std = sqrt( sum (R - mean)^2 / (n - ddof) ).
 * A group whose kept rewards are all equal has a zero numerator, hence A = 0 (the degenerate
 * all-0 / all-1 case).  A group with n - ddof <= 0 also yields 0.  adv is indexed by survivor
 * ordinal (same order as survivor_idx).
 * --------------------------------------------------------------------------------------------- */
void oracle_advantages(const float* rewards, const uint8_t* keep, int N, int G, double eps, int ddof,
                       double* adv) {
    int64_t s = 0;
    for (int g0 = 0; g0 < N; g0 += G) {
        int g1 = g0 + G < N ? g0 + G : N;
        int n = 0;
        double sum = 0.0;
        for (int i = g0; i < g1; ++i)
            if (keep[i]) { sum = sum + (double)rewards[i]; n += 1; }
        if (n == 0) continue;
        double mean = sum / (double)n;
        double ss = 0.0;
        for (int i = g0; i < g1; ++i)
            if (keep[i]) { double dv = (double)rewards[i] - mean; ss = ss + dv * dv; }
        double sd = (n - ddof > 0) ? sqrt(ss / (double)(n - ddof)) : 0.0;
        for (int i = g0; i < g1; ++i)
            if (keep[i]) {
                double num = (double)rewards[i] - mean;
                adv[s++] = (n - ddof > 0) ? num / (sd + eps) : 0.0;
            }
    }
}

/* ---------------------------------------------------------------------------------------------
 * Selected-token log-probability (Section 3: log pi_theta(o_t | o_<t), the numerator of the
 * importance ratio) from the lm_head:  z_v = inv_temp * sum_k H[t,k] W[v,k],
 *   lse = m + log sum_v exp(z_v - m),  m = max_v z_v,   logp_t = z_{y_t} - lse.
 * Two passes over the full vocabulary.  targets[t] < 0 marks an ignored position: logp = 0.
 * `rows` (optional) lists which token rows of H to evaluate; outputs are indexed by position in
 * that list.  zbuf is per-thread scratch of V doubles, allocated here.
 * --------------------------------------------------------------------------------------------- */
int oracle_token_logprob(const void* hidden, const void* W, int dtype, const int32_t* targets,
                         const int64_t* rows, int64_t n_rows, int d, int V, double inv_temp,
                         double* logp, double* lse) {
    int err = 0;
#pragma omp parallel
    {
        double* z = (double*)malloc(sizeof(double) * (size_t)V);
        if (!z) {
#pragma omp atomic write
            err = -1;
        }
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < n_rows; ++r) {
            if (!z) continue;
            int64_t t = rows ? rows[r] : r;
            int32_t y = targets[t];
            for (int v = 0; v < V; ++v) {
                double acc = 0.0;
                for (int k = 0; k < d; ++k)
                    acc = acc + load_as_double(hidden, dtype, t * (int64_t)d + k) *
                                    load_as_double(W, dtype, (int64_t)v * d + k);
                z[v] = acc * inv_temp;
            }
            double m = z[0];
            for (int v = 1; v < V; ++v) if (z[v] > m) m = z[v];
            double sum = 0.0;
            for (int v = 0; v < V; ++v) sum = sum + exp(z[v] - m);
            double l = m + log(sum);
            if (lse) lse[r] = l;
            logp[r] = (y >= 0 && y < V) ? z[y] - l : 0.0;
        }
        free(z);
    }
    return err;
}

/* ---------------------------------------------------------------------------------------------
 * Deployed stochastic pruning rule (Appendix A.4, Eq. "survival"; Algorithm 1, backend).
 *
 * Sliding buffers: positives and negatives are kept in two first-in-first-out buffers of `cap` normalised
 * scores each; pushing into a full buffer drops its oldest entry.  The histogram counts c_b^+ / c_b^- are the
 * counts over what the buffers hold (Eq. "count").
 * buf_pos / buf_neg: [cap] ring storage of s', head_* = index of the oldest entry, n_* = entries held.
 * --------------------------------------------------------------------------------------------- */
void oracle_buffer_push(double* buf_pos, int64_t* head_pos, int64_t* n_pos, double* buf_neg, int64_t* head_neg,
                        int64_t* n_neg, int64_t cap, const double* sprime, const uint8_t* y, int64_t n) {
    for (int64_t k = 0; k < n; ++k) {
        double* buf = y[k] ? buf_pos : buf_neg;
        int64_t* head = y[k] ? head_pos : head_neg;
        int64_t* cnt = y[k] ? n_pos : n_neg;
        if (*cnt < cap) {
            buf[(*head + *cnt) % cap] = sprime[k];
            *cnt += 1;
        } else {
            buf[*head] = sprime[k];          /* overwrite the oldest, which becomes the newest */
            *head = (*head + 1) % cap;
        }
    }
}

/* Survival probability p = clip(kappa + delta + lambda (rho - q), p_min, p_max). */
static double survival_of(double q, double kappa, double delta, double lambda, double rho, double p_min,
                          double p_max) {
    double p = kappa + delta;
    p = p + lambda * (rho - q);
    if (p < p_min) p = p_min;
    if (p > p_max) p = p_max;
    return p;
}

/* delta by bisection so that the expected keep rate under the buffer distribution equals kappa:
 *   E[p] = sum_b w_b clip(kappa + delta + lambda (rho - q_b), p_min, p_max) = kappa,
 *   w_b = (c_b^+ + c_b^-) / n   (every buffered rollout counts once; q_b is the posterior of its bin).
 * E[p] is non-decreasing in delta.  Bracket [-(1 + lambda), 1 + lambda], `iters` halvings (64 in the library);
 * the midpoint moves up when E[p] < kappa.  Empty buffers give delta = 0.  Sums run over bins in index order. */
double oracle_solve_delta(const int64_t* cpos, const int64_t* cneg, const float* q_lut, int B, double kappa,
                          double lambda, double rho, double p_min, double p_max, int iters) {
    double n = 0.0;
    for (int b = 0; b < B; ++b) n = n + (double)(cpos[b] + cneg[b]);
    if (!(n > 0.0)) return 0.0;
    double lo = -(1.0 + lambda), hi = 1.0 + lambda;
    for (int it = 0; it < iters; ++it) {
        double mid = 0.5 * (lo + hi);
        double e = 0.0;
        for (int b = 0; b < B; ++b) {
            double wb = (double)(cpos[b] + cneg[b]);
            e = e + wb * survival_of((double)q_lut[b], kappa, mid, lambda, rho, p_min, p_max);
        }
        e = e / n;
        if (e < kappa) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

/* Per-rollout decision: a rollout that has reached the detection length (eligible) survives iff u < p_i;
 * a rollout that ended earlier is never evaluated and is kept.  p (optional) receives p_i (1 for the
 * ineligible). u in [0,1) are the uniforms drawn for this step, passed in. */
void oracle_select_stochastic(const float* q, const float* u, const uint8_t* eligible, int64_t N, double kappa,
                              double delta, double lambda, double rho, double p_min, double p_max,
                              uint8_t* keep, double* p) {
    for (int64_t i = 0; i < N; ++i) {
        if (eligible && !eligible[i]) {
            keep[i] = 1;
            if (p) p[i] = 1.0;
            continue;
        }
        double pi = survival_of((double)q[i], kappa, delta, lambda, rho, p_min, p_max);
        if (p) p[i] = pi;
        keep[i] = ((double)u[i] < pi) ? 1 : 0;
    }
}
