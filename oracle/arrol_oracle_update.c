/*
 * CPU oracle, policy-update half: the clipped GRPO / DAPO objective on the survivors and the backward of the
 * lm_head log-prob.  TEST INFRASTRUCTURE ONLY (see arrol_oracle.c); plain fp64 loops, no code shared with
 * the CUDA library.  Pinned by finite differences, closed forms and torch autograd in float64.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double widen(const void* base, int dtype, int64_t i) {
    if (dtype == 0) return (double)((const float*)base)[i];
    if (dtype == 2) return ((const double*)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* ---------------------------------------------------------------------------------------------
 * Clipped objective (Section 3):  per token
 *     r = exp(logp - logp_old),   term = min( r A, clip(r, 1 - eps_low, 1 + eps_high) A ),
 * A the group-relative advantage of the token's rollout.  The loss is minus the objective:
 *     agg_mode 0 (GRPO):  loss = -(1/S) sum_s (1/len_s) sum_{t in s} term_t     (rollouts of zero length are skipped)
 *     agg_mode 1 (DAPO):  loss = -(1/T) sum_t term_t
 * plus beta times the same mean of the per-token KL estimate  kl = exp(ref - logp) - (ref - logp) - 1
 * when logp_ref is given.  grad[t] = d loss / d logp[t]:
 *     d term / d logp = r A  if  r A <= clip(r) A  (the unclipped branch is the minimum), else 0.
 * --------------------------------------------------------------------------------------------- */
void oracle_policy_loss(const double* logp, const double* logp_old, const double* logp_ref, const double* tok_adv,
                        const int64_t* cu_seqlens, int64_t S, double eps_low, double eps_high, double beta,
                        int agg_mode, double* loss_out, double* grad) {
    const int64_t T = cu_seqlens[S];
    double loss = 0.0;
    for (int64_t s = 0; s < S; ++s) {
        const int64_t t0 = cu_seqlens[s], t1 = cu_seqlens[s + 1];
        if (t1 <= t0) continue;
        const double w = agg_mode == 0 ? 1.0 / ((double)S * (double)(t1 - t0)) : 1.0 / (double)T;
        for (int64_t t = t0; t < t1; ++t) {
            const double r = exp(logp[t] - logp_old[t]);
            double c = r;
            if (c < 1.0 - eps_low) c = 1.0 - eps_low;
            if (c > 1.0 + eps_high) c = 1.0 + eps_high;
            const double a = r * tok_adv[t], b = c * tok_adv[t];
            const double term = a <= b ? a : b;
            double g = a <= b ? -w * a : 0.0;
            loss = loss - w * term;
            if (logp_ref) {
                const double dlt = logp_ref[t] - logp[t];
                loss = loss + beta * w * (exp(dlt) - dlt - 1.0);
                g = g + beta * w * (1.0 - exp(dlt));
            }
            grad[t] = g;
        }
    }
    *loss_out = loss;
}

/* ---------------------------------------------------------------------------------------------
 * Backward of the selected-token log-prob through the lm_head.  With z = inv_temp H W^T and
 * logp_t = z_{t,y_t} - lse_t:
 *     dz_{t,v} = g_t inv_temp ( [v = y_t] - exp(z_{t,v} - lse_t) ),   dH = dz W,   dW = dz^T H.
 * Positions with y_t < 0 (ignored) or y_t >= V contribute nothing.  dH [T,d], dW [V,d] in double.
 * --------------------------------------------------------------------------------------------- */
int oracle_lm_head_backward(const void* hidden, const void* W, int dtype, const int32_t* targets, const double* g,
                            int64_t T, int d, int V, double inv_temp, double* dH, double* dW) {
    double* z = (double*)malloc(sizeof(double) * (size_t)V);
    if (!z) return -1;
    for (int64_t i = 0; i < (int64_t)V * d; ++i) dW[i] = 0.0;
    for (int64_t t = 0; t < T; ++t) {
        for (int k = 0; k < d; ++k) dH[t * d + k] = 0.0;
        const int32_t y = targets[t];
        if (y < 0 || y >= V) continue;
        double m = -INFINITY;
        for (int v = 0; v < V; ++v) {
            double acc = 0.0;
            for (int k = 0; k < d; ++k) acc = acc + widen(hidden, dtype, t * (int64_t)d + k) * widen(W, dtype, (int64_t)v * d + k);
            z[v] = acc * inv_temp;
            if (z[v] > m) m = z[v];
        }
        double sum = 0.0;
        for (int v = 0; v < V; ++v) sum = sum + exp(z[v] - m);
        const double lse = m + log(sum);
        for (int v = 0; v < V; ++v) {
            const double dz = g[t] * inv_temp * ((v == y ? 1.0 : 0.0) - exp(z[v] - lse));
            for (int k = 0; k < d; ++k) {
                dH[t * d + k] = dH[t * d + k] + dz * widen(W, dtype, (int64_t)v * d + k);
                dW[(int64_t)v * d + k] = dW[(int64_t)v * d + k] + dz * widen(hidden, dtype, t * (int64_t)d + k);
            }
        }
    }
    free(z);
    return 0;
}
