/*
 * CPU oracle, quality-head training step (Section 4.2 "Quality Score Prediction"; Section 4.3 (iii)):
 * the head is trained on the fly with a cross-entropy loss on (score, final reward); gradients flow into the
 * head only (the hidden states are inputs).  TEST INFRASTRUCTURE ONLY (see arrol_oracle.c).
 *
 * With one scalar logit s_i per rollout and label y_i in {0,1} the cross-entropy is the binary one:
 *     loss = (1/n) sum_i [ log(1 + exp(s_i)) - y_i s_i ],   d loss / d s_i = (sigmoid(s_i) - y_i) / n,
 * over the n rollouts with mask[i] != 0 (all when mask is NULL).
 *   linear head  s = w.x + b:                dw = sum_i ds_i x_i,  db = sum_i ds_i
 *   MLP head     s = w2.gelu(W1 x + b1) + b2: dw2_j = sum_i ds_i g_ij,  db2 = sum_i ds_i,
 *                du_ij = ds_i w2_j gelu'(u_ij),  gelu'(u) = Phi(u) + u phi(u),
 *                dW1_jk = sum_i du_ij x_ik,  db1_j = sum_i du_ij.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double widen_h(const void* base, int dtype, int64_t i) {
    if (dtype == 0) return (double)((const float*)base)[i];
    if (dtype == 2) return ((const double*)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int oracle_head_bce_grad(const void* hidden, int dtype, int64_t row_stride, const int64_t* row_index, int N, int d,
                         int h, const void* W1, const void* b1, const void* w2, const void* b2, const uint8_t* y,
                         const uint8_t* mask, double* loss_out, double* dW1, double* db1, double* dw2, double* db2) {
    int n = 0;
    for (int i = 0; i < N; ++i) if (!mask || mask[i]) n += 1;
    const int hh = h > 0 ? h : 1;
    for (int64_t i = 0; i < (int64_t)hh * d; ++i) dW1[i] = 0.0;
    for (int j = 0; j < hh; ++j) db1[j] = 0.0;
    if (h > 0) { for (int j = 0; j < h; ++j) dw2[j] = 0.0; db2[0] = 0.0; }
    *loss_out = 0.0;
    if (n == 0) return 0;
    double* u = (double*)malloc(sizeof(double) * (size_t)hh);
    if (!u) return -1;
    double loss = 0.0;
    for (int i = 0; i < N; ++i) {
        if (mask && !mask[i]) continue;
        const int64_t x0 = (row_index ? row_index[i] : (int64_t)i) * row_stride;
        double s = 0.0;
        if (h == 0) {
            for (int k = 0; k < d; ++k) s = s + widen_h(W1, dtype, k) * widen_h(hidden, dtype, x0 + k);
            if (b1) s = s + widen_h(b1, dtype, 0);
        } else {
            for (int j = 0; j < h; ++j) {
                double a = 0.0;
                for (int k = 0; k < d; ++k) a = a + widen_h(W1, dtype, (int64_t)j * d + k) * widen_h(hidden, dtype, x0 + k);
                if (b1) a = a + widen_h(b1, dtype, j);
                u[j] = a;
                s = s + widen_h(w2, dtype, j) * (0.5 * a * (1.0 + erf(a / sqrt(2.0))));
            }
            if (b2) s = s + widen_h(b2, dtype, 0);
        }
        const double yi = y[i] ? 1.0 : 0.0;
        /* log(1 + exp(s)) evaluated without overflow */
        const double softplus = s > 0.0 ? s + log1p(exp(-s)) : log1p(exp(s));
        loss = loss + (softplus - yi * s) / (double)n;
        const double ds = (1.0 / (1.0 + exp(-s)) - yi) / (double)n;
        if (h == 0) {
            for (int k = 0; k < d; ++k) dW1[k] = dW1[k] + ds * widen_h(hidden, dtype, x0 + k);
            db1[0] = db1[0] + ds;
        } else {
            db2[0] = db2[0] + ds;
            for (int j = 0; j < h; ++j) {
                const double a = u[j];
                const double cdf = 0.5 * (1.0 + erf(a / sqrt(2.0)));
                const double pdf = exp(-0.5 * a * a) / sqrt(2.0 * 3.14159265358979323846);
                dw2[j] = dw2[j] + ds * (a * cdf);
                const double du = ds * widen_h(w2, dtype, j) * (cdf + a * pdf);
                db1[j] = db1[j] + du;
                for (int k = 0; k < d; ++k) dW1[(int64_t)j * d + k] = dW1[(int64_t)j * d + k] + du * widen_h(hidden, dtype, x0 + k);
            }
        }
    }
    free(u);
    *loss_out = loss;
    return 0;
}
