/*
 * CPU oracle: trace confidence (Section 3 "Trace Confidence").  TEST INFRASTRUCTURE ONLY (see arrol_oracle.c).
 *   token confidence   H_t = - sum_{j=1..V} log P_t(j),  P_t = softmax of the position's logits
 *   window confidence  H_w = mean of H_t over a sliding window of `window` tokens
 *   trace score        mode 0: mean of H_t over the trace;  mode 1: minimum window confidence over the trace;
 *                      mode 2: average of the bottom 10 % of the window confidences: the windows are all
 *                      len - w + 1 sliding positions, the k = ceil(0.1 * #windows) smallest H_w are averaged
 *                      (at least one window, so a trace with fewer than ten windows gives its minimum)
 * A trace shorter than the window has one window, the whole trace.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double widen_c(const void* base, int dtype, int64_t i) {
    if (dtype == 0) return (double)((const float*)base)[i];
    if (dtype == 2) return ((const double*)base)[i];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[i]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

int oracle_token_confidence(const void* hidden, const void* W, int dtype, const int64_t* rows, int64_t n_rows, int d,
                            int V, double inv_temp, double* conf) {
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
            const int64_t t = rows ? rows[r] : r;
            double m = -INFINITY;
            for (int v = 0; v < V; ++v) {
                double acc = 0.0;
                for (int k = 0; k < d; ++k) acc = acc + widen_c(hidden, dtype, t * (int64_t)d + k) * widen_c(W, dtype, (int64_t)v * d + k);
                z[v] = acc * inv_temp;
                if (z[v] > m) m = z[v];
            }
            double sum = 0.0;
            for (int v = 0; v < V; ++v) sum = sum + exp(z[v] - m);
            const double lse = m + log(sum);
            double h = 0.0;
            for (int v = 0; v < V; ++v) h = h - (z[v] - lse);
            conf[r] = h;
        }
        free(z);
    }
    return err;
}

static int cmp_double(const void* a, const void* b) {
    const double x = *(const double*)a, y = *(const double*)b;
    return (x > y) - (x < y);
}

void oracle_trace_confidence(const double* H, const int64_t* cu_seqlens, int64_t S, int window, int mode, double* out) {
    for (int64_t s = 0; s < S; ++s) {
        const int64_t t0 = cu_seqlens[s], len = cu_seqlens[s + 1] - t0;
        if (len <= 0) { out[s] = 0.0; continue; }
        if (mode == 0) {
            double sum = 0.0;
            for (int64_t t = 0; t < len; ++t) sum = sum + H[t0 + t];
            out[s] = sum / (double)len;
        } else if (mode == 2) {
            const int64_t w = len < window ? len : window;
            const int64_t n_win = len - w + 1;
            double* hw = (double*)malloc(sizeof(double) * (size_t)n_win);
            if (!hw) { out[s] = NAN; continue; }
            for (int64_t a = 0; a < n_win; ++a) {
                double sum = 0.0;
                for (int64_t t = 0; t < w; ++t) sum = sum + H[t0 + a + t];
                hw[a] = sum / (double)w;
            }
            qsort(hw, (size_t)n_win, sizeof(double), cmp_double);
            const int64_t k = (n_win + 9) / 10;
            double sum = 0.0;
            for (int64_t a = 0; a < k; ++a) sum = sum + hw[a];
            out[s] = sum / (double)k;
            free(hw);
        } else {
            const int64_t w = len < window ? len : window;
            double best = INFINITY;
            for (int64_t a = 0; a + w <= len; ++a) {
                double sum = 0.0;
                for (int64_t t = 0; t < w; ++t) sum = sum + H[t0 + a + t];
                const double mean = sum / (double)w;
                if (mean < best) best = mean;
            }
            out[s] = best;
        }
    }
}
