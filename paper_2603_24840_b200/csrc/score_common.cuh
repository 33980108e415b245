// Probability map shared by the scoring kernels (Appendix A.4).
#pragma once
#include <stdint.h>

// s -> s' = sigmoid(s), b = min(B-1, floor(B s')), q = q_lut[b]
__device__ __forceinline__ float probability_map(float s, int i, int B, const float* __restrict__ q_lut,
                                                 float* score, float* prob, int32_t* bin, float* q) {
    float sp = 1.0f / (1.0f + expf(-s));
    int b = 0;
    if (B > 0) {
        b = (int)floorf((float)B * sp);
        b = min(max(b, 0), B - 1);
    }
    score[i] = s;
    prob[i] = sp;
    if (bin) bin[i] = b;
    const float qv = (q_lut != nullptr) ? __ldg(q_lut + b) : sp;
    q[i] = qv;
    return qv;
}
