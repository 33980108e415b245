// Online binned calibrator and the deployed stochastic pruning rule (Appendix A.4; Algorithm 1).
//
// State (one caller-provided device buffer): two first-in-first-out rings of bin indices (positive / negative
// rollouts), their histogram counts c_b^+ / c_b^-, the posterior table q_lut and the bias delta of the survival
// probability p_i = clip(kappa + delta + lambda (rho - q_i), p_min, p_max).
//
// arrol_calib_update (one block): pushes a step's labelled rollouts in index order (a full ring drops its oldest
// entry), keeps the counts in step with the rings, rebuilds q_lut with the Laplace-smoothed Bayes rule and solves
// delta by 64 bisection steps so that the expected keep rate under the buffer distribution equals kappa.  The
// table and delta are evaluated in fp64 with one rounding per operation, in a fixed order, so they are
// reproducible bit for bit.
// arrol_select_stochastic: survive iff u_i < p_i; rollouts that never reached the detection length are kept.
#include "arrol_internal.h"

namespace {

struct CalibHeader {
    int32_t B, pad;
    int64_t cap;
    int64_t head_pos, n_pos, head_neg, n_neg;
    double alpha;
    double delta;
};
static_assert(sizeof(CalibHeader) == 64, "state header layout");

struct CalibLayout {
    size_t cpos, cneg, q_lut, ring_pos, ring_neg, total;
};

CalibLayout layout_of(int B, int64_t cap) {
    CalibLayout L;
    size_t o = sizeof(CalibHeader);
    L.cpos = o; o += sizeof(int64_t) * (size_t)B;
    L.cneg = o; o += sizeof(int64_t) * (size_t)B;
    L.q_lut = o; o += sizeof(float) * (size_t)B;
    o = (o + 15) & ~(size_t)15;
    L.ring_pos = o; o += sizeof(int16_t) * (size_t)cap;
    o = (o + 15) & ~(size_t)15;
    L.ring_neg = o; o += sizeof(int16_t) * (size_t)cap;
    L.total = (o + 255) & ~(size_t)255;
    return L;
}

constexpr int CAL_THREADS = 1024;
constexpr int MAX_BINS = 1024;

__device__ __forceinline__ double survival_of(double q, double kappa_plus_delta, double lambda, double rho,
                                              double p_min, double p_max) {
    double p = __dadd_rn(kappa_plus_delta, __dmul_rn(lambda, __dsub_rn(rho, q)));
    if (p < p_min) p = p_min;
    if (p > p_max) p = p_max;
    return p;
}

__global__ void calib_init_kernel(uint8_t* state, int B, int64_t cap, double alpha, CalibLayout L) {
    CalibHeader* hd = reinterpret_cast<CalibHeader*>(state);
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        hd->B = B; hd->pad = 0; hd->cap = cap;
        hd->head_pos = hd->n_pos = hd->head_neg = hd->n_neg = 0;
        hd->alpha = alpha;
        hd->delta = 0.0;
    }
    int64_t* cpos = reinterpret_cast<int64_t*>(state + L.cpos);
    int64_t* cneg = reinterpret_cast<int64_t*>(state + L.cneg);
    float* lut = reinterpret_cast<float*>(state + L.q_lut);
    for (int b = blockIdx.x * blockDim.x + threadIdx.x; b < B; b += gridDim.x * blockDim.x) {
        cpos[b] = 0; cneg[b] = 0; lut[b] = 0.5f;    // empty buffers: prior 1/2, flat likelihoods
    }
}

__global__ void __launch_bounds__(CAL_THREADS)
calib_update_kernel(uint8_t* state, CalibLayout L, const int32_t* __restrict__ bin, const float* __restrict__ rewards,
                    const uint8_t* __restrict__ mask, int N, double kappa, double lambda, double rho, double p_min,
                    double p_max, int B_arg, int64_t cap_arg, uint32_t* d_status) {
    CalibHeader* hd = reinterpret_cast<CalibHeader*>(state);
    // The byte layout L comes from the call's (B, cap); the state must have been initialised with the same pair.
    // A mismatched or uninitialised state is left untouched and reported (uniform over the block: no barrier yet).
    if (hd->B != B_arg || hd->cap != cap_arg) {
        if (threadIdx.x == 0) atomicOr(d_status, ARROL_DEV_BAD_STATE);
        return;
    }
    int64_t* cnt[2] = {reinterpret_cast<int64_t*>(state + L.cneg), reinterpret_cast<int64_t*>(state + L.cpos)};
    int16_t* ring[2] = {reinterpret_cast<int16_t*>(state + L.ring_neg), reinterpret_cast<int16_t*>(state + L.ring_pos)};
    float* lut = reinterpret_cast<float*>(state + L.q_lut);
    const int B = hd->B;
    const int64_t cap = hd->cap;

    __shared__ int32_t warp_sum[2][32];
    __shared__ int64_t total_new[2];            // labelled rollouts pushed this call, per label
    __shared__ int64_t head0[2], n0[2];
    __shared__ int32_t hist[2][MAX_BINS];       // signed change of the counts
    __shared__ double term[MAX_BINS];           // lambda (rho - q_b)
    __shared__ double weight[MAX_BINS];         // c_b^+ + c_b^-
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;

    for (int b = threadIdx.x; b < B; b += CAL_THREADS) { hist[0][b] = 0; hist[1][b] = 0; }
    if (threadIdx.x == 0) {
        head0[0] = hd->head_neg; n0[0] = hd->n_neg; head0[1] = hd->head_pos; n0[1] = hd->n_pos;
        total_new[0] = 0; total_new[1] = 0;
    }
    __syncthreads();

    // pass 1: how many new entries per label
    {
        int32_t c[2] = {0, 0};
        for (int i = threadIdx.x; i < N; i += CAL_THREADS)
            if (!mask || mask[i]) c[rewards[i] > 0.5f ? 1 : 0] += 1;
#pragma unroll
        for (int l = 0; l < 2; ++l) {
            int32_t v = c[l];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) warp_sum[l][wid] = v;
        }
        __syncthreads();
        if (threadIdx.x < 2) {
            int64_t t = 0;
            for (int w = 0; w < CAL_THREADS / 32; ++w) t += warp_sum[threadIdx.x][w];
            total_new[threadIdx.x] = t;
        }
        __syncthreads();
    }

    // evict the oldest entries that the push displaces (read the rings before they are overwritten)
    for (int l = 0; l < 2; ++l) {
        const int64_t over = n0[l] + total_new[l] - cap;
        const int64_t evict = over <= 0 ? 0 : (over < n0[l] ? over : n0[l]);
        for (int64_t j = threadIdx.x; j < evict; j += CAL_THREADS)
            atomicSub(&hist[l][ring[l][(head0[l] + j) % cap]], 1);
    }
    __syncthreads();

    // pass 2: write the new entries in index order; entry r of m lands in slot (head + n + r) mod cap, and only the
    // last `cap` of them survive the call
    int64_t carry[2] = {0, 0};
    for (int base = 0; base < N; base += CAL_THREADS) {
        const int i = base + threadIdx.x;
        const bool on = (i < N) && (!mask || mask[i]);
        const int lab = (on && rewards[i] > 0.5f) ? 1 : 0;
        int32_t f[2] = {on && lab == 0 ? 1 : 0, on && lab == 1 ? 1 : 0};
        int32_t incl[2];
#pragma unroll
        for (int l = 0; l < 2; ++l) {
            int32_t v = f[l];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t t = __shfl_up_sync(0xffffffffu, v, o);
                if (lane >= o) v += t;
            }
            incl[l] = v;
            if (lane == 31) warp_sum[l][wid] = v;
        }
        __syncthreads();
        if (wid == 0) {
#pragma unroll
            for (int l = 0; l < 2; ++l) {
                int32_t v = warp_sum[l][lane];
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int32_t t = __shfl_up_sync(0xffffffffu, v, o);
                    if (lane >= o) v += t;
                }
                warp_sum[l][lane] = v;
            }
        }
        __syncthreads();
        if (on) {
            const int64_t r = carry[lab] + (wid ? warp_sum[lab][wid - 1] : 0) + incl[lab] - 1;
            if (r >= total_new[lab] - cap) {
                int b = bin[i];
                b = b < 0 ? 0 : (b >= B ? B - 1 : b);
                ring[lab][(head0[lab] + n0[lab] + r) % cap] = (int16_t)b;
                atomicAdd(&hist[lab][b], 1);
            }
        }
        carry[0] += warp_sum[0][31];
        carry[1] += warp_sum[1][31];
        __syncthreads();
    }

    // counts, ring bookkeeping
    for (int b = threadIdx.x; b < B; b += CAL_THREADS) {
        cnt[0][b] += hist[0][b];
        cnt[1][b] += hist[1][b];
    }
    __syncthreads();
    if (threadIdx.x < 2) {
        const int l = threadIdx.x;
        const int64_t over = n0[l] + total_new[l] - cap;
        const int64_t n1 = over > 0 ? cap : n0[l] + total_new[l];
        const int64_t h1 = over > 0 ? (head0[l] + over) % cap : head0[l];
        if (l == 0) { hd->head_neg = h1; hd->n_neg = n1; } else { hd->head_pos = h1; hd->n_pos = n1; }
        n0[l] = n1;     // totals for the table below
    }
    __syncthreads();

    // posterior table (Laplace-smoothed likelihoods, Bayes rule), fp64, one rounding per operation
    const double n_pos = (double)n0[1], n_neg = (double)n0[0];
    const double alpha = hd->alpha;
    const double prior = (n_pos + n_neg > 0.0) ? __ddiv_rn(n_pos, __dadd_rn(n_pos, n_neg)) : 0.5;
    const double den_pos = __dadd_rn(n_pos, __dmul_rn(alpha, (double)B));
    const double den_neg = __dadd_rn(n_neg, __dmul_rn(alpha, (double)B));
    for (int b = threadIdx.x; b < B; b += CAL_THREADS) {
        const double p1 = __ddiv_rn(__dadd_rn((double)cnt[1][b], alpha), den_pos);
        const double p0 = __ddiv_rn(__dadd_rn((double)cnt[0][b], alpha), den_neg);
        const double num = __dmul_rn(prior, p1);
        const double den = __dadd_rn(num, __dmul_rn(__dsub_rn(1.0, prior), p0));
        const float qb = (float)__ddiv_rn(num, den);
        lut[b] = qb;
        term[b] = __dmul_rn(lambda, __dsub_rn(rho, (double)qb));
        weight[b] = (double)(cnt[0][b] + cnt[1][b]);
    }
    __syncthreads();

    // delta: 64 bisection steps on E[p](delta) = kappa, by the first warp alone (no block barriers in the loop).  The
    // value that decides a step is the expected keep rate summed over the bins in index order, one rounding per
    // operation (so that delta agrees bit for bit with a plain loop).  Per step the lanes form the per-bin products
    // c_b p_b (all >= 0) and a butterfly sum S of them; the in-order sum differs from S by at most
    // (B + 8) 2^-53 S (both are within their standard error bounds of the exact sum), so when S / n is further from
    // kappa than four times that bound plus the rounding of the division, S / n < kappa already is the decision.
    // Only the steps near convergence (about the last twenty) need the serial chain of B additions.
    if (wid == 0) {
        __shared__ double prod[MAX_BINS];
        const double n = __dadd_rn(n_pos, n_neg);
        double delta = 0.0;
        if (n > 0.0) {                                   // uniform for the warp
            double lo = -(1.0 + lambda), hi = 1.0 + lambda;
            const double u = 1.1102230246251565e-16;     // 2^-53
            for (int it = 0; it < 64; ++it) {
                const double mid = __dmul_rn(0.5, __dadd_rn(lo, hi));
                const double base = __dadd_rn(kappa, mid);
                double part = 0.0;
                for (int b = lane; b < B; b += 32) {
                    double p = __dadd_rn(base, term[b]);
                    if (p < p_min) p = p_min;
                    if (p > p_max) p = p_max;
                    const double x = __dmul_rn(weight[b], p);
                    prod[b] = x;
                    part += x;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);   // the same bits in every lane
                const double e_tree = part / n;
                const double slack = 4.0 * ((double)(B + 8) * u * e_tree + 2.0 * u * (e_tree + kappa));
                int below;
                if (fabs(e_tree - kappa) > slack) {
                    below = e_tree < kappa ? 1 : 0;
                } else {
                    __syncwarp();
                    below = 0;
                    if (lane == 0) {
                        double e = 0.0;
#pragma unroll 8
                        for (int b = 0; b < B; ++b) e = __dadd_rn(e, prod[b]);
                        below = __ddiv_rn(e, n) < kappa ? 1 : 0;
                    }
                    below = __shfl_sync(0xffffffffu, below, 0);
                }
                __syncwarp();                            // prod is rewritten by the next step
                if (below) lo = mid; else hi = mid;
            }
            delta = __dmul_rn(0.5, __dadd_rn(lo, hi));
        }
        if (lane == 0) hd->delta = delta;
    }
}

__global__ void select_stochastic_kernel(const float* __restrict__ q, const float* __restrict__ u,
                                         const uint8_t* __restrict__ eligible, int64_t N, double kappa,
                                         const double* __restrict__ d_delta, double delta_value, double lambda,
                                         double rho, double p_min, double p_max, uint8_t* __restrict__ keep,
                                         float* __restrict__ p_out) {
    const double delta = d_delta ? *d_delta : delta_value;
    const double base = __dadd_rn(kappa, delta);
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < N; i += (int64_t)gridDim.x * blockDim.x) {
        if (eligible && !eligible[i]) {
            keep[i] = 1;
            if (p_out) p_out[i] = 1.0f;
            continue;
        }
        const double p = survival_of((double)q[i], base, lambda, rho, p_min, p_max);
        keep[i] = ((double)u[i] < p) ? 1 : 0;
        if (p_out) p_out[i] = (float)p;
    }
}

bool survival_ok(const arrol_survival* sp) {
    return sp && sp->kappa >= 0.0 && sp->kappa <= 1.0 && sp->lambda >= 0.0 && sp->rho >= 0.0 && sp->rho <= 1.0 &&
           sp->p_min >= 0.0 && sp->p_max <= 1.0 && sp->p_min <= sp->p_max;
}

}  // namespace

extern "C" size_t arrol_calib_state_bytes(int32_t B, int64_t cap) {
    if (B <= 0 || B > MAX_BINS || cap <= 0) return 0;
    return layout_of(B, cap).total;
}

extern "C" int arrol_calib_layout(int32_t B, int64_t cap, size_t* offsets6) {
    if (B <= 0 || B > MAX_BINS || cap <= 0 || !offsets6) return ARROL_ERR_INVALID_ARG;
    const CalibLayout L = layout_of(B, cap);
    offsets6[0] = L.cpos; offsets6[1] = L.cneg; offsets6[2] = L.q_lut; offsets6[3] = L.ring_pos;
    offsets6[4] = L.ring_neg; offsets6[5] = L.total;
    return ARROL_OK;
}

extern "C" int arrol_calib_init(arrol_ctx* ctx, void* state, size_t state_bytes, int32_t B, int64_t cap, double alpha,
                                void* stream) {
    if (!ctx || !state || !(alpha >= 0.0)) return ARROL_ERR_INVALID_ARG;
    if (B <= 0 || cap <= 0) return ARROL_ERR_INVALID_ARG;
    if (B > MAX_BINS) return ARROL_ERR_UNSUPPORTED;
    const CalibLayout L = layout_of(B, cap);
    if (state_bytes < L.total || !arrol_aligned(state, 16)) return ARROL_ERR_WORKSPACE;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    calib_init_kernel<<<1, 256, 0, (cudaStream_t)stream>>>(static_cast<uint8_t*>(state), B, cap, alpha, L);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

extern "C" const float* arrol_calib_q_lut(void* state, int32_t B, int64_t cap) {
    if (!state || B <= 0 || B > MAX_BINS || cap <= 0) return nullptr;
    return reinterpret_cast<const float*>(static_cast<uint8_t*>(state) + layout_of(B, cap).q_lut);
}

extern "C" const double* arrol_calib_delta(void* state) {
    if (!state) return nullptr;
    return &reinterpret_cast<CalibHeader*>(state)->delta;
}

extern "C" int arrol_calib_update(arrol_ctx* ctx, void* state, int32_t B, int64_t cap, const int32_t* bin,
                                  const float* rewards, const uint8_t* mask, int32_t N, const arrol_survival* sp,
                                  void* stream) {
    if (!ctx || !state || N < 0 || !survival_ok(sp)) return ARROL_ERR_INVALID_ARG;
    if (B <= 0 || cap <= 0) return ARROL_ERR_INVALID_ARG;
    if (B > MAX_BINS) return ARROL_ERR_UNSUPPORTED;
    if (N > 0 && (!bin || !rewards)) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    calib_update_kernel<<<1, CAL_THREADS, 0, (cudaStream_t)stream>>>(static_cast<uint8_t*>(state), layout_of(B, cap), bin,
                                                                  rewards, mask, N, sp->kappa, sp->lambda, sp->rho,
                                                                  sp->p_min, sp->p_max, B, cap, ctx->d_status);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

extern "C" int arrol_select_stochastic(arrol_ctx* ctx, const float* q, const float* u, const uint8_t* eligible,
                                       int64_t N, const arrol_survival* sp, const double* d_delta, double delta,
                                       uint8_t* keep, float* p_out, void* stream) {
    if (!ctx || N < 0 || !survival_ok(sp)) return ARROL_ERR_INVALID_ARG;
    if (N == 0) return ARROL_OK;
    if (!q || !u || !keep) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    int64_t blocks = (N + 255) / 256;
    if (blocks > (int64_t)ctx->sm_count * 8) blocks = (int64_t)ctx->sm_count * 8;
    select_stochastic_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
        q, u, eligible, N, sp->kappa, d_delta, delta, sp->lambda, sp->rho, sp->p_min, sp->p_max, keep, p_out);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
