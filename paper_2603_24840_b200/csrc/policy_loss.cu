// arrol_policy_loss: the clipped GRPO / DAPO objective on the packed survivors (Section 3) and its gradient with
// respect to the token log-probs.
//   r = exp(logp - logp_old),  term = min(r A, clip(r, 1 - eps_low, 1 + eps_high) A),
//   loss = - sum_t w_t term_t (+ beta sum_t w_t kl_t,  kl = exp(ref - logp) - (ref - logp) - 1),
//   w_t = 1 / (S len(rollout of t))  (agg_mode 0, per-rollout token mean)  or  1 / T  (agg_mode 1, token mean).
// One thread per token; the loss is reduced in two fixed-order stages (per block, then one block over the block
// partials held in the context scratch), so it is reproducible run to run.
#include "arrol_internal.h"

namespace {

constexpr int PL_THREADS = 256;
constexpr int PL_MAX_BLOCKS = 4096;

__global__ void __launch_bounds__(PL_THREADS)
policy_loss_kernel(const float* __restrict__ logp, const float* __restrict__ logp_old,
                   const float* __restrict__ logp_ref, const float* __restrict__ tok_adv,
                   const int32_t* __restrict__ tok_seq, const int64_t* __restrict__ cu_seqlens,
                   const int64_t* __restrict__ d_num, int64_t T_max, float eps_low, float eps_high, float beta,
                   int agg_mode, float* __restrict__ grad, double* __restrict__ block_partial) {
    const int64_t S = d_num[0];
    int64_t T = d_num[1];
    if (T > T_max) T = T_max;
    const float lo = 1.0f - eps_low, hi = 1.0f + eps_high;
    double local = 0.0;
    for (int64_t t = blockIdx.x * (int64_t)PL_THREADS + threadIdx.x; t < T; t += (int64_t)gridDim.x * PL_THREADS) {
        float w;
        if (agg_mode == 0) {
            const int s = tok_seq[t];
            w = 1.0f / ((float)S * (float)(cu_seqlens[s + 1] - cu_seqlens[s]));
        } else {
            w = 1.0f / (float)T;
        }
        const float lp = logp[t];
        const float r = expf(lp - logp_old[t]);
        const float c = fminf(fmaxf(r, lo), hi);
        const float adv = tok_adv[t];
        const float a = r * adv, b = c * adv;
        float term = a <= b ? a : b;
        float g = a <= b ? -w * a : 0.0f;
        float kl = 0.f;
        if (logp_ref) {
            const float dlt = logp_ref[t] - lp;
            const float e = expf(dlt);
            kl = e - dlt - 1.0f;
            g += beta * w * (1.0f - e);
        }
        grad[t] = g;
        local += (double)w * ((double)beta * (double)kl - (double)term);
    }
    // block reduction in a fixed order
    __shared__ double warp_part[PL_THREADS / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = local;
    __syncthreads();
    if (threadIdx.x == 0) {
        double tot = 0.0;
        for (int w = 0; w < PL_THREADS / 32; ++w) tot += warp_part[w];
        block_partial[blockIdx.x] = tot;
    }
}

__global__ void policy_loss_finish_kernel(const double* __restrict__ block_partial, int n, double* __restrict__ loss) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double tot = 0.0;
        for (int i = 0; i < n; ++i) tot += block_partial[i];
        *loss = tot;
    }
}

}  // namespace

extern "C" int arrol_policy_loss(arrol_ctx* ctx, const float* logp, const float* logp_old, const float* logp_ref,
                                 const float* tok_adv, const int32_t* tok_seq, const int64_t* cu_seqlens,
                                 const int64_t* d_num, int64_t T_max, float eps_low, float eps_high, float beta,
                                 int32_t agg_mode, float* grad_logp, double* loss, void* stream) {
    if (!ctx || T_max < 0 || !(eps_low >= 0.f) || !(eps_high >= 0.f) || !(beta >= 0.f)) return ARROL_ERR_INVALID_ARG;
    if (agg_mode != 0 && agg_mode != 1) return ARROL_ERR_UNSUPPORTED;
    if (!d_num || !loss) return ARROL_ERR_INVALID_ARG;
    if (T_max > 0 && (!logp || !logp_old || !tok_adv || !grad_logp || !cu_seqlens)) return ARROL_ERR_INVALID_ARG;
    if (agg_mode == 0 && T_max > 0 && !tok_seq) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    int64_t blocks = (T_max + PL_THREADS - 1) / PL_THREADS;
    if (blocks > PL_MAX_BLOCKS) blocks = PL_MAX_BLOCKS;
    if (blocks < 1) blocks = 1;
    double* partial = reinterpret_cast<double*>(ctx->d_scratch);
    policy_loss_kernel<<<(unsigned)blocks, PL_THREADS, 0, s>>>(logp, logp_old, logp_ref, tok_adv, tok_seq, cu_seqlens,
                                                              d_num, T_max, eps_low, eps_high, beta, agg_mode,
                                                              grad_logp, partial);
    policy_loss_finish_kernel<<<1, 32, 0, s>>>(partial, (int)blocks, loss);
    ctx->launches += 2;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
