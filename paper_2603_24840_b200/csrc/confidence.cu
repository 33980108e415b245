// arrol_trace_confidence: trace-level confidence from per-token confidences (Section 3 "Trace Confidence"):
//   mode 0: mean of H_t over the trace;  mode 1: minimum over the trace of the sliding-window mean of H_t.
// One block per trace.  Traces of up to PREFIX_MAX tokens: the block builds the fp64 inclusive prefix sums of H in
// shared memory (each thread a contiguous run, block scan of the run totals) and every window sum is a difference of
// two of them.  Longer traces: every thread owns a contiguous run of window start positions, sums its first window
// directly and then slides it (add the entering token, drop the leaving one) in double precision.  The block takes
// the minimum.  A trace shorter than the window has one window, the whole trace.
#include "arrol_internal.h"

namespace {

constexpr int TC_THREADS = 256;
constexpr int PREFIX_MAX = 8192;       // tokens whose prefix sums fit the block's 64 KB of shared memory

__global__ void __launch_bounds__(TC_THREADS)
trace_confidence_kernel(const float* __restrict__ H, const int64_t* __restrict__ cu_seqlens,
                        const int64_t* __restrict__ d_num, int window, int mode, float* __restrict__ out) {
    __shared__ double sh[TC_THREADS / 32];
    __shared__ double run_base[TC_THREADS / 32];
    extern __shared__ double prefix[];      // [PREFIX_MAX]
    const int64_t S = d_num[0];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int64_t s = blockIdx.x; s < S; s += gridDim.x) {
        const int64_t t0 = cu_seqlens[s], len = cu_seqlens[s + 1] - t0;
        if (len <= 0) {
            if (threadIdx.x == 0) out[s] = 0.f;
            continue;
        }
        const float* h = H + t0;
        double v;
        if (mode == 0) {
            v = 0.0;
            for (int64_t t = threadIdx.x; t < len; t += TC_THREADS) v += (double)h[t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        } else if (len <= PREFIX_MAX) {
            const int w = (int)(len < window ? len : (int64_t)window);
            const int n = (int)len;
            const int per = (n + TC_THREADS - 1) / TC_THREADS;
            const int r0 = min(n, (int)threadIdx.x * per), r1 = min(n, r0 + per);
            double run = 0.0;
            for (int t = r0; t < r1; ++t) { run += (double)h[t]; prefix[t] = run; }    // prefix inside the run
            // exclusive scan of the run totals: inside each warp by shuffles, then over the warp totals
            double incl = run;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double up = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += up;
            }
            if (lane == 31) run_base[wid] = incl;
            __syncthreads();
            double base = incl - run;
            for (int k = 0; k < wid; ++k) base += run_base[k];
            for (int t = r0; t < r1; ++t) prefix[t] += base;
            __syncthreads();
            v = __longlong_as_double(0x7ff0000000000000LL);
            for (int a = threadIdx.x; a + w <= n; a += TC_THREADS)
                v = fmin(v, prefix[a + w - 1] - (a ? prefix[a - 1] : 0.0));
            v /= (double)w;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(0xffffffffu, v, o));
        } else {
            const int64_t w = len < window ? len : (int64_t)window;
            const int64_t n_win = len - w + 1;
            const int64_t per = (n_win + TC_THREADS - 1) / TC_THREADS;
            const int64_t a0 = (int64_t)threadIdx.x * per, a1 = a0 + per < n_win ? a0 + per : n_win;
            v = __longlong_as_double(0x7ff0000000000000LL);
            if (a0 < a1) {
                double sum = 0.0;
                for (int64_t t = 0; t < w; ++t) sum += (double)h[a0 + t];
                v = sum;
                for (int64_t a = a0 + 1; a < a1; ++a) {
                    sum += (double)h[a + w - 1] - (double)h[a - 1];
                    v = fmin(v, sum);
                }
                v /= (double)w;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(0xffffffffu, v, o));
        }
        __syncthreads();
        if (lane == 0) sh[wid] = v;
        __syncthreads();
        if (threadIdx.x == 0) {
            double r = sh[0];
            for (int i = 1; i < TC_THREADS / 32; ++i) r = mode == 0 ? r + sh[i] : fmin(r, sh[i]);
            out[s] = (float)(mode == 0 ? r / (double)len : r);
        }
    }
}

}  // namespace

extern "C" int arrol_trace_confidence(arrol_ctx* ctx, const float* token_conf, const int64_t* cu_seqlens,
                                      const int64_t* d_num, int32_t S_max, int32_t window, int32_t mode,
                                      float* trace_conf, void* stream) {
    if (!ctx || S_max < 0 || window < 1) return ARROL_ERR_INVALID_ARG;
    if (mode != 0 && mode != 1) return ARROL_ERR_UNSUPPORTED;
    if (S_max == 0) return ARROL_OK;
    if (!token_conf || !cu_seqlens || !d_num || !trace_conf) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    int blocks = S_max < ctx->sm_count * 8 ? S_max : ctx->sm_count * 8;
    const size_t smem = mode == 1 ? sizeof(double) * PREFIX_MAX : 0;
    ARROL_CUDA_OK(cudaFuncSetAttribute(trace_confidence_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)(sizeof(double) * PREFIX_MAX)));
    trace_confidence_kernel<<<blocks, TC_THREADS, smem, (cudaStream_t)stream>>>(token_conf, cu_seqlens, d_num, window,
                                                                              mode, trace_conf);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
