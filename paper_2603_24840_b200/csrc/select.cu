// arrol_select: per-group correctness-balancing selection (Section 4.1; Theorem 1's rule
// j^ = argmin_j |mu_{-j} - rho| applied G - K times per group).
//
// One group occupies a segment of `seg` = next power of two >= G lanes; 32 / seg groups share a warp.  Every
// lane holds one rollout's q in double.  Each round: tau = Sigma - rho (n - 1) (one rounding per operation, no
// fused multiply-add), key = |q - tau|, a segmented shuffle arg-min on (key, index) where of equal keys the
// higher index wins, then the winner leaves the group and Sigma -= q_winner.  Sigma starts as the index-order
// sum, built with broadcasts so that every lane of the segment adds the same values in the same order.
#include "arrol_internal.h"

namespace {

__device__ __forceinline__ double shfl_double(double v, int src_lane, int width) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src_lane, width);
    hi = __shfl_sync(0xffffffffu, hi, src_lane, width);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_xor_double(double v, int mask, int width) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, mask, width);
    hi = __shfl_xor_sync(0xffffffffu, hi, mask, width);
    return __hiloint2double(hi, lo);
}

__global__ void __launch_bounds__(128)
select_kernel(const float* __restrict__ q, int P, int G, int K, double rho, int seg, uint8_t* __restrict__ keep) {
    pdl_launch_dependents();
    pdl_wait();
    q = pdl_acquire(q);
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int groups_per_warp = 32 / seg;
    const int j = lane & (seg - 1);                       // index inside the group
    const int group = warp * groups_per_warp + lane / seg;
    const bool member = (group < P) && (j < G);

    const double qj = member ? (double)q[(int64_t)group * G + j] : 0.0;
    bool alive = member;

    double sigma = 0.0;
    for (int i = 0; i < G; ++i) sigma = __dadd_rn(sigma, shfl_double(qj, i, seg));

    for (int n = G; n > K; --n) {
        const double tau = __dsub_rn(sigma, __dmul_rn(rho, (double)(n - 1)));
        double key = alive ? fabs(__dsub_rn(qj, tau)) : __longlong_as_double(0x7ff0000000000000LL);
        int idx = alive ? j : -1;
        // segmented arg-min; ties -> the higher index
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (o < seg) {
                const double okey = shfl_xor_double(key, o, seg);
                const int oidx = __shfl_xor_sync(0xffffffffu, idx, o, seg);
                if (okey < key || (okey == key && oidx > idx)) { key = okey; idx = oidx; }
            }
        }
        const double q_removed = shfl_double(qj, idx < 0 ? 0 : idx, seg);
        if (idx == j) alive = false;
        sigma = __dsub_rn(sigma, q_removed);
    }
    if (member) keep[(int64_t)group * G + j] = alive ? 1 : 0;
}

}  // namespace

extern "C" int arrol_select(arrol_ctx* ctx, const float* q, int32_t P, int32_t G, int32_t K, double rho,
                            int32_t mode, uint8_t* keep, void* stream) {
    if (!ctx || P < 0 || G < 1 || K < 1 || K > G) return ARROL_ERR_INVALID_ARG;
    if (mode != 0 || G > 32) return ARROL_ERR_UNSUPPORTED;
    if (!(rho >= 0.0 && rho <= 1.0)) return ARROL_ERR_INVALID_ARG;
    if (P == 0) return ARROL_OK;
    if (!q || !keep) return ARROL_ERR_INVALID_ARG;
    int seg = 1;
    while (seg < G) seg <<= 1;
    const int groups_per_warp = 32 / seg;
    const int warps = (P + groups_per_warp - 1) / groups_per_warp;
    const int warps_per_block = 4;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    ARROL_CUDA_OK(arrol_launch_pdl(select_kernel, dim3((warps + warps_per_block - 1) / warps_per_block),
                                   dim3(32 * warps_per_block), 0, (cudaStream_t)stream, q, P, G, K, rho, seg, keep));
    ctx->launches += 1;
    return ARROL_OK;
}
