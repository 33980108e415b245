// arrol_select: per-group correctness-balancing selection (Section 4.1; Theorem 1's rule
// j^ = argmin_j |mu_{-j} - rho| applied G - K times per group).
//
// One group occupies a segment of `seg` = next power of two >= G lanes; 32 / seg groups share a warp.  Every
// lane holds one rollout's q in double.  Each round: tau = Sigma - rho (n - 1) (one rounding per operation, no
// fused multiply-add), key = |q - tau|, a segmented shuffle arg-min on (key, index) where of equal keys the
// higher index wins, then the winner leaves the group and Sigma -= q_winner.  Sigma starts as the index-order
// sum, built with broadcasts so that every lane of the segment adds the same values in the same order.
#include "arrol_internal.h"
#include "prune_kernels.cuh"

namespace {

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
    const bool alive = select_lanes(qj, member, j, G, K, rho, seg);
    if (member) keep[(int64_t)group * G + j] = alive ? 1 : 0;
}

}  // namespace
// Argument checks of arrol_select, shared with arrol_prune_step's fused path.
int arrol_internal_check_select(const float* q, int32_t P, int32_t G, int32_t K, double rho, int32_t mode,
                                const uint8_t* keep) {
    if (P < 0 || G < 1 || K < 1 || K > G) return ARROL_ERR_INVALID_ARG;
    if (mode != 0 || G > 32) return ARROL_ERR_UNSUPPORTED;
    if (!(rho >= 0.0 && rho <= 1.0)) return ARROL_ERR_INVALID_ARG;
    if (P > 0 && (!q || !keep)) return ARROL_ERR_INVALID_ARG;
    return ARROL_OK;
}

extern "C" int arrol_select(arrol_ctx* ctx, const float* q, int32_t P, int32_t G, int32_t K, double rho,
                            int32_t mode, uint8_t* keep, void* stream) {
    if (!ctx) return ARROL_ERR_INVALID_ARG;
    {
        const int rc = arrol_internal_check_select(q, P, G, K, rho, mode, keep);
        if (rc != ARROL_OK) return rc;
    }
    if (P == 0) return ARROL_OK;
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
