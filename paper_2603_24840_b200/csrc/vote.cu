// arrol_rank_vote: test-time rank-weighted voting with quality-head scores (Section 4.4).
// One warp per group of G <= 32 candidates, one lane per candidate: the rank of a candidate is the number of
// candidates that sort before it (lower score, or equal score and lower index), its weight is rank / (G - 1), and
// every lane sums the ranks of the candidates that share its answer.  The winning answer is the one with the
// largest rank sum; of equal sums the one that appears first.  Rank sums are integers, so the decision is exact.
#include "arrol_internal.h"

namespace {

__global__ void __launch_bounds__(128)
rank_vote_kernel(const float* __restrict__ score, const int32_t* __restrict__ answer, int P, int G,
                 float* __restrict__ weight, int32_t* __restrict__ winner, float* __restrict__ winner_weight) {
    const int lane = threadIdx.x & 31;
    const int group = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (group >= P) return;                       // whole warps leave together
    const bool member = lane < G;
    const float s = member ? score[(int64_t)group * G + lane] : 0.f;
    const int a = member ? answer[(int64_t)group * G + lane] : -1;
    int rank = 0;
    for (int j = 0; j < G; ++j) {
        const float sj = __shfl_sync(0xffffffffu, s, j);
        if (sj < s || (sj == s && j < lane)) rank += 1;
    }
    const int w_int = G > 1 ? rank : 1;           // numerator of the weight
    if (member) weight[(int64_t)group * G + lane] = G > 1 ? (float)rank / (float)(G - 1) : 1.0f;
    int total = 0;
    bool first = true;
    for (int j = 0; j < G; ++j) {
        const int aj = __shfl_sync(0xffffffffu, a, j);
        const int wj = __shfl_sync(0xffffffffu, w_int, j);
        if (aj == a) { total += wj; if (j < lane) first = false; }
    }
    // candidates: first occurrences of valid answers; arg-max of (total, then lowest lane)
    int key = (member && a >= 0 && first) ? total : -1;
    int who = lane;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const int okey = __shfl_xor_sync(0xffffffffu, key, o);
        const int owho = __shfl_xor_sync(0xffffffffu, who, o);
        if (okey > key || (okey == key && owho < who)) { key = okey; who = owho; }
    }
    const int win_answer = __shfl_sync(0xffffffffu, a, who);
    if (lane == 0) {
        winner[group] = key >= 0 ? win_answer : -1;
        winner_weight[group] = key >= 0 ? (G > 1 ? (float)key / (float)(G - 1) : (float)key) : 0.f;
    }
}

}  // namespace

extern "C" int arrol_rank_vote(arrol_ctx* ctx, const float* score, const int32_t* answer, int32_t P, int32_t G,
                               float* weight, int32_t* winner, float* winner_weight, void* stream) {
    if (!ctx || P < 0 || G < 1) return ARROL_ERR_INVALID_ARG;
    if (G > 32) return ARROL_ERR_UNSUPPORTED;
    if (P == 0) return ARROL_OK;
    if (!score || !answer || !weight || !winner || !winner_weight) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    const int warps_per_block = 4;
    rank_vote_kernel<<<(P + warps_per_block - 1) / warps_per_block, 32 * warps_per_block, 0, (cudaStream_t)stream>>>(
        score, answer, P, G, weight, winner, winner_weight);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
