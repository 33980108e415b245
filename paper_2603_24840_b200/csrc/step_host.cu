// arrol_prune_rebatch_host: one whole prune-and-rebatch step for callers whose per-step data is in host memory
// (Algorithm 1, frontend: filter pruned rollouts, re-batch, log-probs on the survivors).  Host -> device copies,
// the four library calls on one stream, device -> host copies of the results, one stream synchronisation.
#include "arrol_internal.h"

namespace {

__global__ void row_index_kernel(const int64_t* __restrict__ src_tok_off, int N, int cutoff,
                                 int64_t* __restrict__ row_index) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) row_index[i] = src_tok_off[i] + (int64_t)(cutoff - 1);
}

}  // namespace

extern "C" int arrol_prune_rebatch_host(arrol_ctx* ctx, const arrol_host_step* st, void* stream) {
    if (!ctx || !st) return ARROL_ERR_INVALID_ARG;
    if (st->P < 0 || st->G < 1 || st->K < 1 || st->K > st->G || st->cutoff < 1 || st->d <= 0 || st->V <= 0 ||
        st->T_src < 0 || st->dst_capacity_tokens < 0)
        return ARROL_ERR_INVALID_ARG;
    if (st->head.dtype != ARROL_BF16) return ARROL_ERR_UNSUPPORTED;
    const int64_t N64 = (int64_t)st->P * st->G;
    if (N64 > INT32_MAX) return ARROL_ERR_UNSUPPORTED;
    const int N = (int)N64;
    if (N == 0) {
        if (st->h_num) { st->h_num[0] = 0; st->h_num[1] = 0; }
        return ARROL_OK;
    }
    const void* need[] = {st->h_hidden, st->h_src_tokens, st->h_lengths, st->h_src_tok_off, st->h_rewards,
                          st->W_vocab, st->d_hidden, st->d_src_tokens, st->d_lengths, st->d_src_tok_off,
                          st->d_row_index, st->d_rewards, st->d_score, st->d_prob, st->d_q, st->d_keep,
                          st->d_survivor_idx, st->d_cu_seqlens, st->d_adv, st->d_num, st->d_dst_tokens,
                          st->d_dst_rows, st->d_logp, st->d_workspace, st->h_logp, st->h_adv, st->h_cu_seqlens,
                          st->h_survivor_idx, st->h_num};
    for (const void* p : need)
        if (!p) return ARROL_ERR_INVALID_ARG;

    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t row_bytes = (size_t)st->d * 2;

    // inputs: host -> device
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_lengths, st->h_lengths, sizeof(int32_t) * N, cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_src_tok_off, st->h_src_tok_off, sizeof(int64_t) * N, cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_rewards, st->h_rewards, sizeof(float) * N, cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_src_tokens, st->h_src_tokens, sizeof(int32_t) * (size_t)st->T_src,
                                  cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_hidden, st->h_hidden, row_bytes * (size_t)st->T_src, cudaMemcpyHostToDevice, s));

    row_index_kernel<<<(N + 255) / 256, 256, 0, s>>>(st->d_src_tok_off, N, st->cutoff, st->d_row_index);
    ARROL_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;

    int rc = arrol_score_partial(ctx, st->d_hidden, st->d, st->d_row_index, N, &st->head, &st->calib, st->d_score,
                                 st->d_prob, nullptr, st->d_q, stream);
    if (rc != ARROL_OK) return rc;
    rc = arrol_select(ctx, st->d_q, st->P, st->G, st->K, st->rho, 0, st->d_keep, stream);
    if (rc != ARROL_OK) return rc;
    rc = arrol_compact(ctx, st->d_keep, st->d_lengths, st->d_src_tok_off, N, st->G, st->d_src_tokens, st->d_hidden,
                       (int32_t)row_bytes, st->d_rewards, st->eps, st->ddof, st->dst_capacity_tokens,
                       st->d_dst_tokens, st->d_dst_rows, st->d_cu_seqlens, st->d_survivor_idx, st->d_adv, nullptr,
                       nullptr, st->d_num, stream);
    if (rc != ARROL_OK) return rc;
    rc = arrol_token_logprob(ctx, st->d_dst_rows, st->W_vocab, st->d_dst_tokens, st->dst_capacity_tokens,
                             st->d_num + 1, st->d, st->V, st->inv_temperature, st->d_logp, nullptr, st->d_workspace,
                             st->workspace_bytes, stream);
    if (rc != ARROL_OK) return rc;

    // results: device -> host
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_num, st->d_num, sizeof(int64_t) * 2, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_adv, st->d_adv, sizeof(float) * N, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_cu_seqlens, st->d_cu_seqlens, sizeof(int64_t) * (N + 1), cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_survivor_idx, st->d_survivor_idx, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_logp, st->d_logp, sizeof(float) * (size_t)st->dst_capacity_tokens,
                                  cudaMemcpyDeviceToHost, s));
    return arrol_poll_status(ctx, stream, nullptr);   // synchronises the stream
}
