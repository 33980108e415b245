// arrol_prune_rebatch_host: one whole prune-and-rebatch step for callers whose per-step data is in host memory
// (Algorithm 1, frontend: filter pruned rollouts, re-batch, log-probs on the survivors).
//
// Only what the step needs crosses the bus: the N hidden rows at the detection length (for the head; packed into a
// pinned staging block on the host and sent as one copy), the small per-rollout arrays, and then -- once the keep
// mask is known -- the survivors' hidden rows and token ids, which are copied straight into their packed positions
// (the copy engine does the compaction).  Those uploads run on a
// second stream in token chunks, and the log-prob kernel of chunk c starts as soon as chunk c has landed, so the
// upload of the survivors is hidden behind the tensor-core work.  One host synchronisation in the middle (the mask
// must reach the host to plan the copies) and one at the end.
#include <cstring>
#include <vector>

#include "arrol_internal.h"

namespace {

constexpr int64_t CHUNK_TOKENS = 2 * 74 * 128;   // token tiles per chunk = a multiple of the SM count

// tokens per log-prob launch when T tokens are uploaded: whole multiples of CHUNK_TOKENS, at most one event per chunk
int64_t chunk_for(int64_t T) {
    int64_t chunk = CHUNK_TOKENS;
    while ((T + chunk - 1) / chunk > ARROL_COPY_EVENTS) chunk += CHUNK_TOKENS;
    return chunk < T ? chunk : (T > 0 ? T : 1);
}

}  // namespace

extern "C" int arrol_prune_rebatch_host(arrol_ctx* ctx, const arrol_host_step* st, void* stream) {
    if (!ctx || !st) return ARROL_ERR_INVALID_ARG;
    if (st->P < 0 || st->G < 1 || st->K < 1 || st->K > st->G || st->cutoff < 1 || st->d <= 0 || st->V <= 0 ||
        st->T_src < 0 || st->dst_capacity_tokens < 0)
        return ARROL_ERR_INVALID_ARG;
    if (st->head.dtype != ARROL_BF16 || st->d % 8 != 0) return ARROL_ERR_UNSUPPORTED;
    if (st->head.d != st->d) return ARROL_ERR_INVALID_ARG;      // the head reads whole hidden rows
    const int64_t N64 = (int64_t)st->P * st->G;
    if (N64 > ARROL_MAX_HOST_N) return ARROL_ERR_UNSUPPORTED;
    const int N = (int)N64;
    if (N == 0) {
        if (st->h_num) { st->h_num[0] = 0; st->h_num[1] = 0; }
        return ARROL_OK;
    }
    const void* need[] = {st->h_hidden, st->h_src_tokens, st->h_lengths, st->h_src_tok_off, st->h_rewards,
                          st->W_vocab, st->d_hidden, st->d_lengths, st->d_src_tok_off,
                          st->d_rewards, st->d_score, st->d_prob, st->d_q, st->d_keep,
                          st->d_survivor_idx, st->d_cu_seqlens, st->d_adv, st->d_num, st->d_dst_tokens,
                          st->d_dst_rows, st->d_logp, st->d_workspace, st->h_logp, st->h_adv, st->h_cu_seqlens,
                          st->h_survivor_idx, st->h_num};
    for (const void* p : need)
        if (!p) return ARROL_ERR_INVALID_ARG;
    // the workspace must serve the largest chunk any T <= capacity can lead to (its size is monotone in the tokens)
    if (!arrol_aligned(st->d_workspace, 256) ||
        arrol_token_logprob_workspace(ctx, chunk_for(st->dst_capacity_tokens), st->d, st->V) > st->workspace_bytes)
        return ARROL_ERR_WORKSPACE;
    for (int i = 0; i < N; ++i) {
        const int64_t row = st->h_src_tok_off[i] + st->cutoff - 1;
        if (st->h_src_tok_off[i] < 0 || row >= st->T_src || st->h_lengths[i] < 0 ||
            st->h_src_tok_off[i] + st->h_lengths[i] > st->T_src)
            return ARROL_ERR_INVALID_ARG;
    }

    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    const size_t rb = (size_t)st->d * 2;
    const uint8_t* h_hidden = static_cast<const uint8_t*>(st->h_hidden);
    uint8_t* d_hidden = static_cast<uint8_t*>(st->d_hidden);
    uint8_t* d_dst_rows = static_cast<uint8_t*>(st->d_dst_rows);

    // ---- phase 1: what scoring and selection need ----
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_lengths, st->h_lengths, sizeof(int32_t) * N, cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_src_tok_off, st->h_src_tok_off, sizeof(int64_t) * N, cudaMemcpyHostToDevice, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->d_rewards, st->h_rewards, sizeof(float) * N, cudaMemcpyHostToDevice, s));
    // the hidden row of every rollout at the detection length, packed as [N, d] at the start of d_hidden: through
    // the pinned staging block as one copy when it fits, else row by row
    if ((size_t)N * rb <= ARROL_STAGE_BYTES) {
        for (int i = 0; i < N; ++i)
            std::memcpy(ctx->h_stage + (size_t)i * rb, h_hidden + (size_t)(st->h_src_tok_off[i] + st->cutoff - 1) * rb, rb);
        ARROL_CUDA_OK(cudaMemcpyAsync(d_hidden, ctx->h_stage, (size_t)N * rb, cudaMemcpyHostToDevice, s));
    } else {
        for (int i = 0; i < N; ++i)
            ARROL_CUDA_OK(cudaMemcpyAsync(d_hidden + (size_t)i * rb,
                                          h_hidden + (size_t)(st->h_src_tok_off[i] + st->cutoff - 1) * rb, rb,
                                          cudaMemcpyHostToDevice, s));
    }
    int rc = arrol_score_partial(ctx, st->d_hidden, st->d, nullptr, N, &st->head, &st->calib, st->d_score,
                                 st->d_prob, nullptr, st->d_q, stream);
    if (rc != ARROL_OK) return rc;
    rc = arrol_select(ctx, st->d_q, st->P, st->G, st->K, st->rho, 0, st->d_keep, stream);
    if (rc != ARROL_OK) return rc;
    ARROL_CUDA_OK(cudaMemcpyAsync(ctx->h_keep, st->d_keep, (size_t)N, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaStreamSynchronize(s));

    // ---- phase 2: plan the survivors' uploads on the host (same stable order as the device scan) ----
    std::vector<int32_t> surv;
    std::vector<int64_t> cu(1, 0);
    surv.reserve((size_t)st->P * st->K);
    for (int i = 0; i < N; ++i)
        if (ctx->h_keep[i]) {
            surv.push_back(i);
            cu.push_back(cu.back() + st->h_lengths[i]);
        }
    const int64_t T = cu.back();

    // scan and advantages on the device (no per-token payload: rows and token ids arrive packed)
    rc = arrol_compact(ctx, st->d_keep, st->d_lengths, st->d_src_tok_off, N, st->G, nullptr, nullptr, 0,
                       st->d_rewards, st->eps, st->ddof, st->dst_capacity_tokens, nullptr, nullptr,
                       st->d_cu_seqlens, st->d_survivor_idx, st->d_adv, nullptr, nullptr, st->d_num, stream);
    if (rc != ARROL_OK) return rc;

    if (T > 0 && T <= st->dst_capacity_tokens) {
        const int64_t chunk = chunk_for(T);
        int64_t c = 0;                       // next chunk to launch: tokens [c*chunk, min(T, (c+1)*chunk))
        for (size_t k = 0; k < surv.size(); ++k) {
            const int64_t len = cu[k + 1] - cu[k];
            if (len > 0) {
                ARROL_CUDA_OK(cudaMemcpyAsync(d_dst_rows + (size_t)cu[k] * rb,
                                              h_hidden + (size_t)st->h_src_tok_off[surv[k]] * rb, (size_t)len * rb,
                                              cudaMemcpyHostToDevice, ctx->copy_stream));
                ARROL_CUDA_OK(cudaMemcpyAsync(st->d_dst_tokens + cu[k], st->h_src_tokens + st->h_src_tok_off[surv[k]],
                                              (size_t)len * sizeof(int32_t), cudaMemcpyHostToDevice, ctx->copy_stream));
            }
            const bool last = (k + 1 == surv.size());
            while (c * chunk < T && (cu[k + 1] >= (c + 1) * chunk || last)) {
                const int64_t t0 = c * chunk, t1 = (t0 + chunk < T) ? t0 + chunk : T;
                cudaEvent_t ev = ctx->copy_events[c % ARROL_COPY_EVENTS];
                ARROL_CUDA_OK(cudaEventRecord(ev, ctx->copy_stream));
                ARROL_CUDA_OK(cudaStreamWaitEvent(s, ev, 0));
                rc = arrol_token_logprob(ctx, d_dst_rows + (size_t)t0 * rb, st->W_vocab, st->d_dst_tokens + t0, t1 - t0,
                                         nullptr, st->d, st->V, st->inv_temperature, st->d_logp + t0, nullptr,
                                         st->d_workspace, st->workspace_bytes, stream);
                if (rc != ARROL_OK) {
                    (void)cudaStreamSynchronize(ctx->copy_stream);
                    return rc;
                }
                ++c;
            }
        }
    }

    // ---- results: device -> host ----
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_num, st->d_num, sizeof(int64_t) * 2, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_adv, st->d_adv, sizeof(float) * N, cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_cu_seqlens, st->d_cu_seqlens, sizeof(int64_t) * (N + 1), cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemcpyAsync(st->h_survivor_idx, st->d_survivor_idx, sizeof(int32_t) * N, cudaMemcpyDeviceToHost, s));
    if (T > 0 && T <= st->dst_capacity_tokens)
        ARROL_CUDA_OK(cudaMemcpyAsync(st->h_logp, st->d_logp, sizeof(float) * (size_t)T, cudaMemcpyDeviceToHost, s));
    return arrol_poll_status(ctx, stream, nullptr);   // synchronises the stream (which waited for every upload)
}
