// arrol_prune_step: score -> select -> compact issued back to back from one call, for callers that want the
// prune-and-rebatch part of the step (Algorithm 1: quality check at the detection length, filter, re-batch) without
// host work between the launches.  Pure sequencing: each stage is the public call of the same name.
#include "arrol_internal.h"

extern "C" int arrol_prune_step(arrol_ctx* ctx, const arrol_prune_step_args* a, void* stream) {
    if (!ctx || !a) return ARROL_ERR_INVALID_ARG;
    if (a->P < 0 || a->G < 1) return ARROL_ERR_INVALID_ARG;
    const int64_t N64 = (int64_t)a->P * a->G;
    if (N64 > INT32_MAX) return ARROL_ERR_UNSUPPORTED;
    const int32_t N = (int32_t)N64;
    int rc = arrol_score_partial(ctx, a->hidden, a->row_stride_elems, a->row_index, N, &a->head, &a->calib, a->score,
                                 a->prob, a->bin, a->q, stream);
    if (rc != ARROL_OK) return rc;
    rc = arrol_select(ctx, a->q, a->P, a->G, a->K, a->rho, 0, a->keep, stream);
    if (rc != ARROL_OK) return rc;
    return arrol_compact(ctx, a->keep, a->lengths, a->src_tok_off, N, a->G, a->src_tokens, a->src_rows, a->row_bytes,
                         a->rewards, a->eps, a->ddof, a->dst_capacity_tokens, a->dst_tokens, a->dst_rows, a->cu_seqlens,
                         a->survivor_idx, a->adv, a->tok_adv, a->tok_seq, a->d_num, stream);
}
