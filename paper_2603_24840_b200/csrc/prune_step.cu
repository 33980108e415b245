// arrol_prune_step: score -> select -> compact from one call, for callers that want the prune-and-rebatch part of the
// step (Algorithm 1: quality check at the detection length, filter, re-batch) without host work between the launches.
//
// The chain is a handful of microsecond kernels, each a few dependent round trips to memory, so what it costs is
// launches and latency, not work.  Fast path: ONE grid runs scoring, selection, the survivor scan and the advantages,
// and a second launch writes the per-token outputs.
//   prune_fused_kernel   a block owns 32 / G whole groups (at most 32 rollouts, one warp each).  Linear head: every
//                        warp scores its rollout (the row reduction and probability map of score_linear_kernel) and
//                        leaves q in shared memory; MLP head: q comes from the scoring kernel that ran before (blocks
//                        of two warps then, always 32 / G groups each).  One or
//                        two warps run the per-group selection (select_lanes, as select_kernel) and write the keep
//                        flags.  The first warp then scans the block's rollouts (kept, kept length), publishes the
//                        block's totals, adds up the totals of the blocks before it as they appear (a chained scan:
//                        every block only waits for lower-numbered blocks, and the grid never exceeds the SM count, so
//                        all blocks are resident), and writes survivor_idx, cu_seqlens and the advantages of its own
//                        groups (group_statistics, as scan_adv_kernel); the last block writes {S, T}.  Nothing is
//                        re-read from global memory and no block waits for the whole grid.  The block that finishes
//                        last clears the published totals for the next call.
// The device functions are the ones the three separate kernels use, so the results are bit-identical to the three
// public calls, which remain the general path (more than SM-count blocks of 32 / G groups; group sizes above 32 are
// rejected by arrol_select either way).
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "prune_kernels.cuh"

namespace {

struct FusedParams {
    // scoring (linear head) / its outputs
    const void* hidden;
    int64_t row_stride;
    const int64_t* row_index;
    const void* w;
    const void* bias;
    const float* q_lut;
    float *score, *prob, *q;
    int32_t* bin;
    int N, d, B;
    // selection
    int P, G, K, seg, gpb;     // gpb: groups per block
    double rho;
    uint8_t* keep;
    // scan + advantages
    const int32_t* lengths;
    const float* rewards;
    const int64_t* src_tok_off;
    double eps;
    int ddof;
    int64_t capacity, source_rows;
    int32_t* survivor_idx;
    int64_t* cu_seqlens;
    float* adv;
    int64_t* d_num;
    uint32_t* d_status;
    // chained scan: words [0] finished blocks, [1] a kept rollout left the source (index check), then per block
    // {kept tokens, kept rollouts}, each with bit 63 set once published; all zero between calls
    unsigned long long* chain;
    uint32_t spin_limit;
};

constexpr unsigned long long PUBLISHED = 1ull << 63;

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// SCORE: the block scores its rollouts itself (linear head, element type T); otherwise q was written by an earlier
// kernel on the stream.
template <typename T, bool SCORE>
__global__ void __launch_bounds__(SCAN_THREADS)
prune_fused_kernel(const FusedParams p) {
    __shared__ float q_s[32], rew_s[32];
    __shared__ uint8_t keep_s[32];
    __shared__ int32_t len_s[32];
    __shared__ double inv_count[SCAN_INV], g_mean[32], g_den[32];
    extern __shared__ uint4 w_stage[];                       // linear head: the weights, d * sizeof(T) bytes
    pdl_launch_dependents();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int group0 = blockIdx.x * p.gpb;
    const int groups_here = min(p.gpb, p.P - group0);
    const int first = group0 * p.G;
    const int n_here = groups_here * p.G;                   // rollouts of this block, one warp each
    if (threadIdx.x >= 1 && threadIdx.x < SCAN_INV) inv_count[threadIdx.x] = 1.0 / (double)threadIdx.x;
    pdl_wait();
    bool bad_index = false;
    if (warp == 1 && lane < n_here) {                        // the block's lengths and rewards, while the others score
        const int i = first + lane;
        len_s[lane] = max(pdl_acquire(p.lengths)[i], 0);
        rew_s[lane] = pdl_acquire(p.rewards)[i];
    }
    if constexpr (SCORE) {
        // every warp fetches its row number while the block stages the head's weights
        constexpr int VN = Vec16<T>::N;
        typedef typename Vec16<T>::Raw Raw;
        Raw* w_s = reinterpret_cast<Raw*>(w_stage);
        const int i = first + warp;
        int64_t row = 0;
        if (warp < n_here) {
            const int64_t* row_index = pdl_acquire(p.row_index);
            row = row_index ? row_index[i] : (int64_t)i;
        }
        const T* w = pdl_acquire(static_cast<const T*>(p.w));
        for (int c = threadIdx.x; c < p.d / VN; c += blockDim.x) w_s[c] = Vec16<T>::load_raw(w + (int64_t)c * VN);
        __syncthreads();
        if (warp < n_here) {
            const T* hidden = pdl_acquire(static_cast<const T*>(p.hidden));
            const T* bias = pdl_acquire(static_cast<const T*>(p.bias));
            const float* q_lut = pdl_acquire(p.q_lut);
            int nvec = p.d / VN;
            if (p.source_rows > 0 && (row < 0 || row >= p.source_rows)) {   // never read, scored as zeros
                if (lane == 0) atomicOr(p.d_status, ARROL_DEV_BAD_INDEX);
                nvec = 0;
            }
            float s = linear_row_dot_ws<T>(hidden + row * p.row_stride, w_s, nvec, lane);
            if (lane == 0) {
                if (bias) s += to_f32(bias[0]);
                q_s[warp] = probability_map(s, i, p.B, q_lut, p.score, p.prob, p.bin, p.q);
            }
        }
    } else {
        if (threadIdx.x < n_here) q_s[threadIdx.x] = pdl_acquire(p.q)[first + threadIdx.x];
    }
    __syncthreads();
    // selection on the block's groups: a group per segment of `seg` lanes
    const int groups_per_warp = 32 / p.seg;
    if (warp * groups_per_warp < groups_here) {
        const int gl = warp * groups_per_warp + lane / p.seg;
        const int j = lane & (p.seg - 1);
        const bool member = gl < groups_here && j < p.G;
        const double qj = member ? (double)q_s[gl * p.G + j] : 0.0;
        const bool alive = select_lanes(qj, member, j, p.G, p.K, p.rho, p.seg);
        if (member) {
            keep_s[gl * p.G + j] = alive ? 1 : 0;
            p.keep[first + gl * p.G + j] = alive ? 1 : 0;
        }
    }
    __syncthreads();
    if (warp != 0) return;

    // ---- first warp: scan of the block's rollouts, chained over the blocks, outputs of the block's groups ----
    const bool kept = lane < n_here && keep_s[lane] != 0;
    const int32_t own_c = kept ? 1 : 0;
    const int64_t own_t = kept ? (int64_t)len_s[lane] : 0;
    if (kept && p.source_rows > 0) {
        const int64_t o = pdl_acquire(p.src_tok_off)[first + lane];
        bad_index = o < 0 || o + own_t > p.source_rows;
    }
    int32_t c = own_c;
    int64_t t = own_t;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t oc = __shfl_up_sync(0xffffffffu, c, o);
        const int64_t ot = __shfl_up_sync(0xffffffffu, t, o);
        if (lane >= o) { c += oc; t += ot; }
    }
    const int32_t block_c = __shfl_sync(0xffffffffu, c, 31);
    const int64_t block_t = __shfl_sync(0xffffffffu, t, 31);
    unsigned long long* totals = p.chain + 2;
    if (lane == 0) {
        totals[2 * blockIdx.x] = PUBLISHED | (unsigned long long)block_t;
        totals[2 * blockIdx.x + 1] = PUBLISHED | (unsigned long long)block_c;
    }
    // statistics of the block's groups, one lane per group, while the other blocks publish
    if (lane < groups_here) {
        auto flag = [&](int r) { return keep_s[r] != 0; };
        auto rew = [&](int r) { return rew_s[r]; };
        double mean, den;
        group_statistics(lane * p.G, lane * p.G + p.G, p.ddof, p.eps, inv_count, flag, rew, mean, den);
        g_mean[lane] = mean;
        g_den[lane] = den;
    }
    // totals of the blocks before this one (each lane takes every 32nd of them)
    int64_t base_t = 0;
    int32_t base_c = 0;
    bool expired = false;
    for (int b = lane; b < (int)blockIdx.x; b += 32) {
        unsigned long long wt = 0, wc = 0;
        uint32_t it = 0;
        for (;;) {
            wt = ld_acquire_u64(totals + 2 * b);
            wc = ld_acquire_u64(totals + 2 * b + 1);
            if ((wt & wc & PUBLISHED) != 0) break;
            if (++it >= p.spin_limit) { expired = true; break; }
        }
        base_t += (int64_t)(wt & ~PUBLISHED);
        base_c += (int32_t)(wc & ~PUBLISHED);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        base_t += __shfl_xor_sync(0xffffffffu, base_t, o);
        base_c += __shfl_xor_sync(0xffffffffu, base_c, o);
    }
    __syncwarp();
    if (kept) {
        const int32_t pos = base_c + (c - own_c);
        p.survivor_idx[pos] = first + lane;
        p.cu_seqlens[pos + 1] = base_t + t;
        const int g = lane / p.G;
        p.adv[pos] = (float)(((double)rew_s[lane] - g_mean[g]) * g_den[g]);      // den holds 1 / (std + eps), or 0
    }
    if (blockIdx.x == 0 && lane == 0) p.cu_seqlens[0] = 0;
    if (blockIdx.x == gridDim.x - 1 && lane == 0) {
        p.d_num[0] = base_c + block_c;
        p.d_num[1] = base_t + block_t;
        if (base_t + block_t > p.capacity) atomicOr(p.d_status, ARROL_DEV_CAPACITY);
    }
    const bool any_bad = __any_sync(0xffffffffu, bad_index);
    const bool any_expired = __any_sync(0xffffffffu, expired);
    if (lane == 0) {
        if (any_expired) atomicOr(p.d_status, ARROL_DEV_WAIT_EXPIRED);
        if (any_bad) atomicOr(reinterpret_cast<unsigned int*>(p.chain + 1), 1u);
        __threadfence();
        // the block that finishes last has seen every block read what it needed: clear the chain for the next call
        const unsigned long long done = atomicAdd(p.chain, 1ull);
        if (done == gridDim.x - 1) {
            __threadfence();
            const unsigned int bad = *reinterpret_cast<volatile unsigned int*>(p.chain + 1);
            if (bad) atomicOr(p.d_status, ARROL_DEV_BAD_INDEX);
            p.d_status[1] = bad ? 1u : 0u;       // gate word: the gather kernels of this call copy nothing when set
            for (unsigned int b = 0; b < 2 * gridDim.x; ++b) totals[b] = 0ull;
            p.chain[1] = 0ull;
            p.chain[0] = 0ull;
        }
    }
}

}  // namespace

extern "C" int arrol_prune_step(arrol_ctx* ctx, const arrol_prune_step_args* a, void* stream) {
    if (!ctx || !a) return ARROL_ERR_INVALID_ARG;
    if (a->P < 0 || a->G < 1) return ARROL_ERR_INVALID_ARG;
    const int64_t N64 = (int64_t)a->P * a->G;
    if (N64 > INT32_MAX) return ARROL_ERR_UNSUPPORTED;
    const int32_t N = (int32_t)N64;

    // Everything is validated before the first launch, so that a bad argument of a later stage leaves nothing half done.
    if (N > 0) {
        int rc = arrol_internal_check_score(a->hidden, a->row_stride_elems, N, &a->head, &a->calib, a->score, a->prob, a->q);
        if (rc != ARROL_OK) return rc;
    }
    int rc = arrol_internal_check_select(a->q, a->P, a->G, a->K, a->rho, 0, a->keep);
    if (rc != ARROL_OK) return rc;
    rc = arrol_internal_check_compact(a->keep, a->lengths, a->src_tok_off, N, a->G, a->src_tokens, a->src_rows,
                                      a->row_bytes, a->rewards, a->eps, a->ddof, a->dst_capacity_tokens, a->dst_tokens,
                                      a->dst_rows, a->cu_seqlens, a->survivor_idx, a->adv, a->d_num);
    if (rc != ARROL_OK) return rc;
    if (N == 0)       // nothing to score or select; the scan still writes {0, 0}
        return arrol_compact(ctx, a->keep, a->lengths, a->src_tok_off, N, a->G, a->src_tokens, a->src_rows, a->row_bytes,
                             a->rewards, a->eps, a->ddof, a->dst_capacity_tokens, a->dst_tokens, a->dst_rows, a->cu_seqlens,
                             a->survivor_idx, a->adv, a->tok_adv, a->tok_seq, a->d_num, stream);

    const bool linear = a->head.h == 0;
    // groups per block: as many as 32 warps hold, fewer while that leaves most SMs without a block
    int gpb = 32 / a->G;
    while (gpb > 1 && (a->P + gpb - 1) / gpb < ctx->sm_count / 2) gpb = (gpb + 1) / 2;
    int threads = 32 * gpb * a->G;
    if (threads < 64) threads = 64;                          // warp 1 fetches the lengths and rewards
    if (!linear) {                                           // nothing to score: two warps per block, full blocks
        gpb = 32 / a->G;
        threads = 64;
    }
    const int64_t fused_blocks = ((int64_t)a->P + gpb - 1) / gpb;
    const size_t w_bytes = linear ? (size_t)a->head.d * (a->head.dtype == ARROL_F32 ? 4 : 2) : 0;
    // the chained scan needs every block resident: at most (SMs x blocks that fit an SM) blocks
    const int per_sm = 2048 / threads < 1 ? 1 : 2048 / threads;
    if (fused_blocks > (int64_t)ctx->sm_count * (per_sm > 2 ? 2 : per_sm) || fused_blocks > ARROL_CHAIN_BLOCKS ||
        w_bytes > 40 * 1024) {
        // too many blocks for the chained scan to be resident at once (or a head too wide to stage): the three calls,
        // back to back
        rc = arrol_score_partial(ctx, a->hidden, a->row_stride_elems, a->row_index, N, &a->head, &a->calib, a->score,
                                 a->prob, a->bin, a->q, stream);
        if (rc != ARROL_OK) return rc;
        rc = arrol_select(ctx, a->q, a->P, a->G, a->K, a->rho, 0, a->keep, stream);
        if (rc != ARROL_OK) return rc;
        return arrol_compact(ctx, a->keep, a->lengths, a->src_tok_off, N, a->G, a->src_tokens, a->src_rows, a->row_bytes,
                             a->rewards, a->eps, a->ddof, a->dst_capacity_tokens, a->dst_tokens, a->dst_rows, a->cu_seqlens,
                             a->survivor_idx, a->adv, a->tok_adv, a->tok_seq, a->d_num, stream);
    }
    if (!linear) {    // MLP head: its own kernels score; the fused kernel starts at the selection
        rc = arrol_score_partial(ctx, a->hidden, a->row_stride_elems, a->row_index, N, &a->head, &a->calib, a->score,
                                 a->prob, a->bin, a->q, stream);
        if (rc != ARROL_OK) return rc;
    }
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    FusedParams p;
    p.hidden = a->hidden;
    p.row_stride = a->row_stride_elems;
    p.row_index = a->row_index;
    p.w = a->head.W1;
    p.bias = a->head.b1;
    p.q_lut = a->calib.q_lut;
    p.B = a->calib.B > 0 ? a->calib.B : 0;
    p.score = a->score; p.prob = a->prob; p.q = a->q; p.bin = a->bin;
    p.N = N; p.d = a->head.d;
    p.P = a->P; p.G = a->G; p.K = a->K; p.rho = a->rho;
    p.seg = 1;
    while (p.seg < a->G) p.seg <<= 1;
    p.gpb = gpb;
    p.keep = a->keep;
    p.lengths = a->lengths; p.rewards = a->rewards; p.src_tok_off = a->src_tok_off;
    p.eps = (double)a->eps; p.ddof = a->ddof;
    p.capacity = a->dst_capacity_tokens; p.source_rows = ctx->source_rows;
    p.survivor_idx = a->survivor_idx; p.cu_seqlens = a->cu_seqlens; p.adv = a->adv; p.d_num = a->d_num;
    p.d_status = ctx->d_status;
    p.chain = ctx->d_chain;
    p.spin_limit = ctx->test_spin_limit ? ctx->test_spin_limit : (1u << 22);
    const dim3 grid((unsigned)fused_blocks), block((unsigned)threads);
    cudaStream_t s = (cudaStream_t)stream;
    if (!linear)
        ARROL_CUDA_OK(arrol_launch_pdl(prune_fused_kernel<float, false>, grid, block, 0, s, p));
    else if (a->head.dtype == ARROL_F32)
        ARROL_CUDA_OK(arrol_launch_pdl(prune_fused_kernel<float, true>, grid, block, w_bytes, s, p));
    else
        ARROL_CUDA_OK(arrol_launch_pdl(prune_fused_kernel<__nv_bfloat16, true>, grid, block, w_bytes, s, p));
    ctx->launches += 1;
    return arrol_internal_compact(ctx, a->keep, a->lengths, a->src_tok_off, N, a->G, a->src_tokens, a->src_rows,
                                  a->row_bytes, a->rewards, a->eps, a->ddof, a->dst_capacity_tokens, a->dst_tokens,
                                  a->dst_rows, a->cu_seqlens, a->survivor_idx, a->adv, a->tok_adv, a->tok_seq, a->d_num,
                                  stream, true);
}
