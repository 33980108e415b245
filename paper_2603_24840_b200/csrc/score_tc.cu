// MLP quality head (Section 4.2) on the tensor cores, for bf16 heads: the first layer U[N,h] = X[N,d] x W1[h,d]^T is
// a dense contraction, so it runs as tcgen05 MMAs fed by TMA, and the rest of the head (bias, exact GELU, w2 dot
// product, sigmoid, bin, posterior look-up: Appendix A.4) is finished in the same kernel.
//
//   pack_rows_kernel      copies the N scored rows (one per rollout, anywhere in the hidden buffer) into a packed
//                         [N,d] block so that TMA can tile them; skipped when the rows are already evenly strided.
//                         (Fetching the rows in place from inside the contraction, four warps of 16-byte cp.async
//                         copies into the swizzled stage layout, was built and measured: correct, but the
//                         load/store path holds about 20 KB in flight per SM against the ring's 192 KB by TMA, and
//                         every block of a row tile fetches the same rows: 18.5 us per call against 14.6 us.)
//   score_mlp_tc_kernel   one block per (128 rollouts x 64 hidden units); shared memory is one ring of eight stages
//                         (128 x 64 of X, 64 x 64 of W1 per K step of 64), filled by two TMA producer threads on
//                         alternate K steps.  Four MMA issuer threads take the K steps round robin (ks mod 4), each
//                         into its own 64-column tensor-memory accumulator: one thread's wait -> four MMAs -> commit
//                         round costs several hundred cycles per K step against the 32 cycles a 128 x 64 x 16 MMA
//                         keeps the tensor pipe busy, so the loop's length is rounds / issuers.
//                         Eight epilogue warps: thread = rollout x half of the tile's 64 hidden units; accumulators
//                         added in index order, then sum_j w2_j gelu(u_j + b1_j) over the 32 units in index order,
//                         the two halves added low + high -> partial[h_tile][N].  The last block of a row tile to
//                         finish (a counter per row tile) adds the h tiles in index order, adds b2 and applies the
//                         probability map, so the result does not depend on block order.
// Every wait is bounded; on expiry the block records ARROL_DEV_WAIT_EXPIRED, drains and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "score_common.cuh"
#include "tc_common.cuh"

namespace {

constexpr int SBN = 64;                      // hidden units per tile (MMA N)
constexpr int S_ISSUERS = 4;                 // MMA issuer threads, each with its own accumulator
constexpr int S_PRODUCERS = 2;               // TMA producer threads (lane 0 of the first warps)
constexpr int S_PRODUCER_WARPS = 4;          // warps before the issuers (two of them idle: the epilogue warps start at a multiple of 4)
constexpr int S_EPI_WARP0 = S_PRODUCER_WARPS + S_ISSUERS;      // a multiple of 4: epilogue warp w reads lane quarter w % 4
constexpr int S_EPI_WARPS = 8;
constexpr int SB_BYTES = SBN * BK * 2;       //  8 KB
constexpr int S_TMEM_COLS = S_ISSUERS * SBN; // a power of two >= 32
constexpr int S_THREADS = (S_EPI_WARP0 + S_EPI_WARPS) * 32;
constexpr int S_TAIL_BYTES = 2048;           // barriers, tensor-memory slot, flags | b1, w2 of the tile | half sums
constexpr int TM = 128;                      // rollouts per tile (MMA M)
constexpr int STAGES = 8;
constexpr int A_BYTES = TM * BK * 2;         // 16 KB
constexpr int STAGE_BYTES = A_BYTES + SB_BYTES;
constexpr size_t S_SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 + S_TAIL_BYTES;

// one warp per rollout: 16-byte copies, all of a row's loads in flight before the first store
__global__ void __launch_bounds__(128)
pack_rows_kernel(const __nv_bfloat16* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index,
                 int N, int d, __nv_bfloat16* __restrict__ out, int64_t source_rows, uint32_t* d_status) {
    pdl_launch_dependents();
    pdl_wait();
    hidden = pdl_acquire(hidden); row_index = pdl_acquire(row_index);
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (i >= N) return;
    const int64_t row = row_index[i];
    const uint4* src = reinterpret_cast<const uint4*>(hidden + row * row_stride);
    uint4* dst = reinterpret_cast<uint4*>(out + (int64_t)i * d);
    const int nvec = d / 8;
    if (source_rows > 0 && (row < 0 || row >= source_rows)) {   // outside the caller's buffer: never read, packed as zeros
        if (lane == 0) atomicOr(d_status, ARROL_DEV_BAD_INDEX);
        for (int c = lane; c < nvec; c += 32) dst[c] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    for (int c0 = lane; c0 < nvec; c0 += 256) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (c0 + 32 * u < nvec) v[u] = __ldg(src + c0 + 32 * u);
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (c0 + 32 * u < nvec) dst[c0 + 32 * u] = v[u];
    }
}

struct ScoreTcParams {
    int N, h;
    int k_steps;                       // ceil(d / 64)
    const __nv_bfloat16* b1;           // [h] or NULL
    const __nv_bfloat16* w2;           // [h]
    const __nv_bfloat16* b2;           // [1] or NULL
    float* partial;                    // [h_tiles][N]
    float* u_out;                      // [N][h] pre-activations (bias included) for the head training step, or NULL
    uint32_t* counters;                // [row tiles], zero between calls
    int B;
    const float* q_lut;
    float* score;
    float* prob;
    int32_t* bin;
    float* q;
    uint32_t* d_status;
};

__global__ void __launch_bounds__(S_THREADS, 1)
score_mlp_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                    const ScoreTcParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_a = smem;
    uint8_t* stage_b = smem + (size_t)STAGES * A_BYTES;
    uint8_t* tail = smem + (size_t)STAGES * STAGE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(tail);          // [STAGES] producers -> MMA
    uint64_t* empty = full + STAGES;                             // [STAGES] MMA -> producers
    uint64_t* acc_full = empty + STAGES;                         // [1] every MMA of the block has finished
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* is_last = tmem_slot + 2;
    float* b1_s = reinterpret_cast<float*>(tail + 256);          // [SBN]
    float* w2_s = b1_s + SBN;                                    // [SBN]
    float* half_s = reinterpret_cast<float*>(tail + 1024);       // [TM] sums over the tile's upper 32 hidden units

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * TM, j0 = blockIdx.y * SBN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, S_ISSUERS);
        *abort_flag = 0u;
        *is_last = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    }
    if (warp == S_PRODUCER_WARPS) {         // first MMA warp owns the tensor-memory allocation
        tcgen05_alloc(tmem_slot, S_TMEM_COLS);
        tcgen05_relinquish();
    }
    pdl_launch_dependents();
    pdl_wait();                  // set-up above overlaps the previous kernel; global memory is read from here on
    if (warp >= S_EPI_WARP0) {   // the tile's slice of b1 and w2, zero past h so that padded columns add nothing
        const int e = threadIdx.x - S_EPI_WARP0 * 32;
        if (e < SBN) {
            const int j = j0 + e;
            b1_s[e] = (j < p.h && p.b1) ? __bfloat162float(p.b1[j]) : 0.f;
            w2_s[e] = (j < p.h) ? __bfloat162float(p.w2[j]) : 0.f;
        }
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // K step ks uses stage ks % STAGES in round ks / STAGES of the ring and issuer / accumulator ks % S_ISSUERS.
    if (warp < S_PRODUCER_WARPS) {
        if (lane == 0 && warp < S_PRODUCERS) {
            int last = -1;
            bool ok = true;
            for (int ks = warp; ks < p.k_steps; ks += S_PRODUCERS) {
                const int st = ks % STAGES;
                const uint32_t round = (uint32_t)(ks / STAGES);
                if (!mbar_wait(&empty[st], (round & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&full[st], STAGE_BYTES);
                tma_load_2d(stage_a + (size_t)st * A_BYTES, &map_x, ks * BK, m0, &full[st]);
                tma_load_2d(stage_b + (size_t)st * SB_BYTES, &map_w, ks * BK, j0, &full[st]);
                last = ks;
            }
            if (!ok || *abort_flag) {   // let this thread's copies in flight land before the block's shared memory goes away
                for (int ks = last; ks >= 0 && ks > last - STAGES; ks -= S_PRODUCERS)
                    for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
                        if (mbar_try_wait(&full[ks % STAGES], (uint32_t)(ks / STAGES) & 1u)) break;
            }
        }
    } else if (warp < S_EPI_WARP0) {
        if (lane == 0) {
            const int r = warp - S_PRODUCER_WARPS;
            const uint32_t d_tmem = tmem_base + (uint32_t)(r * SBN);
            constexpr uint32_t idesc = make_idesc(TM, SBN);
            for (int ks = r; ks < p.k_steps; ks += S_ISSUERS) {
                const int st = ks % STAGES;
                if (!mbar_wait(&full[st], (uint32_t)(ks / STAGES) & 1u, abort_flag)) break;
                tcgen05_fence_after();
                const uint64_t a_desc = make_smem_desc(smem_u32(stage_a + (size_t)st * A_BYTES));
                const uint64_t b_desc = make_smem_desc(smem_u32(stage_b + (size_t)st * SB_BYTES));
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k)
                    tcgen05_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                     (ks >= S_ISSUERS || k > 0) ? 1u : 0u);
                tcgen05_commit(&empty[st]);
            }
            // Arrives once every MMA issued by this thread has finished: publishes the accumulator on the normal
            // path, and on the give-up path it is what this thread waits for before shared and tensor memory go away.
            tcgen05_commit(acc_full);
            if (*abort_flag)
                for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
                    if (mbar_try_wait(acc_full, 0u)) break;
        }
    } else {
        const int quarter = warp & 3;                           // accumulator row r is tensor-memory lane r
        const int half = (warp - S_EPI_WARP0) >> 2;             // which 32 of the tile's 64 hidden units
        const int r_tile = quarter * 32 + lane;
        const int m = m0 + r_tile;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int used_accs = p.k_steps < S_ISSUERS ? p.k_steps : S_ISSUERS;   // an issuer without K steps wrote nothing
        bool ok = mbar_wait(acc_full, 0u, abort_flag);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag) != 0;
        float part = 0.f;
        if (ok) {
            tcgen05_fence_after();
            float v[32];
            tcgen05_ld_32x32(tmem_base + lane_addr + half * 32, v);
            for (int a = 1; a < used_accs; ++a) {      // fixed order: ((acc0 + acc1) + acc2) + acc3
                float w[32];
                tcgen05_ld_32x32(tmem_base + lane_addr + a * SBN + half * 32, w);
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) v[jj] += w[jj];
            }
#pragma unroll
            for (int jj = 0; jj < 32; ++jj) {
                const float u = v[jj] + b1_s[half * 32 + jj];
                v[jj] = u;
                const float g = 0.5f * u * (1.0f + erff(u * 0.70710678118654752440f));
                part = fmaf(w2_s[half * 32 + jj], g, part);
            }
            if (p.u_out && m < p.N) {
                float* urow = p.u_out + (int64_t)m * p.h + j0 + half * 32;
#pragma unroll
                for (int jj = 0; jj < 32; jj += 4)      // h % 4 == 0: a float4 never straddles the edge
                    if (j0 + half * 32 + jj < p.h)
                        *reinterpret_cast<float4*>(urow + jj) = make_float4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]);
            }
        }
        if (half == 1) half_s[r_tile] = part;
        asm volatile("bar.sync 2, 256;" ::: "memory");
        if (half == 0) {
            part += half_s[r_tile];                             // low half + high half
            // The counter protocol runs whatever happened above, so the counters are back at zero after every launch
            // (after an expired wait the scores of the call are not meaningful and the status word says so).
            if (m < p.N) p.partial[(int64_t)blockIdx.y * p.N + m] = part;
            __threadfence();
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (threadIdx.x == S_EPI_WARP0 * 32) {
                const uint32_t done = atomicAdd(&p.counters[blockIdx.x], 1u);
                if (done == gridDim.y - 1) {
                    *is_last = 1u;
                    p.counters[blockIdx.x] = 0u;    // every block of this row tile has arrived: ready for the next call
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (*is_last && m < p.N) {
                __threadfence();
                float s = 0.f;
                for (int t = 0; t < (int)gridDim.y; ++t) s += __ldcg(&p.partial[(int64_t)t * p.N + m]);
                if (p.b2) s += __bfloat162float(p.b2[0]);
                probability_map(s, m, p.B, p.q_lut, p.score, p.prob, p.bin, p.q);
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.d_status, ARROL_DEV_WAIT_EXPIRED);
    if (warp == S_PRODUCER_WARPS) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, S_TMEM_COLS);
    }
}

}  // namespace

// Scores of a bf16 MLP head on the tensor cores.  Returns ARROL_ERR_UNSUPPORTED (nothing launched) when the sizes
// do not fit the context's buffers; the caller then takes the SIMT path.  Indexed rows are left packed as bf16
// [N][d] in the context's packing buffer (the head training step's second contraction reads them there).
int arrol_internal_score_mlp_tc(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index,
                                int N, const arrol_head* head, int B, const float* q_lut, float* score, float* prob,
                                int32_t* bin, float* q, float* u_out, cudaStream_t s) {
    const int d = head->d, h = head->h;
    const int h_tiles = (h + SBN - 1) / SBN;
    const int m_tiles = (N + TM - 1) / TM;
    if ((size_t)N * (size_t)h_tiles > ARROL_SCRATCH_FLOATS || m_tiles > ARROL_SCORE_ROW_TILES)
        return ARROL_ERR_UNSUPPORTED;
    const bool pack = row_index != nullptr;
    if (pack && (size_t)N * (size_t)d * 2 > ARROL_PACK_BYTES) return ARROL_ERR_UNSUPPORTED;
    if (!row_index && ((uint64_t)row_stride * 2) >= (1ull << 40)) return ARROL_ERR_UNSUPPORTED;

    const void* x = hidden;
    int64_t ld = row_stride;
    if (pack) {
        ARROL_CUDA_OK(arrol_launch_pdl(pack_rows_kernel, dim3((N + 3) / 4), dim3(128), 0, s,
                                       static_cast<const __nv_bfloat16*>(hidden), row_stride, row_index, N, d,
                                       static_cast<__nv_bfloat16*>(ctx->d_pack), ctx->source_rows, ctx->d_status));
        ctx->launches += 1;
        x = ctx->d_pack;
        ld = d;
    }
    CUtensorMap map_x, map_w;
    if (make_map(ctx, &map_w, head->W1, (uint64_t)h, (uint64_t)d, SBN) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map_ld(ctx, &map_x, x, (uint64_t)N, (uint64_t)d, (uint64_t)ld, TM) != ARROL_OK) return ARROL_ERR_CUDA;

    ScoreTcParams p;
    p.N = N;
    p.h = h;
    p.k_steps = (d + BK - 1) / BK;
    p.b1 = static_cast<const __nv_bfloat16*>(head->b1);
    p.w2 = static_cast<const __nv_bfloat16*>(head->w2);
    p.b2 = static_cast<const __nv_bfloat16*>(head->b2);
    p.partial = ctx->d_scratch;
    p.u_out = u_out;
    p.counters = ctx->d_tile_counters;
    p.B = B;
    p.q_lut = q_lut;
    p.score = score;
    p.prob = prob;
    p.bin = bin;
    p.q = q;
    p.d_status = ctx->d_status;
    dim3 grid(m_tiles, h_tiles);
    if (!ctx->score_tc_smem_set) {      // once per context: this call is on the prune step's microsecond path
        ARROL_CUDA_OK(cudaFuncSetAttribute(score_mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)S_SMEM_BYTES));
        ctx->score_tc_smem_set = true;
    }
    ARROL_CUDA_OK(arrol_launch_pdl(score_mlp_tc_kernel, grid, dim3(S_THREADS), S_SMEM_BYTES, s, map_x, map_w, p));
    ctx->launches += 1;
    return ARROL_OK;
}
