// MLP quality head (Section 4.2) on the tensor cores, for bf16 heads: the first layer U[N,h] = X[N,d] x W1[h,d]^T is
// a dense contraction, so it runs as tcgen05 MMAs fed by TMA, and the rest of the head (bias, exact GELU, w2 dot
// product, sigmoid, bin, posterior look-up: Appendix A.4) is finished in the same kernel.
//
//   pack_rows_kernel      copies the N scored rows (one per rollout, anywhere in the hidden buffer) into a packed
//                         [N,d] block so that TMA can tile them; skipped when the rows are already evenly strided
//   score_mlp_tc_kernel   one block per (128 rollouts x 64 hidden units): two TMA producer / MMA issuer thread pairs
//                         (128 x 64 x 16 MMAs, alternate K steps, one 64-column tensor-memory accumulator per
//                         pair), four epilogue warps: thread = rollout, accumulators added in index order, then
//                         sum_j w2_j gelu(u_j + b1_j) over the tile's hidden units -> partial[h_tile][N].  The last
//                         block of a row tile to finish (a counter per row tile) adds the h tiles in index order,
//                         adds b2 and applies the probability map, so the result does not depend on block order.
// Every wait is bounded; on expiry the block records ARROL_DEV_WAIT_EXPIRED, drains and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "score_common.cuh"
#include "tc_common.cuh"

namespace {

constexpr int SBM = 128;                     // rollouts per tile (MMA M)
constexpr int SBN = 64;                      // hidden units per tile (MMA N)
constexpr int S_PAIRS = 2;                   // producer / MMA-issuer thread pairs, each with its own ring and accumulator
constexpr int S_RING = 4;                    // stages per pair
constexpr int S_STAGES = S_PAIRS * S_RING;
constexpr int SA_BYTES = SBM * BK * 2;       // 16 KB
constexpr int SB_BYTES = SBN * BK * 2;       //  8 KB
constexpr int S_STAGE_BYTES = SA_BYTES + SB_BYTES;
constexpr int S_TMEM_COLS = S_PAIRS * SBN;   // a power of two >= 32
constexpr int S_THREADS = (2 * S_PAIRS + 4) * 32;   // producers, issuers, four epilogue warps
constexpr int S_TAIL_BYTES = 1024;           // barriers, tensor-memory slot, flags, b1 / w2 of the tile
constexpr size_t S_SMEM_BYTES = (size_t)S_STAGES * S_STAGE_BYTES + 1024 + S_TAIL_BYTES;

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
    uint8_t* stage_b = smem + (size_t)S_STAGES * SA_BYTES;
    uint8_t* tail = smem + (size_t)S_STAGES * S_STAGE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(tail);          // [S_STAGES] TMA -> MMA
    uint64_t* empty = full + S_STAGES;                           // [S_STAGES] MMA -> TMA
    uint64_t* acc_full = empty + S_STAGES;                       // [1] every MMA of the block has finished
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;
    volatile uint32_t* is_last = tmem_slot + 2;
    float* b1_s = reinterpret_cast<float*>(tail + 256);          // [SBN]
    float* w2_s = b1_s + SBN;                                    // [SBN]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * SBM, j0 = blockIdx.y * SBN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        mbar_init(acc_full, S_PAIRS);
        *abort_flag = 0u;
        *is_last = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_x) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    }
    if (warp == S_PAIRS) {                  // first MMA warp owns the tensor-memory allocation
        tcgen05_alloc(tmem_slot, S_TMEM_COLS);
        tcgen05_relinquish();
    }
    pdl_launch_dependents();
    pdl_wait();                  // set-up above overlaps the previous kernel; global memory is read from here on
    if (warp >= 2 * S_PAIRS) {   // the tile's slice of b1 and w2, zero past h so that padded columns add nothing
        const int e = threadIdx.x - 2 * S_PAIRS * 32;
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

    // Producer / issuer pair r takes the K steps ks = r, r + S_PAIRS, ... through its own ring of stages into its
    // own accumulator: one thread's wait -> issue -> commit round costs several hundred cycles per K step, far more
    // than the 32 cycles a 128 x 64 x 16 MMA keeps the tensor pipe busy, so the rounds of the pairs overlap.
    if (warp < S_PAIRS) {
        if (lane == 0) {
            const int r = warp;
            const uint32_t s0 = (uint32_t)r * S_RING;
            uint32_t stage = 0, phase = 0, issued = 0;
            bool ok = true;
            for (int ks = r; ks < p.k_steps; ks += S_PAIRS) {
                const uint32_t st = s0 + stage;
                if (!mbar_wait(&empty[st], phase ^ 1u, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&full[st], S_STAGE_BYTES);
                tma_load_2d(stage_a + (size_t)st * SA_BYTES, &map_x, ks * BK, m0, &full[st]);
                tma_load_2d(stage_b + (size_t)st * SB_BYTES, &map_w, ks * BK, j0, &full[st]);
                ++issued;
                if (++stage == S_RING) { stage = 0; phase ^= 1u; }
            }
            if (!ok) {   // let the copies already issued land before the block's shared memory goes away
                const uint32_t pending = issued < (uint32_t)S_RING ? issued : (uint32_t)S_RING;
                uint32_t s = stage, ph = phase;
                for (uint32_t i = 0; i < pending; ++i) {
                    if (s == 0) { s = S_RING - 1; ph ^= 1u; } else { --s; }
                    for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
                        if (mbar_try_wait(&full[s0 + s], ph)) break;
                }
            }
        }
    } else if (warp < 2 * S_PAIRS) {
        if (lane == 0) {
            const int r = warp - S_PAIRS;
            const uint32_t s0 = (uint32_t)r * S_RING;
            const uint32_t d_tmem = tmem_base + (uint32_t)(r * SBN);
            constexpr uint32_t idesc = make_idesc(SBM, SBN);
            uint32_t stage = 0, phase = 0;
            for (int ks = r; ks < p.k_steps; ks += S_PAIRS) {
                const uint32_t st = s0 + stage;
                if (!mbar_wait(&full[st], phase, abort_flag)) break;
                tcgen05_fence_after();
                const uint64_t a_desc = make_smem_desc(smem_u32(stage_a + (size_t)st * SA_BYTES));
                const uint64_t b_desc = make_smem_desc(smem_u32(stage_b + (size_t)st * SB_BYTES));
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k)
                    tcgen05_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                     (ks >= S_PAIRS || k > 0) ? 1u : 0u);
                tcgen05_commit(&empty[st]);
                if (++stage == S_RING) { stage = 0; phase ^= 1u; }
            }
            // Arrives once every MMA issued by this thread has finished: publishes the accumulator on the normal
            // path, and on the give-up path it is what this thread waits for before shared and tensor memory go away.
            tcgen05_commit(acc_full);
            if (*abort_flag)
                for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
                    if (mbar_try_wait(acc_full, 0u)) break;
        }
    } else {
        const int quarter = warp & 3;
        const int m = m0 + quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        const int used_accs = p.k_steps < S_PAIRS ? p.k_steps : S_PAIRS;     // a pair without K steps wrote nothing
        bool ok = mbar_wait(acc_full, 0u, abort_flag);
        ok = __all_sync(0xffffffffu, ok && !*abort_flag) != 0;
        float part = 0.f;
        if (ok) {
            tcgen05_fence_after();
#pragma unroll
            for (int piece = 0; piece < SBN / 32; ++piece) {
                float v[32];
                tcgen05_ld_32x32(tmem_base + lane_addr + piece * 32, v);
                for (int a = 1; a < used_accs; ++a) {      // fixed order: (acc0 + acc1) + ...
                    float w[32];
                    tcgen05_ld_32x32(tmem_base + lane_addr + a * SBN + piece * 32, w);
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) v[jj] += w[jj];
                }
#pragma unroll
                for (int jj = 0; jj < 32; ++jj) {
                    const float u = v[jj] + b1_s[piece * 32 + jj];
                    v[jj] = u;
                    const float g = 0.5f * u * (1.0f + erff(u * 0.70710678118654752440f));
                    part = fmaf(w2_s[piece * 32 + jj], g, part);
                }
                if (p.u_out && m < p.N) {
                    float* urow = p.u_out + (int64_t)m * p.h + j0 + piece * 32;
#pragma unroll
                    for (int jj = 0; jj < 32; jj += 4)      // h % 4 == 0: a float4 never straddles the edge
                        if (j0 + piece * 32 + jj < p.h)
                            *reinterpret_cast<float4*>(urow + jj) = make_float4(v[jj], v[jj + 1], v[jj + 2], v[jj + 3]);
                }
            }
        }
        // The counter protocol runs whatever happened above, so the counters are back at zero after every launch
        // (after an expired wait the scores of the call are not meaningful and the status word says so).
        if (m < p.N) p.partial[(int64_t)blockIdx.y * p.N + m] = part;
        __threadfence();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (threadIdx.x == 2 * S_PAIRS * 32) {
            const uint32_t done = atomicAdd(&p.counters[blockIdx.x], 1u);
            if (done == gridDim.y - 1) {
                *is_last = 1u;
                p.counters[blockIdx.x] = 0u;        // every block of this row tile has arrived: ready for the next call
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

    tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.d_status, ARROL_DEV_WAIT_EXPIRED);
    if (warp == S_PAIRS) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, S_TMEM_COLS);
    }
}

}  // namespace

// Scores of a bf16 MLP head on the tensor cores.  Returns ARROL_ERR_UNSUPPORTED (nothing launched) when the sizes
// do not fit the context's buffers; the caller then takes the SIMT path.
int arrol_internal_score_mlp_tc(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index,
                                int N, const arrol_head* head, int B, const float* q_lut, float* score, float* prob,
                                int32_t* bin, float* q, float* u_out, cudaStream_t s) {
    const int d = head->d, h = head->h;
    const int m_tiles = (N + SBM - 1) / SBM, h_tiles = (h + SBN - 1) / SBN;
    if ((size_t)N * (size_t)h_tiles > ARROL_SCRATCH_FLOATS || m_tiles > ARROL_TILE_COUNTERS)
        return ARROL_ERR_UNSUPPORTED;
    if (row_index && (size_t)N * (size_t)d * 2 > ARROL_PACK_BYTES) return ARROL_ERR_UNSUPPORTED;
    if (!row_index && ((uint64_t)row_stride * 2) >= (1ull << 40)) return ARROL_ERR_UNSUPPORTED;

    const void* x = hidden;
    int64_t ld = row_stride;
    if (row_index) {
        ARROL_CUDA_OK(arrol_launch_pdl(pack_rows_kernel, dim3((N + 3) / 4), dim3(128), 0, s,
                                       static_cast<const __nv_bfloat16*>(hidden), row_stride, row_index, N, d,
                                       static_cast<__nv_bfloat16*>(ctx->d_pack), ctx->source_rows, ctx->d_status));
        ctx->launches += 1;
        x = ctx->d_pack;
        ld = d;
    }
    CUtensorMap map_x, map_w;
    if (make_map_ld(ctx, &map_x, x, (uint64_t)N, (uint64_t)d, (uint64_t)ld, SBM) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map(ctx, &map_w, head->W1, (uint64_t)h, (uint64_t)d, SBN) != ARROL_OK) return ARROL_ERR_CUDA;

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
    if (!ctx->score_tc_smem_set) {      // once per context: this call is on the prune step's microsecond path
        ARROL_CUDA_OK(cudaFuncSetAttribute(score_mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)S_SMEM_BYTES));
        ctx->score_tc_smem_set = true;
    }
    dim3 grid(m_tiles, h_tiles);
    ARROL_CUDA_OK(arrol_launch_pdl(score_mlp_tc_kernel, grid, dim3(S_THREADS), S_SMEM_BYTES, s, map_x, map_w, p));
    ctx->launches += 1;
    return ARROL_OK;
}
