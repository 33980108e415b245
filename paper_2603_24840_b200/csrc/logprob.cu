// arrol_token_logprob: selected-token log-probability of every survivor token from the lm_head
// (Section 3: log pi_theta(o_t | o_<t); Algorithm 1 "log-probs on R'"), as a fused contraction
// hidden[T,d] x W_vocab[V,d]^T with an online max / log-sum-exp epilogue.  The T x V logits never leave the SM.
//
// One thread block per SM, persistent over work items (token tile of 128 rows, vocabulary split).  Per item the
// block walks its vocabulary range in chunks of 256 columns.  Warp roles:
//   warp 0      TMA producer: K-major, 128-byte-swizzled tiles of hidden (128 x 64) and W_vocab (256 x 64) into
//               a ring of shared-memory stages, completion on mbarriers
//   warp 1      tcgen05.mma issuer (one elected lane): 128 x 256 x 16 bf16 MMAs into one of two 256-column fp32
//               accumulators in tensor memory; tcgen05.commit releases stages / publishes accumulators
//   warps 2..5  epilogue: thread r owns token row r of the tile; tcgen05.ld of its accumulator row, running
//               maximum and sum of 2^(z log2e - max), and the target column's logit, all in registers
// The two accumulators let the epilogue of chunk c overlap the MMAs of chunk c + 1.
// Every wait is bounded; when one runs out the block records ARROL_DEV_WAIT_EXPIRED, drains and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128;          // token rows per tile  (MMA M)
constexpr int BN = 256;          // vocabulary columns per chunk (MMA N)
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
constexpr int B_STAGE_BYTES = BN * BK * 2;   // 32 KB
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int TMEM_COLS = 512;   // two fp32 accumulators of BN columns
constexpr int NUM_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr size_t SMEM_BYTES = (size_t)STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

struct PartialLse {   // per (split, token): running maximum and sum in the base-2 domain, target logit,
    float m2, l, zy2, pad;   // pad: sum of the raw accumulators of the split (only when the confidence is asked for)
};

struct LogprobParams {
    const int32_t* targets;
    const int64_t* d_T;
    int64_t T_max;
    int d, V;
    int splits;            // vocabulary splits per token tile
    int chunks_per_split;  // chunks of BN columns per split
    float scale2;          // inv_temperature * log2(e)
    float* logp;
    float* lse;
    float* conf;           // token confidence H_t = -sum_v log P_t(v) = V lse - sum_v z_v, or NULL
    float inv_temp;
    PartialLse* partial;   // [splits][T_max] when splits > 1
    uint32_t spin_limit;   // tries per pipeline wait
    int mute_producer;     // test hook: the producer issues no copies
    uint32_t* d_status;
};

template <bool CONF>
__global__ void __launch_bounds__(NUM_THREADS, 1)
token_logprob_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                     const LogprobParams p) {
    extern __shared__ uint8_t smem_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_a = smem;
    uint8_t* stage_b = smem + (size_t)STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t* full = bars;                    // [STAGES]  TMA -> MMA
    uint64_t* empty = bars + STAGES;          // [STAGES]  MMA -> TMA
    uint64_t* acc_full = bars + 2 * STAGES;   // [2]       MMA -> epilogue
    uint64_t* acc_empty = acc_full + 2;       // [2]       epilogue -> MMA
    uint64_t* drain = acc_empty + 2;          // [1]       used only when giving up: MMAs in flight -> done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    int64_t T = p.T_max;
    if (p.d_T) { const int64_t t = *p.d_T; T = t < 0 ? 0 : (t < T ? t : T); }
    const int64_t m_tiles = (T + BM - 1) / BM;
    const int64_t items = m_tiles * p.splits;
    const int k_steps = (p.d + BK - 1) / BK;
    const int total_chunks = (p.V + BN - 1) / BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], EPI_THREADS / 32); }
        mbar_init(drain, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
    }
    if (warp == 1) {
        tcgen05_alloc(tmem_slot, TMEM_COLS);
        tcgen05_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            for (int64_t item = blockIdx.x; item < items && ok && !p.mute_producer; item += gridDim.x) {
                const int m_tile = (int)(item / p.splits), split = (int)(item % p.splits);
                const int c0 = split * p.chunks_per_split;
                const int c1 = min(c0 + p.chunks_per_split, total_chunks);
                for (int c = c0; c < c1 && ok; ++c) {
                    for (int ks = 0; ks < k_steps; ++ks) {
                        if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
                        mbar_expect_tx(&full[stage], STAGE_BYTES);
                        tma_load_2d(stage_a + (size_t)stage * A_STAGE_BYTES, &map_h, ks * BK, m_tile * BM, &full[stage]);
                        tma_load_2d(stage_b + (size_t)stage * B_STAGE_BYTES, &map_w, ks * BK, c * BN, &full[stage]);
                        ++issued;
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!ok) {
                // Gave up: let the copies already issued land before the block's shared memory goes away.
                // The last min(issued, STAGES) stages may still be in flight; wait for each (bounded).
                const uint32_t pending = issued < (uint32_t)STAGES ? issued : (uint32_t)STAGES;
                uint32_t s = stage, ph = phase;
                for (uint32_t i = 0; i < pending; ++i) {
                    if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
                    for (uint32_t it = 0; it < p.spin_limit; ++it)
                        if (mbar_try_wait(&full[s], ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc(BM, BN);
            uint32_t stage = 0, phase = 0;
            uint32_t acc = 0, acc_phase = 0;
            bool ok = true;
            for (int64_t item = blockIdx.x; item < items && ok; item += gridDim.x) {
                const int split = (int)(item % p.splits);
                const int c0 = split * p.chunks_per_split;
                const int c1 = min(c0 + p.chunks_per_split, total_chunks);
                for (int c = c0; c < c1 && ok; ++c) {
                    if (!mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
                    tcgen05_fence_after();
                    const uint32_t d_tmem = tmem_base + acc * BN;
                    for (int ks = 0; ks < k_steps; ++ks) {
                        if (!mbar_wait(&full[stage], phase, abort_flag, p.spin_limit)) { ok = false; break; }
                        tcgen05_fence_after();
                        const uint64_t a_desc = make_smem_desc(smem_u32(stage_a + (size_t)stage * A_STAGE_BYTES));
                        const uint64_t b_desc = make_smem_desc(smem_u32(stage_b + (size_t)stage * B_STAGE_BYTES));
#pragma unroll
                        for (int k = 0; k < BK / UMMA_K; ++k) {
                            // advancing K by 16 elements = 32 bytes inside the swizzle row: +2 in address units
                            tcgen05_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                             (ks | k) != 0 ? 1u : 0u);
                        }
                        tcgen05_commit(&empty[stage]);   // stage reusable once these MMAs have read it
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) tcgen05_commit(&acc_full[acc]);   // accumulator complete
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
            }
            if (!ok) {
                // Gave up: wait (bounded) until the MMAs already issued have finished with shared and tensor memory.
                tcgen05_commit(drain);
                for (uint32_t it = 0; it < p.spin_limit; ++it)
                    if (mbar_try_wait(drain, 0u)) break;
            }
        }
    } else {
        // ---------------- epilogue: one token row per thread ----------------
        const int quarter = warp & 3;                       // TMEM lanes 32*quarter .. 32*quarter+31
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int64_t item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int m_tile = (int)(item / p.splits), split = (int)(item % p.splits);
            const int c0 = split * p.chunks_per_split;
            const int c1 = min(c0 + p.chunks_per_split, total_chunks);
            const int64_t t = (int64_t)m_tile * BM + row_in_tile;
            const int y = (t < T) ? p.targets[t] : -1;
            float m2 = -INFINITY, l = 0.f, zy2 = -INFINITY, sumz = 0.f;
            for (int c = c0; c < c1 && ok; ++c) {
                ok = mbar_wait(&acc_full[acc], acc_phase, abort_flag, p.spin_limit);
                ok = __all_sync(0xffffffffu, ok) != 0;     // keep the warp converged for the aligned tensor-memory loads
                if (!ok) break;
                tcgen05_fence_after();
                const int col0 = c * BN;
#pragma unroll 1
                for (int piece = 0; piece < BN / 32; ++piece) {
                    const int pc0 = col0 + piece * 32;
                    if (pc0 >= p.V) break;                  // columns past the vocabulary (zero-filled by TMA)
                    float v[32];
                    tcgen05_ld_32x32(tmem_base + lane_addr + acc * BN + piece * 32, v);
                    if constexpr (CONF) {                   // sum of the valid logits of the piece (before masking)
                        float ps[4] = {0.f, 0.f, 0.f, 0.f};           // four chains; only the last piece needs the mask
                        if (pc0 + 32 <= p.V) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) ps[j & 3] += v[j];
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) ps[j & 3] += (pc0 + j < p.V) ? v[j] : 0.f;
                        }
                        sumz += (ps[0] + ps[1]) + (ps[2] + ps[3]);
                    }
                    if (pc0 + 32 > p.V) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (pc0 + j >= p.V) v[j] = -INFINITY;
                    }
                    if ((unsigned)(y - pc0) < 32u) {
                        const int jy = y - pc0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) if (j == jy) zy2 = v[j] * p.scale2;
                    }
                    float bmax = v[0];
#pragma unroll
                    for (int j = 1; j < 32; ++j) bmax = fmaxf(bmax, v[j]);
                    const float m_new = fmaxf(m2, bmax * p.scale2);
                    float sum = 0.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) sum += ex2_approx(fmaf(v[j], p.scale2, -m_new));
                    l = fmaf(l, ex2_approx(m2 - m_new), sum);
                    m2 = m_new;
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[acc]);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (ok && t < T) {
                if (p.splits == 1) {
                    const float lse2 = m2 + log2f(l);
                    const float ln2 = 0.69314718055994530942f;
                    float out = 0.f;
                    if (y >= 0) {
                        if (y < p.V) out = (zy2 - lse2) * ln2;
                        else atomicOr(p.d_status, ARROL_DEV_BAD_TARGET);
                    }
                    p.logp[t] = out;
                    if (p.lse) p.lse[t] = lse2 * ln2;
                    if constexpr (CONF) p.conf[t] = (float)p.V * (lse2 * ln2) - sumz * p.inv_temp;
                } else {
                    PartialLse pr;
                    pr.m2 = m2; pr.l = l; pr.zy2 = zy2; pr.pad = sumz;
                    *reinterpret_cast<float4*>(&p.partial[(int64_t)split * p.T_max + t]) =
                        make_float4(pr.m2, pr.l, pr.zy2, pr.pad);
                }
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.d_status, ARROL_DEV_WAIT_EXPIRED);
    if (warp == 1) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, TMEM_COLS);
    }
}

// Merge of the per-split (max, sum, target logit) triples: M = max m_s, L = sum l_s 2^(m_s - M).
__global__ void combine_splits_kernel(const PartialLse* __restrict__ partial, const int32_t* __restrict__ targets,
                                      const int64_t* __restrict__ d_T, int64_t T_max, int V, int splits,
                                      float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ conf,
                                      float inv_temp, uint32_t* d_status) {
    int64_t T = T_max;
    if (d_T) { const int64_t t = *d_T; T = t < 0 ? 0 : (t < T ? t : T); }
    for (int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; t < T; t += (int64_t)gridDim.x * blockDim.x) {
        float M = -INFINITY, zy2 = -INFINITY;
        for (int s = 0; s < splits; ++s) {
            const float4 pr = *reinterpret_cast<const float4*>(&partial[(int64_t)s * T_max + t]);
            M = fmaxf(M, pr.x);
            zy2 = fmaxf(zy2, pr.z);          // exactly one split holds the target column; the others hold -inf
        }
        float L = 0.f, sumz = 0.f;
        for (int s = 0; s < splits; ++s) {
            const float4 pr = *reinterpret_cast<const float4*>(&partial[(int64_t)s * T_max + t]);
            L += pr.y * exp2f(pr.x - M);
            sumz += pr.w;
        }
        const float lse2 = M + log2f(L);
        const float ln2 = 0.69314718055994530942f;
        const int y = targets[t];
        float out = 0.f;
        if (y >= 0) {
            if (y < V) out = (zy2 - lse2) * ln2;
            else atomicOr(d_status, ARROL_DEV_BAD_TARGET);
        }
        logp[t] = out;
        if (lse) lse[t] = lse2 * ln2;
        if (conf) conf[t] = (float)V * (lse2 * ln2) - sumz * inv_temp;
    }
}

// How many vocabulary splits per token tile.  With one split every resident block streams a different token
// tile (128 x d x 2 bytes each) against the same W chunks; when those tiles together outgrow about half of L2
// the tiles are re-fetched from HBM once per chunk, so the vocabulary is split until they fit (80 MB of the 126 MB L2).
int choose_splits(const arrol_ctx* ctx, int64_t T_max, int d, int V) {
    const int total_chunks = (V + BN - 1) / BN;
    const int64_t m_tiles = (T_max + BM - 1) / BM;
    int splits = 1;
    const double l2_budget = 80.0 * 1024 * 1024;   // measured: 74 MB of token tiles still stay L2-resident, 148 MB thrash
    const double tile_bytes = (double)BM * d * 2;
    while (splits < 8 && (ctx->sm_count / splits) * tile_bytes > l2_budget) splits *= 2;
    // few token tiles: split so that every SM has work
    while (splits < 16 && m_tiles * splits < ctx->sm_count && splits * 2 <= total_chunks) splits *= 2;
    if (splits > total_chunks) splits = total_chunks;
    return splits < 1 ? 1 : splits;
}

}  // namespace

extern "C" size_t arrol_token_logprob_workspace(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V) {
    if (!ctx || T_max <= 0 || d <= 0 || V <= 0) return 0;
    // splits x tokens partial records.  Few token tiles get more splits (to fill the SMs) but then splits x tokens stays
    // below two waves of tiles, so flooring the count there makes the size monotone in T_max: a workspace sized for
    // T_max also serves any call on fewer tokens with the same d and V.
    const int splits = choose_splits(ctx, T_max, d, V);
    const size_t floor_records = (size_t)2 * ctx->sm_count * BM;
    size_t records = (size_t)(splits > 1 ? splits : 0) * (size_t)T_max;
    if (records < floor_records) records = floor_records;
    return records * sizeof(PartialLse) + 256;
}

extern "C" int32_t arrol_token_logprob_splits(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V) {
    if (!ctx || T_max <= 0 || d <= 0 || V <= 0) return 0;
    const int total_chunks = (V + BN - 1) / BN;
    int splits = choose_splits(ctx, T_max, d, V);
    const int chunks_per_split = (total_chunks + splits - 1) / splits;
    return (total_chunks + chunks_per_split - 1) / chunks_per_split;
}

static int run_token_logprob(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                             int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                             float* logp, float* lse, float* conf, void* workspace, size_t workspace_bytes,
                             void* stream) {
    if (!ctx || T_max < 0 || d <= 0 || V <= 0 || !(inv_temperature > 0.f)) return ARROL_ERR_INVALID_ARG;
    if (T_max == 0) return ARROL_OK;
    if (!hidden || !W_vocab || !targets || !logp) return ARROL_ERR_INVALID_ARG;
    if (d % 8 != 0) return ARROL_ERR_UNSUPPORTED;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(W_vocab, 16)) return ARROL_ERR_INVALID_ARG;
    if (T_max > (int64_t)INT32_MAX - BM) return ARROL_ERR_UNSUPPORTED;   // TMA coordinates are 32-bit
    const size_t need = arrol_token_logprob_workspace(ctx, T_max, d, V);
    if (!workspace || workspace_bytes < need || !arrol_aligned(workspace, 256)) return ARROL_ERR_WORKSPACE;

    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;

    CUtensorMap map_h, map_w;
    if (make_map(ctx, &map_h, hidden, (uint64_t)T_max, (uint64_t)d, BM) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map(ctx, &map_w, W_vocab, (uint64_t)V, (uint64_t)d, BN) != ARROL_OK) return ARROL_ERR_CUDA;

    LogprobParams p;
    p.targets = targets;
    p.d_T = d_T;
    p.T_max = T_max;
    p.d = d;
    p.V = V;
    p.splits = choose_splits(ctx, T_max, d, V);
    const int total_chunks = (V + BN - 1) / BN;
    p.chunks_per_split = (total_chunks + p.splits - 1) / p.splits;
    p.splits = (total_chunks + p.chunks_per_split - 1) / p.chunks_per_split;   // no empty split
    p.scale2 = inv_temperature * 1.44269504088896340736f;
    p.logp = logp;
    p.lse = lse;
    p.conf = conf;
    p.inv_temp = inv_temperature;
    p.partial = static_cast<PartialLse*>(workspace);
    p.d_status = ctx->d_status;
    p.spin_limit = ctx->test_spin_limit ? ctx->test_spin_limit : SPIN_LIMIT;
    p.mute_producer = ctx->test_mute_producer;

    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SMEM_BYTES));
    const int64_t m_tiles = (T_max + BM - 1) / BM;
    int64_t grid = m_tiles * p.splits;
    if (grid > ctx->sm_count) grid = ctx->sm_count;
    if (conf) token_logprob_kernel<true><<<(unsigned)grid, NUM_THREADS, SMEM_BYTES, s>>>(map_h, map_w, p);
    else token_logprob_kernel<false><<<(unsigned)grid, NUM_THREADS, SMEM_BYTES, s>>>(map_h, map_w, p);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    if (p.splits > 1) {
        int64_t blocks = (T_max + 255) / 256;
        if (blocks > (int64_t)ctx->sm_count * 8) blocks = (int64_t)ctx->sm_count * 8;
        combine_splits_kernel<<<(unsigned)blocks, 256, 0, s>>>(p.partial, targets, d_T, T_max, V, p.splits, logp,
                                                              lse, conf, inv_temperature, ctx->d_status);
        ctx->launches += 1;
        ARROL_CUDA_OK(cudaGetLastError());
    }
    return ARROL_OK;
}

extern "C" int arrol_token_logprob(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                                   int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                                   float* logp, float* lse, void* workspace, size_t workspace_bytes,
                                   void* stream) {
    return run_token_logprob(ctx, hidden, W_vocab, targets, T_max, d_T, d, V, inv_temperature, logp, lse, nullptr,
                             workspace, workspace_bytes, stream);
}

extern "C" int arrol_token_logprob_conf(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                                        int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                                        float* logp, float* lse, float* token_conf, void* workspace,
                                        size_t workspace_bytes, void* stream) {
    if (T_max > 0 && !token_conf) return ARROL_ERR_INVALID_ARG;
    return run_token_logprob(ctx, hidden, W_vocab, targets, T_max, d_T, d, V, inv_temperature, logp, lse, token_conf,
                             workspace, workspace_bytes, stream);
}
