// arrol_token_logprob: selected-token log-probability of every survivor token from the lm_head
// (Section 3: log pi_theta(o_t | o_<t); Algorithm 1 "log-probs on R'"), as a fused contraction
// hidden[T,d] x W_vocab[V,d]^T with an online max / log-sum-exp epilogue.  The T x V logits never leave the SM.
//
// One thread block per SM, persistent over work items (token tile, vocabulary split).  By default the blocks work as
// PAIRS (clusters of two, tcgen05 cta_group::2) on 256-row token tiles, see PAIR below; described first is the
// one-block form on 128-row tiles, which the pair form extends.  Per item the block walks its vocabulary range in
// chunks of 256 columns.  Warp roles:
//   warp 0      TMA producer: K-major, 128-byte-swizzled tiles of hidden (128 x 64) and W_vocab (256 x 64) into
//               a ring of shared-memory stages, completion on mbarriers
//   warp 1      tcgen05.mma issuer (one elected lane): 128 x 256 x 16 bf16 MMAs into one of two 256-column fp32
//               accumulators in tensor memory; tcgen05.commit releases stages / publishes accumulators
//   warps 2..5  epilogue: thread r owns token row r of the tile; tcgen05.ld of its accumulator row, running
//               maximum and sum of 2^(z log2e - max), and the target column's logit, all in registers
// The two accumulators let the epilogue of chunk c overlap the MMAs of chunk c + 1.
//
// Waves in step.  The resident blocks all stream the same W_vocab chunks; as long as they do so at about the same
// time a chunk comes from HBM once and from L2 147 times.  Nothing in a persistent kernel keeps them together,
// though: measured on 6.5 M tokens (1,373 work items per block), the blocks' start times spread from 0.02 of an item
// after two waves to 2 items after 50 and 40 items after 800; once a block lags by more than L2 holds it re-streams
// its chunks from HBM, falls further behind, and the extra HBM traffic costs power: the SM clock under the 1 kW cap
// fell from 1.40 GHz in the first waves to 0.72 GHz.  So the blocks are held in step: before issuing the loads of
// wave k (its k-th work item) every producer arrives on a counter in global memory and waits until all blocks have
// arrived for that wave.  All blocks must then be resident: single blocks are launched cooperatively whenever there is
// more than one wave; for pairs the host asks cudaOccupancyMaxActiveClusters how many fit at once and launches no
// more (a cooperative launch of clusters that fills the GPU is the one launch the profiler cannot make).  Like every
// other wait this one is bounded.
// Every wait is bounded; when one runs out the block records ARROL_DEV_WAIT_EXPIRED, drains and returns.
//
// Gathered variant (arrol_token_logprob_gathered; Section 4.3 (ii): the survivors are re-batched "to compute
// log-probabilities"): the token rows are read straight from the pre-prune source buffer, so the packed copy of the
// hidden rows never exists.  A 128-row token tile that lies inside one survivor is 128 consecutive source rows: its
// TMA box simply starts at that source row.  Only a tile that crosses a survivor boundary is not contiguous in the
// source; those tiles (at most one per survivor) are first copied into a small scratch block, slot = the survivor
// of the tile's first row, by pack_boundary_tiles_kernel, and the main kernel reads them from there through a second
// tensor map.  Every tile therefore costs the same single box per K step.  That matters beyond the tile itself: the
// resident blocks stream the same W_vocab chunks at about the same time and share them through L2, and a block that
// falls behind by more than the L2 holds has to re-fetch its chunks from HBM (measured with multi-box copies for the
// boundary tiles: +10 % cycles on those tiles spread the blocks out, HBM traffic and power rose, and the SM clock
// fell from 1.27 to 0.8 GHz under the power cap).
#include <cuda.h>
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128;          // token rows per tile  (MMA M)
constexpr int BN = 256;          // vocabulary columns per chunk (MMA N)
constexpr int SOLO_STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;   // 16 KB
constexpr int SOLO_B_STAGE_BYTES = BN * BK * 2;   // 32 KB
constexpr int SOLO_STAGE_BYTES = A_STAGE_BYTES + SOLO_B_STAGE_BYTES;
// pair variant (two blocks of a cluster on one 256-row tile): every block stages its 128 rows of A and its half of
// the B tile, so a stage is 32 KB and six of them fit
constexpr int PAIR_STAGES = 6;
constexpr int PAIR_B_ROWS = BN / 2;
constexpr int PAIR_B_STAGE_BYTES = PAIR_B_ROWS * BK * 2;   // 16 KB
constexpr int PAIR_STAGE_BYTES = A_STAGE_BYTES + PAIR_B_STAGE_BYTES;
static_assert(PAIR_STAGES * PAIR_STAGE_BYTES == SOLO_STAGES * SOLO_STAGE_BYTES, "both variants fill the same shared memory");
constexpr int TMEM_COLS = 512;   // two fp32 accumulators of BN columns
constexpr int NUM_THREADS = 192;
constexpr int EPI_THREADS = 128;
constexpr size_t SMEM_BYTES = (size_t)SOLO_STAGES * SOLO_STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;

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
    // gathered variant: packed token t of survivor s is source row src_tok_off[survivor_idx[s]] + (t - cu_seqlens[s])
    const int64_t* cu_seqlens;
    const int32_t* survivor_idx;
    const int64_t* src_tok_off;
    const int64_t* d_num;  // {S, T}
    int S_max;
    unsigned int* wave_counter;   // producers that have arrived, over all waves of this launch (zeroed before it)
    unsigned long long* timing;   // test hook: per work item {globaltimer start, end, clock64 start, end}, or NULL
    int64_t timing_items;
};

__device__ __forceinline__ unsigned int ld_acquire_u32(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

// Survivor of packed token row t: the last s in [0, S) with cu_seqlens[s] <= t (this skips empty survivors).
__device__ __forceinline__ int survivor_of_row(const int64_t* __restrict__ cu_seqlens, int S, int64_t t) {
    int lo = 0, hi = S;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu_seqlens[mid] <= t) lo = mid; else hi = mid;
    }
    return lo;
}

// GATHER: map_h covers the pre-prune source rows and map_s the scratch of pre-packed boundary tiles
// ([S_max * 128, d], slot s at rows 128 s ...); otherwise map_h covers the packed rows and map_s is unused.
// PAIR: the kernel runs as clusters of two blocks; a pair works on 256 token rows (block r of the pair owns rows
// 128 r ...), block 0 issues 256 x 256 x 16 MMAs (cta_group::2) that read both blocks' shared memory and write both
// blocks' tensor memory, every block loads its own 128 rows of A and its own 128 of the chunk's 256 W_vocab rows and
// runs the epilogue of its own rows.  Per block and K step 32 KB come in from L2 instead of 48 KB and the tensor
// core reads 8 KB of operands per MMA from shared memory instead of 12 KB.
template <bool CONF, bool GATHER, bool PAIR>
__global__ void __launch_bounds__(NUM_THREADS, 1)
token_logprob_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_s,
                     const __grid_constant__ CUtensorMap map_w, const LogprobParams p) {
    constexpr int STAGES = PAIR ? PAIR_STAGES : SOLO_STAGES;
    constexpr int B_STAGE_BYTES = PAIR ? PAIR_B_STAGE_BYTES : SOLO_B_STAGE_BYTES;
    constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* stage_a = smem;
    uint8_t* stage_b = smem + (size_t)STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
    uint64_t* full = bars;                    // [STAGES]  TMA -> MMA (pair: block 0's receive both blocks' bytes)
    uint64_t* empty = bars + STAGES;          // [STAGES]  MMA -> TMA
    uint64_t* acc_full = bars + 2 * STAGES;   // [2]       MMA -> epilogue
    uint64_t* acc_empty = acc_full + 2;       // [2]       epilogue -> MMA
    uint64_t* drain = acc_empty + 2;          // [1]       used only when giving up: MMAs in flight -> done
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
    volatile uint32_t* abort_flag = tmem_slot + 1;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // pair: rank of this block in its cluster (block 0 leads), unit = cluster; otherwise unit = block
    const uint32_t rank = PAIR ? cluster_cta_rank() : 0u;
    const int64_t unit = PAIR ? (int64_t)(blockIdx.x >> 1) : (int64_t)blockIdx.x;
    const int64_t units = PAIR ? (int64_t)(gridDim.x >> 1) : (int64_t)gridDim.x;

    int64_t T = p.T_max;
    if (p.d_T) { const int64_t t = *p.d_T; T = t < 0 ? 0 : (t < T ? t : T); }
    const int64_t m_tiles = (T + BM - 1) / BM;
    const int64_t items = (PAIR ? (m_tiles + 1) / 2 : m_tiles) * p.splits;   // (pairs of) token tiles x splits
    const int k_steps = (p.d + BK - 1) / BK;
    const int total_chunks = (p.V + BN - 1) / BN;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        // pair: the leading block's acc_empty collects the epilogue warps of both blocks
        for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], (PAIR ? 2 : 1) * (EPI_THREADS / 32)); }
        mbar_init(drain, 1);
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_h) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
        if constexpr (GATHER) asm volatile("prefetch.tensormap [%0];" ::"l"(&map_s) : "memory");
    }
    if (warp == 1) {
        if constexpr (PAIR) { tcgen05_alloc_pair(tmem_slot, TMEM_COLS); tcgen05_relinquish_pair(); }
        else { tcgen05_alloc(tmem_slot, TMEM_COLS); tcgen05_relinquish(); }
    }
    tcgen05_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();     // the peer's barriers exist before anything arrives on them
    tcgen05_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // pair: shared::cluster addresses, in the leading block, of the barriers both blocks signal
    uint32_t lead_full0 = 0, lead_acc_empty0 = 0;
    if constexpr (PAIR) {
        lead_full0 = map_to_cta(smem_u32(&full[0]), 0u);
        lead_acc_empty0 = map_to_cta(smem_u32(&acc_empty[0]), 0u);
    }

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            uint32_t stage = 0, phase = 0;
            uint32_t issued = 0;
            bool ok = true;
            int S = 0;
            if constexpr (GATHER) {
                const int64_t s64 = p.d_num[0];
                S = (int)(s64 < 0 ? 0 : (s64 > (int64_t)p.S_max ? (int64_t)p.S_max : s64));
            }
            const int64_t waves = (items + units - 1) / units;
            unsigned int wave = 0;
            for (int64_t item = unit; ok && !p.mute_producer; item += units, ++wave) {
                if (wave > 0 && wave < waves) {
                    // hold the blocks in step: arrive for this wave (one arrival per unit), then wait for everybody (a
                    // unit without a work item in the last, partial wave arrives as well and leaves)
                    if (rank == 0) {
                        __threadfence();
                        atomicAdd(p.wave_counter, 1u);
                    }
                    if (item < items) {
                        const unsigned int target = wave * (unsigned int)units;
                        uint32_t it = 0;
                        while (ld_acquire_u32(p.wave_counter) < target) {
                            __nanosleep(64);
                            if (++it >= p.spin_limit || ((it & 1023u) == 1023u && *abort_flag)) { ok = false; break; }
                        }
                        if (!ok) { *abort_flag = 1u; break; }
                    }
                }
                if (item >= items) break;
                const int tile_unit = (int)(item / p.splits), split = (int)(item % p.splits);
                const int m_tile = PAIR ? 2 * tile_unit + (int)rank : tile_unit;      // this block's 128 rows
                const int c0 = split * p.chunks_per_split;
                const int c1 = min(c0 + p.chunks_per_split, total_chunks);
                // where the tile's 128 rows come from: the packed rows, a run of source rows, or a scratch slot
                const CUtensorMap* a_map = &map_h;
                int a_row = m_tile * BM;
                if constexpr (GATHER) {
                    const int64_t t0 = (int64_t)m_tile * BM;
                    a_row = 0;                              // a pair's second tile may lie past T: any rows will do
                    if (t0 < T) {
                        const int s0 = survivor_of_row(p.cu_seqlens, S, t0);
                        const int64_t s_end = p.cu_seqlens[s0 + 1];
                        if (s_end < t0 + BM && s_end < T) {     // the tile runs on into the next survivor: pre-packed
                            a_map = &map_s;
                            a_row = s0 * BM;
                        } else {
                            a_row = (int)(p.src_tok_off[p.survivor_idx[s0]] + (t0 - p.cu_seqlens[s0]));
                        }
                    }
                }
                for (int c = c0; c < c1 && ok; ++c) {
                    for (int ks = 0; ks < k_steps; ++ks) {
                        if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag, p.spin_limit)) { ok = false; break; }
                        if constexpr (PAIR) {
                            // both blocks' bytes are counted on the leading block's barrier
                            const uint32_t bar = lead_full0 + stage * (uint32_t)sizeof(uint64_t);
                            if (rank == 0) mbar_expect_tx(&full[stage], 2 * STAGE_BYTES);
                            tma_load_2d_pair(stage_a + (size_t)stage * A_STAGE_BYTES, a_map, ks * BK, a_row, bar);
                            tma_load_2d_pair(stage_b + (size_t)stage * B_STAGE_BYTES, &map_w, ks * BK,
                                             c * BN + (int)rank * PAIR_B_ROWS, bar);
                        } else {
                            mbar_expect_tx(&full[stage], STAGE_BYTES);
                            tma_load_2d(stage_a + (size_t)stage * A_STAGE_BYTES, a_map, ks * BK, a_row, &full[stage]);
                            tma_load_2d(stage_b + (size_t)stage * B_STAGE_BYTES, &map_w, ks * BK, c * BN, &full[stage]);
                        }
                        ++issued;
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                }
            }
            if (!ok && rank == 0) {
                // Gave up: let the copies already issued land before the block's shared memory goes away.
                // The last min(issued, STAGES) stages may still be in flight; wait for each (bounded).  (In a pair the
                // second block's copies are counted on the leading block's barriers; the cluster barrier at the end
                // of the kernel keeps its shared memory alive until the leading block has got here.)
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
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = make_idesc(PAIR ? 2 * BM : BM, BN);
            uint32_t stage = 0, phase = 0;
            uint32_t acc = 0, acc_phase = 0;
            bool ok = true;
            for (int64_t item = unit; item < items && ok; item += units) {
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
                            if constexpr (PAIR)
                                tcgen05_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                                      (ks | k) != 0 ? 1u : 0u);
                            else
                                tcgen05_mma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                                 (ks | k) != 0 ? 1u : 0u);
                        }
                        // stage reusable (in both blocks of a pair) once these MMAs have read it
                        if constexpr (PAIR) tcgen05_commit_pair(&empty[stage], (uint16_t)3);
                        else tcgen05_commit(&empty[stage]);
                        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                    }
                    if (ok) {                                 // accumulator complete
                        if constexpr (PAIR) tcgen05_commit_pair(&acc_full[acc], (uint16_t)3);
                        else tcgen05_commit(&acc_full[acc]);
                    }
                    if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
                }
            }
            if (!ok) {
                // Gave up: wait (bounded) until the MMAs already issued have finished with shared and tensor memory.
                if constexpr (PAIR) tcgen05_commit_pair(drain, (uint16_t)1);
                else tcgen05_commit(drain);
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
        for (int64_t item = unit; item < items && ok; item += units) {
            const int tile_unit = (int)(item / p.splits), split = (int)(item % p.splits);
            const int m_tile = PAIR ? 2 * tile_unit + (int)rank : tile_unit;
            const int c0 = split * p.chunks_per_split;
            const int c1 = min(c0 + p.chunks_per_split, total_chunks);
            const int64_t t = (int64_t)m_tile * BM + row_in_tile;
            const int y = (t < T) ? p.targets[t] : -1;
            float m2 = -INFINITY, l = 0.f, zy2 = -INFINITY, sumz = 0.f;
            const bool stamp = p.timing != nullptr && threadIdx.x == 64 && rank == 0 && item < p.timing_items;
            if (stamp) { p.timing[4 * item] = global_timer_ns(); p.timing[4 * item + 2] = (unsigned long long)clock64(); }
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
                if (lane == 0) {
                    if constexpr (PAIR) mbar_arrive_cluster(lead_acc_empty0 + acc * (uint32_t)sizeof(uint64_t));
                    else mbar_arrive(&acc_empty[acc]);
                }
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
            if (stamp) { p.timing[4 * item + 1] = global_timer_ns(); p.timing[4 * item + 3] = (unsigned long long)clock64(); }
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
    if constexpr (PAIR) cluster_sync_all();     // neither block's shared or tensor memory goes away under the other
    if (threadIdx.x == 0 && *abort_flag) atomicOr(p.d_status, ARROL_DEV_WAIT_EXPIRED);
    if (warp == 1) {
        tcgen05_fence_after();
        if constexpr (PAIR) tcgen05_dealloc_pair(tmem_base, TMEM_COLS);
        else tcgen05_dealloc(tmem_base, TMEM_COLS);
    }
}

// Gathered variant, first kernel: copies every token tile that crosses a survivor boundary into its scratch slot.
// Block s looks at the tile that holds survivor s's last row: if that tile starts inside s (so s owns it) and runs on
// past the end of s, its rows are copied, run by run, with 16-byte loads/stores (eight in flight per thread).
constexpr int PACK_THREADS = 256;
__global__ void __launch_bounds__(PACK_THREADS)
pack_boundary_tiles_kernel(const uint4* __restrict__ src_rows, const int64_t* __restrict__ cu_seqlens,
                           const int32_t* __restrict__ survivor_idx, const int64_t* __restrict__ src_tok_off,
                           const int64_t* __restrict__ d_num, int S_max, int64_t T_max, int vec_per_row,
                           uint4* __restrict__ scratch) {
    __shared__ int64_t src_row_of[BM];
    pdl_launch_dependents();
    pdl_wait();
    cu_seqlens = pdl_acquire(cu_seqlens); survivor_idx = pdl_acquire(survivor_idx); d_num = pdl_acquire(d_num);
    src_tok_off = pdl_acquire(src_tok_off); src_rows = pdl_acquire(src_rows);
    int64_t S64 = d_num[0], T = d_num[1];
    const int S = (int)(S64 < 0 ? 0 : (S64 > (int64_t)S_max ? (int64_t)S_max : S64));
    T = T < 0 ? 0 : (T < T_max ? T : T_max);
    for (int s0 = blockIdx.x; s0 < S; s0 += gridDim.x) {
        const int64_t begin = cu_seqlens[s0], end = cu_seqlens[s0 + 1];
        if (end <= begin || end >= T) continue;                 // empty, or nothing follows
        const int64_t t0 = (end - 1) / BM * BM;                 // tile of the survivor's last row
        if (t0 < begin || t0 + BM <= end) continue;             // owned by an earlier survivor / ends with the tile
        const int rows = (int)min((int64_t)BM, T - t0);
        __syncthreads();                                        // src_row_of is free again
        for (int r = threadIdx.x; r < rows; r += PACK_THREADS) {
            const int64_t t = t0 + r;
            int sv = s0;
            while (sv + 1 < S && cu_seqlens[sv + 1] <= t) ++sv;
            src_row_of[r] = src_tok_off[survivor_idx[sv]] + (t - cu_seqlens[sv]);
        }
        __syncthreads();
        uint4* dst = scratch + (int64_t)s0 * BM * vec_per_row;
        const int total = rows * vec_per_row;
        for (int v0 = 0; v0 < total; v0 += 8 * PACK_THREADS) {
            uint4 buf[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int vv = v0 + u * PACK_THREADS + threadIdx.x;
                if (vv < total) {
                    const int r = vv / vec_per_row;
                    buf[u] = __ldg(src_rows + src_row_of[r] * vec_per_row + (vv - r * vec_per_row));
                }
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int vv = v0 + u * PACK_THREADS + threadIdx.x;
                if (vv < total) dst[vv] = buf[u];
            }
        }
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
// the tiles are re-fetched from HBM once per chunk, so the vocabulary is split until they fit.
int splits_for(const arrol_ctx* ctx, int64_t T_max, int d, int V, bool pair) {
    const int total_chunks = (V + BN - 1) / BN;
    const int64_t m_tiles = (T_max + BM - 1) / BM;
    // Measured with the blocks in step (TFLOP/s, packed rows / rows read in place by the gathered variant):
    //   d = 2048: 1 split (148 resident tiles, 74 MB) 1,380 / 1,200;  2 splits (74 tiles, 37 MB) 1,377 / 1,378
    //   d = 2560: 1 split (95 MB) 1,041 / 1,070;  2 splits (47 MB) 1,392 / 1,391;  4 splits (24 MB) 1,362 / 1,362
    //   d = 4096: 1 split (148 MB) 990 / 987;  2 splits (74 MB) 1,391 / 1,377;  4 splits (37 MB) 1,363 / 1,363
    // and as pairs of blocks (cta_group::2), same order:
    //   d = 2048: 1 split 1,389 / 1,271;  2 splits 1,411-1,427 / 1,403-1,410
    //   d = 2560: 2 splits 1,428 / 1,413;  4 splits 1,403 / 1,396
    //   d = 4096: 2 splits (74 MB) 1,235 / 1,232;  4 splits (37 MB) 1,392 / 1,371;  8 splits 1,357 / 1,352
    // Token tiles beyond what L2 keeps are re-fetched from HBM once per chunk; every split beyond that streams
    // W_vocab from HBM once more per wave.  So: two splits whenever there is a full wave of tiles (tiles read in place
    // are scattered over the source buffer and 148 of them do not stay resident even at 74 MB), more only while the
    // resident tiles exceed 80 MB (one block per tile) or 50 MB (pairs).  The packed and the in-place variant follow
    // the same rule, so their results are bit-identical.
    // Which form: pairs are 1.5-3 % faster at equal split counts; where they need more splits than single blocks
    // (d = 4096: four against two) the extra W_vocab streams and the busier tensor pipe draw more power, and in a
    // seconds-long run under the 1 kW cap the SM clock settles 4 % lower (1,195 against 1,250 MHz, read by the kernel)
    // and the step is 2 % SLOWER (1,369 against 1,392-1,396 TFLOP/s).  So pairs only where they need no more splits.
    if (ctx->logprob_splits > 0) return ctx->logprob_splits < total_chunks ? ctx->logprob_splits : total_chunks;
    int splits = m_tiles >= ctx->sm_count ? 2 : 1;
    const double l2_budget = (pair ? 50.0 : 80.0) * 1024 * 1024;
    const double tile_bytes = (double)BM * d * 2;
    while (splits < 8 && (ctx->sm_count / splits) * tile_bytes > l2_budget) splits *= 2;
    // few token tiles: split so that every SM has work
    while (splits < 16 && m_tiles * splits < ctx->sm_count && splits * 2 <= total_chunks) splits *= 2;
    if (splits > total_chunks) splits = total_chunks;
    return splits < 1 ? 1 : splits;
}

// The form of the kernel for these sizes: pairs of blocks unless switched off, forced, or costlier in splits.
bool pair_for(const arrol_ctx* ctx, int64_t T_max, int d, int V) {
    if (ctx->sm_count < 2 || ctx->logprob_pair == 0) return false;
    if (ctx->logprob_pair == 1) return true;
    return splits_for(ctx, T_max, d, V, true) <= splits_for(ctx, T_max, d, V, false);
}

int choose_splits(const arrol_ctx* ctx, int64_t T_max, int d, int V) {
    return splits_for(ctx, T_max, d, V, pair_for(ctx, T_max, d, V));
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

extern "C" int32_t arrol_token_logprob_form(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V) {
    if (!ctx || T_max <= 0 || d <= 0 || V <= 0) return 0;
    return pair_for(ctx, T_max, d, V) ? 2 : 1;
}

extern "C" int32_t arrol_token_logprob_splits(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V) {
    if (!ctx || T_max <= 0 || d <= 0 || V <= 0) return 0;
    const int total_chunks = (V + BN - 1) / BN;
    int splits = choose_splits(ctx, T_max, d, V);
    const int chunks_per_split = (total_chunks + splits - 1) / splits;
    return (total_chunks + chunks_per_split - 1) / chunks_per_split;
}

// Gather description of the gathered variant: the token rows come from `hidden` = the source buffer of
// `source_rows` rows through (cu_seqlens, survivor_idx, src_tok_off); NULL = `hidden` is the packed [T_max, d] block.
struct GatherArgs {
    const int64_t* cu_seqlens;
    const int32_t* survivor_idx;
    const int64_t* src_tok_off;
    const int64_t* d_num;
    int64_t source_rows;
    int32_t S_max;
};

// bytes of the boundary-tile scratch, placed after the split records in the gathered variant's workspace
static size_t boundary_scratch_bytes(int32_t S_max, int32_t d) { return (size_t)S_max * BM * (size_t)d * 2; }

static int run_token_logprob(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                             int64_t T_max, const int64_t* d_T, int32_t d, int32_t V, float inv_temperature,
                             float* logp, float* lse, float* conf, void* workspace, size_t workspace_bytes,
                             void* stream, const GatherArgs* ga = nullptr) {
    if (!ctx || T_max < 0 || d <= 0 || V <= 0 || !(inv_temperature > 0.f)) return ARROL_ERR_INVALID_ARG;
    if (T_max == 0) return ARROL_OK;
    if (!hidden || !W_vocab || !targets || !logp) return ARROL_ERR_INVALID_ARG;
    if (d % 8 != 0) return ARROL_ERR_UNSUPPORTED;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(W_vocab, 16)) return ARROL_ERR_INVALID_ARG;
    if (T_max > (int64_t)INT32_MAX - BM) return ARROL_ERR_UNSUPPORTED;   // TMA coordinates are 32-bit
    const size_t split_bytes = arrol_token_logprob_workspace(ctx, T_max, d, V);
    const size_t need = split_bytes + (ga ? boundary_scratch_bytes(ga->S_max, d) : 0);
    if (!workspace || workspace_bytes < need || !arrol_aligned(workspace, 256)) return ARROL_ERR_WORKSPACE;

    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;

    CUtensorMap map_h, map_s, map_w;
    void* scratch = static_cast<uint8_t*>(workspace) + split_bytes;      // split_bytes is a multiple of 16 (256-aligned + records)
    if (make_map(ctx, &map_h, hidden, (uint64_t)(ga ? ga->source_rows : T_max), (uint64_t)d, BM) != ARROL_OK)
        return ARROL_ERR_CUDA;
    if (ga) {
        if (make_map(ctx, &map_s, scratch, (uint64_t)ga->S_max * BM, (uint64_t)d, BM) != ARROL_OK) return ARROL_ERR_CUDA;
    } else {
        map_s = map_h;
    }
    // pair variant (clusters of two blocks): every block loads half of a chunk's W_vocab rows
    const bool pair = pair_for(ctx, T_max, d, V);
    if (make_map(ctx, &map_w, W_vocab, (uint64_t)V, (uint64_t)d, pair ? PAIR_B_ROWS : BN) != ARROL_OK) return ARROL_ERR_CUDA;

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
    p.cu_seqlens = ga ? ga->cu_seqlens : nullptr;
    p.survivor_idx = ga ? ga->survivor_idx : nullptr;
    p.src_tok_off = ga ? ga->src_tok_off : nullptr;
    p.d_num = ga ? ga->d_num : nullptr;
    p.S_max = ga ? ga->S_max : 0;
    p.wave_counter = ctx->d_tile_counters + ARROL_TILE_COUNTERS - 1;   // last word of the page: not a scoring counter
    p.timing = ctx->logprob_timing;
    p.timing_items = ctx->logprob_timing_items;

    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<false, false, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<true, false, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<false, true, false>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<false, false, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<false, true, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(token_logprob_kernel<true, false, true>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    const int64_t m_tiles = (T_max + BM - 1) / BM;
    typedef void (*KernelFn)(CUtensorMap, CUtensorMap, CUtensorMap, LogprobParams);
    const int variant = ga ? 2 : (conf ? 1 : 0);
    KernelFn fn;
    if (pair) fn = ga ? token_logprob_kernel<false, true, true> : (conf ? token_logprob_kernel<true, false, true>
                                                                         : token_logprob_kernel<false, false, true>);
    else fn = ga ? token_logprob_kernel<false, true, false> : (conf ? token_logprob_kernel<true, false, false>
                                                                     : token_logprob_kernel<false, false, false>);
    // work items and the units that take them: blocks, or pairs of blocks on 256 rows
    const int64_t items_max = (pair ? (m_tiles + 1) / 2 : m_tiles) * p.splits;
    int64_t units = pair ? ctx->sm_count / 2 : ctx->sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (pair) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 2;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
        // Pairs that wait for one another per wave must all be resident.  The cooperative attribute would have the
        // driver check that, but the profiler cannot launch a cooperative grid of clusters that fills the GPU
        // ("LaunchFailed"; the same grid without the attribute profiles), so the check is made here instead: never
        // more pairs than the occupancy query says fit at once (asked once per context and kernel variant).  The
        // waits themselves are bounded either way.
        if (ctx->pair_max_clusters[variant] == 0) {
            cfg.gridDim = dim3((unsigned)(2 * units));
            cfg.attrs = attr;
            cfg.numAttrs = n_attr;
            int fit = 0;
            ARROL_CUDA_OK(cudaOccupancyMaxActiveClusters(&fit, fn, &cfg));
            if (fit < 1) return ARROL_ERR_CUDA;
            ctx->pair_max_clusters[variant] = fit;
        }
        if (units > ctx->pair_max_clusters[variant]) units = ctx->pair_max_clusters[variant];
    }
    if (units > items_max) units = items_max;
    const int64_t grid = pair ? 2 * units : units;
    // more than one wave: the blocks wait for one another, so they must all be resident (single blocks: cooperative
    // launch)
    const bool several_waves = items_max > units;
    if (several_waves) ARROL_CUDA_OK(cudaMemsetAsync(p.wave_counter, 0, sizeof(unsigned int), s));
    if (several_waves && !pair) {
        attr[n_attr].id = cudaLaunchAttributeCooperative;
        attr[n_attr].val.cooperative = 1;
        ++n_attr;
    }
    cfg.gridDim = dim3((unsigned)grid);
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    if (ga) {
        int blocks = ga->S_max < ctx->sm_count * 4 ? ga->S_max : ctx->sm_count * 4;
        ARROL_CUDA_OK(arrol_launch_pdl(pack_boundary_tiles_kernel, dim3((unsigned)blocks), dim3(PACK_THREADS), 0, s,
                                       static_cast<const uint4*>(hidden), ga->cu_seqlens, ga->survivor_idx,
                                       ga->src_tok_off, ga->d_num, ga->S_max, T_max, d / 8, static_cast<uint4*>(scratch)));
        ctx->launches += 1;
    }
    ARROL_CUDA_OK(cudaLaunchKernelEx(&cfg, fn, map_h, map_s, map_w, p));
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

extern "C" size_t arrol_token_logprob_gathered_workspace(arrol_ctx* ctx, int32_t S_max, int64_t T_max, int32_t d,
                                                         int32_t V) {
    if (!ctx || S_max <= 0 || T_max <= 0 || d <= 0 || V <= 0) return 0;
    return arrol_token_logprob_workspace(ctx, T_max, d, V) + boundary_scratch_bytes(S_max, d);
}

extern "C" int arrol_token_logprob_gathered(arrol_ctx* ctx, const void* src_rows, int64_t source_rows,
                                            const void* W_vocab, const int32_t* targets, const int64_t* cu_seqlens,
                                            const int32_t* survivor_idx, const int64_t* src_tok_off,
                                            const int64_t* d_num, int32_t S_max, int64_t T_max, int32_t d, int32_t V,
                                            float inv_temperature, float* logp, float* lse, void* workspace,
                                            size_t workspace_bytes, void* stream) {
    if (!ctx || S_max < 0 || source_rows < 0 || T_max < 0) return ARROL_ERR_INVALID_ARG;
    if (T_max == 0 || S_max == 0) return ARROL_OK;
    if (!cu_seqlens || !survivor_idx || !src_tok_off || !d_num || source_rows == 0) return ARROL_ERR_INVALID_ARG;
    if (source_rows > (int64_t)INT32_MAX - BM || (int64_t)S_max * BM > (int64_t)INT32_MAX - BM)
        return ARROL_ERR_UNSUPPORTED;                                            // TMA coordinates are 32-bit
    GatherArgs ga = {cu_seqlens, survivor_idx, src_tok_off, d_num, source_rows, S_max};
    return run_token_logprob(ctx, src_rows, W_vocab, targets, T_max, d_num + 1, d, V, inv_temperature, logp, lse,
                             nullptr, workspace, workspace_bytes, stream, &ga);
}
