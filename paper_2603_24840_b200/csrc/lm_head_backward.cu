// arrol_lm_head_backward: gradient of the selected-token log-probs through the lm_head (Section 3: the policy
// update differentiates log pi_theta(o_t | o_<t); Algorithm 1 "Backprop ... on policy").
//
//   z = inv_temp H W^T,  logp_t = z_{t,y_t} - lse_t,  given g_t = dL/dlogp_t and lse_t from the forward call:
//   dz_{t,v} = g_t inv_temp ([v = y_t] - exp(z_{t,v} - lse_t)),   dH = dz W,   dW = dz^T H.
//
// The tokens are processed in chunks of TC rows.  Per chunk, three tensor-core kernels with the same
// TMA -> shared memory -> tcgen05.mma -> tensor memory pipeline as the forward kernel:
//   dz_kernel     recomputes the chunk's logits tile by tile and turns each accumulator tile into dz (bf16),
//                 written once as dZ [TC, V]
//   gemm_kernel   dH[chunk] = dZ . W       A = dZ K-major (K = V contiguous), B = W MN-major (N = d contiguous)
//   gemm_kernel   dW       += dZ^T . H     A = dZ MN-major (M = V contiguous), B = H chunk MN-major
// The MN-major operands are read by the tensor core straight from their row-major storage (transpose bits in the
// instruction descriptor, MN-major shared-memory descriptors), so nothing is transposed in memory and the T x V
// matrix exists only one chunk at a time, once, in the workspace.
#include "arrol_internal.h"
#include "tc_common.cuh"

namespace {

constexpr int BM = 128, BN = 256;
constexpr int STAGES = 4;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int B_STAGE_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int MN_BLOCK_BYTES = BK * 128;   // one 64-element MN block of an MN-major stage: BK rows of 128 bytes
constexpr int TMEM_COLS = 512;
constexpr int EPI_WARPS = 8;            // two warps per tensor-memory lane quarter, each takes half of the columns
constexpr int NUM_THREADS = 64 + 32 * EPI_WARPS;
constexpr int EPI_PIECES = BN / 32 / (EPI_WARPS / 4);   // 32-column pieces per epilogue warp and accumulator
// every kernel: one 32-row x 128-byte staging tile per epilogue warp behind the barrier block (1 KB), 1024-byte
// aligned, from which the results leave as TMA tile stores / reductions
constexpr int EPI_STAGE_TILE = 32 * 128;
constexpr size_t EPI_STAGE_OFFSET = (size_t)STAGES * STAGE_BYTES + 1024;
constexpr size_t SMEM_BYTES = EPI_STAGE_OFFSET + (size_t)EPI_WARPS * EPI_STAGE_TILE + 1024;
constexpr int TC = 74 * BM;      // tokens per chunk: 74 token tiles, so that TC/128 x d/256 tiles fill 148 SMs evenly

struct PipeSmem {
    uint8_t* stage_a;
    uint8_t* stage_b;
    uint64_t *full, *empty, *acc_full, *acc_empty, *drain;
    uint32_t* tmem_slot;
    volatile uint32_t* abort_flag;
};

__device__ __forceinline__ PipeSmem carve_smem(uint8_t* smem_raw) {
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    PipeSmem ps;
    ps.stage_a = smem;
    ps.stage_b = smem + (size_t)STAGES * A_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)STAGES * STAGE_BYTES);
    ps.full = bars;
    ps.empty = bars + STAGES;
    ps.acc_full = bars + 2 * STAGES;
    ps.acc_empty = ps.acc_full + 2;
    ps.drain = ps.acc_empty + 2;
    ps.tmem_slot = reinterpret_cast<uint32_t*>(ps.drain + 1);
    ps.abort_flag = ps.tmem_slot + 1;
    return ps;
}

// Common prologue: barriers, tensor-memory allocation.  Returns the tensor-memory base address.
__device__ __forceinline__ uint32_t pipe_setup(const PipeSmem& ps, const CUtensorMap* ma, const CUtensorMap* mb) {
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&ps.full[s], 1); mbar_init(&ps.empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&ps.acc_full[b], 1); mbar_init(&ps.acc_empty[b], EPI_WARPS); }
        mbar_init(ps.drain, 1);
        *ps.abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(ma) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(mb) : "memory");
    }
    if (warp == 1) {
        tcgen05_alloc(ps.tmem_slot, TMEM_COLS);
        tcgen05_relinquish();
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    return *ps.tmem_slot;
}

__device__ __forceinline__ void pipe_teardown(const PipeSmem& ps, uint32_t tmem_base, uint32_t* d_status) {
    tcgen05_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *ps.abort_flag) atomicOr(d_status, ARROL_DEV_WAIT_EXPIRED);
    if ((threadIdx.x >> 5) == 1) {
        tcgen05_fence_after();
        tcgen05_dealloc(tmem_base, TMEM_COLS);
    }
}

// Producer role (one thread).  For every accumulator tile `coords(it, a_mn0, b_mn0)` gives the operands' MN
// origins (it returns false when the tile list is exhausted); for every K step the stage receives
//   K-major operand:  one box  [MN rows x 64 K columns]           at (x = k, y = mn0)
//   MN-major operand: MN/64 blocks [64 K rows x 64 MN columns], BK*128 bytes apart: one three-dimensional box
//                     (64 elements, 64 K rows, MN/64 blocks) at (0, k, mn0/64) when the map is of that kind
//                     (a3d / b3d), else one two-dimensional box per block at (x = mn0 + 64 b, y = k).
// Issuing a copy costs the thread about 60 cycles, and a stage's MMAs last 512: with one copy per operand the
// producer keeps ahead of the tensor pipe, with six it does not.
template <bool A_MN, bool B_MN, typename Coords>
__device__ __forceinline__ void producer_loop(const PipeSmem& ps, const CUtensorMap* ma, const CUtensorMap* mb,
                                              int k_steps, Coords coords, bool a3d = false, bool b3d = false,
                                              const CUtensorMap* mb_tail = nullptr, int tail_ks = -1) {
    uint32_t stage = 0, phase = 0, issued = 0;
    bool ok = true;
    int ay, by;
    for (int64_t it = 0; ok && coords(it, ay, by); ++it) {
        for (int ks = 0; ks < k_steps; ++ks) {
            if (!mbar_wait(&ps.empty[stage], phase ^ 1u, ps.abort_flag)) { ok = false; break; }
            mbar_expect_tx(&ps.full[stage], STAGE_BYTES);
            uint8_t* sa = ps.stage_a + (size_t)stage * A_STAGE_BYTES;
            uint8_t* sb = ps.stage_b + (size_t)stage * B_STAGE_BYTES;
            if constexpr (A_MN) {
                if (a3d) {
                    tma_load_3d(sa, ma, 0, ks * BK, ay >> 6, &ps.full[stage]);
                } else {
#pragma unroll
                    for (int b = 0; b < BM / 64; ++b)
                        tma_load_2d(sa + b * MN_BLOCK_BYTES, ma, ay + 64 * b, ks * BK, &ps.full[stage]);
                }
            } else {
                tma_load_2d(sa, ma, ks * BK, ay, &ps.full[stage]);
            }
            if constexpr (B_MN) {
                // the K step that holds the last, partly live block of rows is read from its zero-padded copy
                const bool tail = ks == tail_ks;
                const CUtensorMap* m = tail ? mb_tail : mb;
                const int ky = tail ? 0 : ks * BK;
                if (b3d) {
                    tma_load_3d(sb, m, 0, ky, by >> 6, &ps.full[stage]);
                } else {
#pragma unroll
                    for (int b = 0; b < BN / 64; ++b)
                        tma_load_2d(sb + b * MN_BLOCK_BYTES, m, by + 64 * b, ky, &ps.full[stage]);
                }
            } else {
                tma_load_2d(sb, mb, ks * BK, by, &ps.full[stage]);
            }
            ++issued;
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
    }
    if (!ok) {   // gave up: let the copies already issued land before shared memory goes away (bounded)
        const uint32_t pending = issued < (uint32_t)STAGES ? issued : (uint32_t)STAGES;
        uint32_t s = stage, ph = phase;
        for (uint32_t i = 0; i < pending; ++i) {
            if (s == 0) { s = STAGES - 1; ph ^= 1u; } else { --s; }
            for (uint32_t spin = 0; spin < SPIN_LIMIT; ++spin)
                if (mbar_try_wait(&ps.full[s], ph)) break;
        }
    }
}

// MMA role (one thread): n_items accumulator tiles of k_steps K steps each, alternating the two accumulators.
// Inside a stage the four K = 16 slices are 32 bytes apart for a K-major operand (columns of the swizzled row) and
// 16 rows = 2048 bytes apart for an MN-major one.
template <bool A_MN, bool B_MN>
__device__ __forceinline__ void mma_loop(const PipeSmem& ps, uint32_t tmem_base, int64_t n_items, int k_steps) {
    constexpr uint32_t idesc = make_idesc(BM, BN, A_MN, B_MN);
    constexpr uint64_t a_step = A_MN ? (UMMA_K * 128) >> 4 : (UMMA_K * 2) >> 4;
    constexpr uint64_t b_step = B_MN ? (UMMA_K * 128) >> 4 : (UMMA_K * 2) >> 4;
    uint32_t stage = 0, phase = 0, acc = 0, acc_phase = 0;
    bool ok = true;
    for (int64_t it = 0; it < n_items && ok; ++it) {
        if (!mbar_wait(&ps.acc_empty[acc], acc_phase ^ 1u, ps.abort_flag)) { ok = false; break; }
        tcgen05_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BN;
        for (int ks = 0; ks < k_steps; ++ks) {
            if (!mbar_wait(&ps.full[stage], phase, ps.abort_flag)) { ok = false; break; }
            tcgen05_fence_after();
            const uint32_t sa = smem_u32(ps.stage_a + (size_t)stage * A_STAGE_BYTES);
            const uint32_t sb = smem_u32(ps.stage_b + (size_t)stage * B_STAGE_BYTES);
            const uint64_t a_desc = A_MN ? make_smem_desc_mn(sa, BK) : make_smem_desc(sa);
            const uint64_t b_desc = B_MN ? make_smem_desc_mn(sb, BK) : make_smem_desc(sb);
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k)
                tcgen05_mma_bf16(d_tmem, a_desc + a_step * k, b_desc + b_step * k, idesc, (ks | k) != 0 ? 1u : 0u);
            tcgen05_commit(&ps.empty[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (ok) tcgen05_commit(&ps.acc_full[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (!ok) {
        tcgen05_commit(ps.drain);
        for (uint32_t spin = 0; spin < SPIN_LIMIT; ++spin)
            if (mbar_try_wait(ps.drain, 0u)) break;
    }
}

__device__ __forceinline__ int64_t live_tokens(const int64_t* d_T, int64_t T_max) {
    int64_t T = T_max;
    if (d_T) { const int64_t t = *d_T; T = t < 0 ? 0 : (t < T ? t : T); }
    return T;
}

// ---- dz: recompute logits, write the softmax gradient of one token chunk --------------------------------------
struct DzParams {
    const int32_t* targets;
    const float* grad_logp;
    const float* lse;
    const int64_t* d_T;
    int64_t T_max, t0;        // chunk = tokens [t0, t0 + TC)
    int d, V;
    int64_t ldz;              // row pitch of dZ (V rounded up to 8)
    int splits, chunks_per_split;
    float scale2, inv_temp;
    __nv_bfloat16* dZ;        // [TC, ldz]
    uint32_t* d_status;
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
dz_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
          const __grid_constant__ CUtensorMap map_dz, const DzParams p) {
    extern __shared__ uint8_t smem_raw[];
    const PipeSmem ps = carve_smem(smem_raw);
    uint8_t* dz_stage = ps.stage_a + EPI_STAGE_OFFSET;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t T = live_tokens(p.d_T, p.T_max);
    if (p.t0 >= T) return;                                  // chunk past the live tokens (uniform for the grid)
    const int64_t items = (int64_t)(TC / BM) * p.splits;
    const int k_steps = (p.d + BK - 1) / BK;
    const int total_chunks = (p.V + BN - 1) / BN;
    const uint32_t tmem_base = pipe_setup(ps, &map_h, &map_w);

    // work item -> (token tile, vocabulary range); the accumulator tiles of one item are its vocabulary chunks
    auto item_range = [&](int64_t item, int& m_tile, int& c0, int& c1) {
        m_tile = (int)(item / p.splits);
        const int split = (int)(item % p.splits);
        c0 = split * p.chunks_per_split;
        c1 = min(c0 + p.chunks_per_split, total_chunks);
    };

    if (warp == 0) {
        if (lane == 0) {
            int64_t item = blockIdx.x;
            int m_tile = 0, c = 0, c1 = 0;
            bool have = false;
            producer_loop<false, false>(ps, &map_h, &map_w, k_steps, [&](int64_t, int& ay, int& by) {
                while (!have || c >= c1) {
                    if (have) item += gridDim.x;
                    if (item >= items) return false;
                    item_range(item, m_tile, c, c1);
                    have = true;
                }
                ay = (int)(p.t0 + (int64_t)m_tile * BM);
                by = c * BN;
                ++c;
                return true;
            });
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int64_t n_tiles = 0;
            for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
                int m_tile, c0, c1;
                item_range(item, m_tile, c0, c1);
                n_tiles += max(c1 - c0, 0);
            }
            mma_loop<false, false>(ps, tmem_base, n_tiles, k_steps);
        }
    } else {
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;           // 0 or 1: which half of the accumulator's columns
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int64_t item = blockIdx.x; item < items && ok; item += gridDim.x) {
            int m_tile, c0, c1;
            item_range(item, m_tile, c0, c1);
            const int row_in_chunk = m_tile * BM + row_in_tile;
            const int64_t t = p.t0 + row_in_chunk;
            int y = -1;
            float coef = 0.f, lse2 = 0.f;
            if (t < T) {
                y = p.targets[t];
                if (y >= 0 && y < p.V) {
                    coef = p.grad_logp[t] * p.inv_temp;
                    lse2 = p.lse[t] * 1.44269504088896340736f;
                } else {
                    y = -1;
                }
            }
            // dz leaves through shared memory: the warp's 32 rows x 64 columns (two pieces, 128 bytes per row, 128-byte
            // swizzle) are staged and written by one TMA tile store, i.e. in whole 128-byte lines; columns past V are
            // clipped by the copy.  (16-byte stores straight from the registers touch 32 lines per instruction and
            // cost the kernel 14 %.)
            uint8_t* stg = dz_stage + (size_t)(warp - 2) * EPI_STAGE_TILE;
            const int row0 = m_tile * BM + quarter * 32;
            for (int c = c0; c < c1 && ok; ++c) {
                ok = mbar_wait(&ps.acc_full[acc], acc_phase, ps.abort_flag);
                ok = __all_sync(0xffffffffu, ok) != 0;
                if (!ok) break;
                tcgen05_fence_after();
                // Two register buffers: the tensor-memory load of piece i + 1 is in flight while piece i is turned
                // into dz and staged.
                const uint32_t tacc = tmem_base + lane_addr + acc * BN;
                auto to_dz = [&](const uint32_t (&raw)[32], int piece, uint32_t (&packed)[16]) {
                    const int pc0 = c * BN + piece * 32;
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        // dz = coef ([v = y] - 2^(z log2e - lse log2e)); coef = 0 for rows that carry no gradient
                        float d0 = -coef * ex2_approx(fmaf(__uint_as_float(raw[j]), p.scale2, -lse2));
                        float d1 = -coef * ex2_approx(fmaf(__uint_as_float(raw[j + 1]), p.scale2, -lse2));
                        if (pc0 + j == y) d0 += coef;
                        if (pc0 + j + 1 == y) d1 += coef;
                        if (coef == 0.f) { d0 = 0.f; d1 = 0.f; }      // also guards 0 * inf from stale lse values
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(d0, d1);
                        packed[j >> 1] = *reinterpret_cast<const uint32_t*>(&h2);
                    }
                };
                auto stage_piece = [&](const uint32_t (&packed)[16], int piece) {
                    const int chunk0 = (piece & 1) * 4;               // 16-byte chunks of the 128-byte staging row
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4)
                        *reinterpret_cast<uint4*>(stg + lane * 128 + (((chunk0 + q4) ^ (lane & 7)) << 4)) =
                            make_uint4(packed[4 * q4], packed[4 * q4 + 1], packed[4 * q4 + 2], packed[4 * q4 + 3]);
                };
                uint32_t ra[32], rb[32];
                const int p0 = col_half * EPI_PIECES, p1 = p0 + EPI_PIECES;   // this warp's pieces of the accumulator
                tcgen05_ld_32x32_issue(tacc + p0 * 32, ra);
#pragma unroll 1
                for (int piece = p0; piece < p1; piece += 2) {
                    tcgen05_ld_wait(ra);
                    tcgen05_ld_32x32_issue(tacc + (piece + 1) * 32, rb);
                    uint32_t pa[16], pb[16];
                    to_dz(ra, piece, pa);
                    tcgen05_ld_wait(rb);
                    if (piece + 2 < p1) tcgen05_ld_32x32_issue(tacc + (piece + 2) * 32, ra);
                    to_dz(rb, piece + 1, pb);
                    if (lane == 0) bulk_wait_read_all();          // the previous tile store has read the staging tile
                    __syncwarp();
                    stage_piece(pa, piece);
                    stage_piece(pb, piece + 1);
                    fence_proxy_async_smem();
                    __syncwarp();
                    const int col0 = c * BN + piece * 32;
                    if (lane == 0 && col0 < p.V) {
                        tma_store_2d(&map_dz, col0, row0, stg);
                        bulk_commit_group();
                    }
                }
                tcgen05_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ps.acc_empty[acc]);
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
        if (lane == 0) bulk_wait_all();       // the tile stores have completed before the block's shared memory goes
    }
    pipe_teardown(ps, tmem_base, p.d_status);
}

// ---- C[M,N] (+)= op(A) op(B): bf16 operands in either orientation, fp32 result ------------------------------------
//   A_MN = false: A stored [M, K] row-major;  A_MN = true: A stored [K, M] row-major (used as its transpose)
//   B_MN = false: B stored [N, K] row-major;  B_MN = true: B stored [K, N] row-major
struct GemmParams {
    int M, N, K;
    float* C;
    int64_t ldc;
    int accumulate;           // 1: C += ..., 0: C = ...
    int k_is_tokens;          // 1: K counts the chunk's tokens: only the live ones (T - t0) are contracted
    int a3d, b3d;             // the MN-major operand's maps are three-dimensional (one copy per stage)
    const int64_t* d_T;       // the launch is skipped when t0 >= live tokens
    int64_t T_max, t0;
    uint32_t* d_status;
};

template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_b_tail, const __grid_constant__ CUtensorMap map_c,
            const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const PipeSmem ps = carve_smem(smem_raw);
    uint8_t* c_stage = ps.stage_a + EPI_STAGE_OFFSET;      // one 32 x 32 fp32 staging tile per epilogue warp
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t T_live = live_tokens(p.d_T, p.T_max);
    if (p.t0 >= T_live) return;
    const int m_tiles = (p.M + BM - 1) / BM, n_tiles = (p.N + BN - 1) / BN;
    const int64_t items = (int64_t)m_tiles * n_tiles;
    const int K = p.k_is_tokens ? (int)min((int64_t)p.K, T_live - p.t0) : p.K;
    const int k_steps = (K + BK - 1) / BK;
    const uint32_t tmem_base = pipe_setup(ps, &map_a, &map_b);

    if (warp == 0) {
        if (lane == 0) {
            const int tail_ks = (p.k_is_tokens && (K % BK) != 0) ? k_steps - 1 : -1;
            producer_loop<A_MN, B_MN>(ps, &map_a, &map_b, k_steps, [&](int64_t it, int& ay, int& by) {
                const int64_t item = blockIdx.x + it * gridDim.x;
                if (item >= items) return false;
                ay = (int)(item / n_tiles) * BM;       // consecutive blocks share the A panel, walk the B panels
                by = (int)(item % n_tiles) * BN;
                return true;
            }, p.a3d != 0, p.b3d != 0, &map_b_tail, tail_ks);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const int64_t mine = items > blockIdx.x ? (items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
            mma_loop<A_MN, B_MN>(ps, tmem_base, mine, k_steps);
        }
    } else {
        const int quarter = warp & 3;
        const int col_half = (warp - 2) >> 2;           // 0 or 1: which half of the accumulator's columns
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        uint32_t acc = 0, acc_phase = 0;
        bool ok = true;
        for (int64_t item = blockIdx.x; item < items && ok; item += gridDim.x) {
            const int col0 = (int)(item % n_tiles) * BN;
            ok = mbar_wait(&ps.acc_full[acc], acc_phase, ps.abort_flag);
            ok = __all_sync(0xffffffffu, ok) != 0;
            if (!ok) break;
            tcgen05_fence_after();
            // The warp's 32 rows x 32 columns leave through shared memory (128-byte swizzle) as one TMA tile store, or
            // as one TMA reduction (global += tile) when the result is accumulated: whole 128-byte lines, no read of C by
            // the SM, and rows / columns past M / N are clipped by the copy.
            uint8_t* stg = c_stage + (size_t)(warp - 2) * EPI_STAGE_TILE;
            const int row0 = (int)(item / n_tiles) * BM + quarter * 32;
#pragma unroll 1
            for (int piece = col_half * EPI_PIECES; piece < (col_half + 1) * EPI_PIECES; ++piece) {
                const int pc0 = col0 + piece * 32;
                if (pc0 >= p.N) break;
                float v[32];
                tcgen05_ld_32x32(tmem_base + lane_addr + acc * BN + piece * 32, v);
                if (lane == 0) bulk_wait_read_all();          // the previous tile copy has read the staging tile
                __syncwarp();
#pragma unroll
                for (int q4 = 0; q4 < 8; ++q4)
                    *reinterpret_cast<float4*>(stg + lane * 128 + ((q4 ^ (lane & 7)) << 4)) =
                        make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0 && row0 < p.M) {
                    if (p.accumulate) tma_reduce_add_2d(&map_c, pc0, row0, stg);
                    else tma_store_2d(&map_c, pc0, row0, stg);
                    bulk_commit_group();
                }
            }
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&ps.acc_empty[acc]);
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_all();       // the tile copies have completed before the block's shared memory goes
    }
    pipe_teardown(ps, tmem_base, p.d_status);
}

// Copies the last, partly live 64-row block of the chunk's hidden rows into `tail` [64, d] and pads it with zeros,
// so that rows past the live tokens (caller memory that may hold anything) never reach the tensor core.
__global__ void tail_block_kernel(const uint16_t* __restrict__ hidden, int d, const int64_t* d_T, int64_t T_max,
                                  int64_t t0, uint16_t* __restrict__ tail) {
    const int64_t T = live_tokens(d_T, T_max);
    if (t0 >= T) return;
    const int64_t live = min((int64_t)TC, T - t0);
    const int64_t r0 = live / BK * BK;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < (int64_t)BK * d; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / d, c = i - r * d;
        tail[i] = (r0 + r < live) ? hidden[(t0 + r0 + r) * d + c] : (uint16_t)0;
    }
}

struct BackwardLayout {
    int64_t ldz;       // V rounded up to 8
    size_t dz, tail, total;
};

BackwardLayout backward_layout(int d, int V) {
    BackwardLayout L;
    L.ldz = ((int64_t)V + 7) & ~(int64_t)7;
    L.dz = 0;
    L.tail = (((size_t)TC * L.ldz * 2) + 255) & ~(size_t)255;
    L.total = L.tail + (((size_t)BK * d * 2 + 255) & ~(size_t)255);
    return L;
}

}  // namespace

int arrol_internal_gemm_tn(arrol_ctx* ctx, const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K,
                           float* C, int64_t ldc, int accumulate, cudaStream_t s) {
    if (M <= 0 || N <= 0 || K <= 0 || lda % 8 != 0 || ldb % 8 != 0) return ARROL_ERR_UNSUPPORTED;
    ARROL_CUDA_OK(cudaFuncSetAttribute(gemm_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    CUtensorMap map_a, map_b, map_c;
    if (make_map_f32_tile(ctx, &map_c, C, (uint64_t)M, (uint64_t)N, (uint64_t)ldc) != ARROL_OK) return ARROL_ERR_CUDA;
    bool a3 = M % 64 == 0, b3 = N % 64 == 0;
    if (a3 && make_map_mn3d(ctx, &map_a, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BM / 64) != ARROL_OK) a3 = false;
    if (b3 && make_map_mn3d(ctx, &map_b, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, BN / 64) != ARROL_OK) b3 = false;
    if (!a3 && make_map_ld(ctx, &map_a, A, (uint64_t)K, (uint64_t)M, (uint64_t)lda, BK) != ARROL_OK) return ARROL_ERR_CUDA;
    if (!b3 && make_map_ld(ctx, &map_b, B, (uint64_t)K, (uint64_t)N, (uint64_t)ldb, BK) != ARROL_OK) return ARROL_ERR_CUDA;
    GemmParams g;
    g.M = M; g.N = N; g.K = K; g.C = C; g.ldc = ldc; g.accumulate = accumulate; g.k_is_tokens = 0;
    g.a3d = a3; g.b3d = b3; g.d_T = nullptr; g.T_max = 1; g.t0 = 0; g.d_status = ctx->d_status;
    const int64_t items = (int64_t)((M + BM - 1) / BM) * ((N + BN - 1) / BN);
    gemm_kernel<true, true><<<(unsigned)(items < ctx->sm_count ? items : ctx->sm_count), NUM_THREADS, SMEM_BYTES, s>>>(
        map_a, map_b, map_b, map_c, g);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

extern "C" size_t arrol_lm_head_backward_workspace(arrol_ctx* ctx, int64_t T_max, int32_t d, int32_t V) {
    if (!ctx || T_max <= 0 || d <= 0 || V <= 0) return 0;
    return backward_layout(d, V).total;
}

extern "C" int arrol_lm_head_backward(arrol_ctx* ctx, const void* hidden, const void* W_vocab, const int32_t* targets,
                                      const float* grad_logp, const float* lse, int64_t T_max, const int64_t* d_T,
                                      int32_t d, int32_t V, float inv_temperature, float* dH, float* dW,
                                      void* workspace, size_t workspace_bytes, void* stream) {
    if (!ctx || T_max < 0 || d <= 0 || V <= 0 || !(inv_temperature > 0.f)) return ARROL_ERR_INVALID_ARG;
    if (!dW) return ARROL_ERR_INVALID_ARG;
    if (d % 8 != 0) return ARROL_ERR_UNSUPPORTED;
    if (T_max > (int64_t)INT32_MAX - TC) return ARROL_ERR_UNSUPPORTED;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    ARROL_CUDA_OK(cudaMemsetAsync(dW, 0, sizeof(float) * (size_t)V * d, s));
    if (T_max == 0) return ARROL_OK;
    if (!hidden || !W_vocab || !targets || !grad_logp || !lse || !dH) return ARROL_ERR_INVALID_ARG;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(W_vocab, 16) || !arrol_aligned(dH, 16) || !arrol_aligned(dW, 16))
        return ARROL_ERR_INVALID_ARG;
    const BackwardLayout L = backward_layout(d, V);
    if (!workspace || workspace_bytes < L.total || !arrol_aligned(workspace, 256)) return ARROL_ERR_WORKSPACE;
    __nv_bfloat16* dZ = reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(workspace) + L.dz);
    uint16_t* Htail = reinterpret_cast<uint16_t*>(static_cast<uint8_t*>(workspace) + L.tail);

    ARROL_CUDA_OK(cudaFuncSetAttribute(dz_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(gemm_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    ARROL_CUDA_OK(cudaFuncSetAttribute(gemm_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));

    // tensor maps: K-major operands are fetched as [MN rows x 64 K columns] boxes; MN-major ones (the same row-major
    // storage read the other way) as one three-dimensional box per stage when the MN extent is a whole number of
    // 64-element blocks, else as one [64 K rows x 64 MN columns] box per block
    CUtensorMap map_h_k, map_w_k, map_dz_k, map_dz_st, map_w_mn, map_dz_mn, map_h_mn, map_h_tail;
    if (make_map(ctx, &map_h_k, hidden, (uint64_t)T_max, (uint64_t)d, BM) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map(ctx, &map_w_k, W_vocab, (uint64_t)V, (uint64_t)d, BN) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map_ld(ctx, &map_dz_k, dZ, TC, (uint64_t)V, (uint64_t)L.ldz, BM) != ARROL_OK) return ARROL_ERR_CUDA;
    if (make_map_ld(ctx, &map_dz_st, dZ, TC, (uint64_t)V, (uint64_t)L.ldz, 32) != ARROL_OK) return ARROL_ERR_CUDA;   // store tiles
    CUtensorMap map_dw;
    if (make_map_f32_tile(ctx, &map_dw, dW, (uint64_t)V, (uint64_t)d, (uint64_t)d) != ARROL_OK) return ARROL_ERR_CUDA;
    bool d3 = d % 64 == 0, v3 = V % 64 == 0;
    if (d3 && (make_map_mn3d(ctx, &map_w_mn, W_vocab, (uint64_t)V, (uint64_t)d, (uint64_t)d, BN / 64) != ARROL_OK ||
               make_map_mn3d(ctx, &map_h_tail, Htail, (uint64_t)BK, (uint64_t)d, (uint64_t)d, BN / 64) != ARROL_OK))
        d3 = false;
    if (v3 && make_map_mn3d(ctx, &map_dz_mn, dZ, TC, (uint64_t)V, (uint64_t)L.ldz, BM / 64) != ARROL_OK) v3 = false;
    if (!d3) {
        if (make_map(ctx, &map_w_mn, W_vocab, (uint64_t)V, (uint64_t)d, BK) != ARROL_OK) return ARROL_ERR_CUDA;
        if (make_map(ctx, &map_h_tail, Htail, (uint64_t)BK, (uint64_t)d, BK) != ARROL_OK) return ARROL_ERR_CUDA;
    }
    if (!v3 && make_map_ld(ctx, &map_dz_mn, dZ, TC, (uint64_t)V, (uint64_t)L.ldz, BK) != ARROL_OK) return ARROL_ERR_CUDA;

    const int total_chunks = (V + BN - 1) / BN;
    int splits = 1;
    while ((TC / BM) * splits < ctx->sm_count && splits * 2 <= total_chunks) splits *= 2;
    const int chunks_per_split = (total_chunks + splits - 1) / splits;
    splits = (total_chunks + chunks_per_split - 1) / chunks_per_split;

    for (int64_t t0 = 0; t0 < T_max; t0 += TC) {
        const int64_t rows = (T_max - t0) < TC ? (T_max - t0) : (int64_t)TC;
        // the chunk of hidden as an MN-major B operand: [rows (K), d (N)]; rows past T_max read as zero
        const void* h_chunk = static_cast<const uint8_t*>(hidden) + (size_t)t0 * d * 2;
        if ((d3 ? make_map_mn3d(ctx, &map_h_mn, h_chunk, (uint64_t)rows, (uint64_t)d, (uint64_t)d, BN / 64)
                : make_map(ctx, &map_h_mn, h_chunk, (uint64_t)rows, (uint64_t)d, BK)) != ARROL_OK)
            return ARROL_ERR_CUDA;

        DzParams zp;
        zp.targets = targets; zp.grad_logp = grad_logp; zp.lse = lse; zp.d_T = d_T; zp.T_max = T_max; zp.t0 = t0;
        zp.d = d; zp.V = V; zp.ldz = L.ldz; zp.splits = splits; zp.chunks_per_split = chunks_per_split;
        zp.scale2 = inv_temperature * 1.44269504088896340736f; zp.inv_temp = inv_temperature;
        zp.dZ = dZ; zp.d_status = ctx->d_status;
        int64_t grid = (int64_t)(TC / BM) * splits;
        if (grid > ctx->sm_count) grid = ctx->sm_count;
        dz_kernel<<<(unsigned)grid, NUM_THREADS, SMEM_BYTES, s>>>(map_h_k, map_w_k, map_dz_st, zp);

        GemmParams gh;    // dH[chunk] = dZ . W
        gh.M = (int)rows; gh.N = d; gh.K = V; gh.C = dH + t0 * d; gh.ldc = d; gh.accumulate = 0; gh.k_is_tokens = 0; gh.a3d = 0; gh.b3d = d3;
        gh.d_T = d_T; gh.T_max = T_max; gh.t0 = t0; gh.d_status = ctx->d_status;
        const int64_t gh_items = (int64_t)((rows + BM - 1) / BM) * ((d + BN - 1) / BN);
        CUtensorMap map_dh;      // this chunk's rows of dH: rows past the chunk are clipped by the tile stores
        if (make_map_f32_tile(ctx, &map_dh, dH + t0 * d, (uint64_t)rows, (uint64_t)d, (uint64_t)d) != ARROL_OK)
            return ARROL_ERR_CUDA;
        gemm_kernel<false, true><<<(unsigned)(gh_items < ctx->sm_count ? gh_items : ctx->sm_count), NUM_THREADS,
                                   SMEM_BYTES, s>>>(map_dz_k, map_w_mn, map_w_mn, map_dh, gh);
        tail_block_kernel<<<64, 256, 0, s>>>(static_cast<const uint16_t*>(hidden), d, d_T, T_max, t0, Htail);
        GemmParams gw;    // dW += dZ^T . H[chunk]
        gw.M = V; gw.N = d; gw.K = (int)rows; gw.C = dW; gw.ldc = d; gw.accumulate = 1; gw.k_is_tokens = 1; gw.a3d = v3; gw.b3d = d3;
        gw.d_T = d_T; gw.T_max = T_max; gw.t0 = t0; gw.d_status = ctx->d_status;
        const int64_t gw_items = (int64_t)((V + BM - 1) / BM) * ((d + BN - 1) / BN);
        gemm_kernel<true, true><<<(unsigned)(gw_items < ctx->sm_count ? gw_items : ctx->sm_count), NUM_THREADS,
                                  SMEM_BYTES, s>>>(map_dz_mn, map_h_mn, map_h_tail, map_dw, gw);
        ctx->launches += 4;
        ARROL_CUDA_OK(cudaGetLastError());
    }
    return ARROL_OK;
}
