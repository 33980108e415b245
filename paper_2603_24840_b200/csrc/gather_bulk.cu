// Hidden-row plane of arrol_compact (Section 4.3 (ii): filter the pruned rollouts and re-batch the survivors) moved
// by the copy engine: global -> shared -> global bulk copies (cp.async.bulk), so the payload never passes through
// registers and one thread per role keeps a queue of 32 KB transfers in flight.
//
// Three blocks per SM, each with a ring of two stages (192 KB in flight per SM), own contiguous runs of destination
// tiles (as many whole rows as fit 32 KB).  Measured: one block per SM with six stages 5,274 / 5,703 GB/s on the
// Llama- / Qwen-3-4B-shaped steps, two blocks with three stages 5,288 / 5,708, three blocks with two stages
// 5,540-5,562 / 6,036-6,082 (the same bytes in flight, more threads issuing copies), four blocks of two 24 KB stages
// 5,473 / 6,114.  A ring needs at least two stages: a stage is freed when the NEXT store has been issued.
//   thread 0 (producer)  for each tile: finds the survivors its rows belong to (binary search once, then a forward
//                        walk in cu_seqlens) and issues one bulk load per contiguous source segment into a ring of
//                        shared-memory stages; completion by transaction count on the stage's mbarrier
//   thread 32 (storer)   waits for a stage, issues one bulk store of the tile to its (contiguous) destination, and
//                        frees a stage once the store that used it has finished reading shared memory
// Every wait is bounded; on expiry the block records ARROL_DEV_WAIT_EXPIRED, lets its copies land and returns.
#include "arrol_internal.h"
#include "tc_common.cuh"

namespace {

constexpr int GB_STAGES = 2;
constexpr int GB_BLOCKS_PER_SM = 3;
static_assert(GB_STAGES >= 2, "the storer frees a stage only after it has issued the following store");
constexpr int GB_TILE_BYTES = 32 * 1024;
constexpr int GB_THREADS = 64;
constexpr size_t GB_SMEM = (size_t)GB_STAGES * GB_TILE_BYTES + 1024 + 256;

__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                 ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes) : "memory");
}
// all but the most recent bulk store of this thread have finished reading shared memory
__device__ __forceinline__ void bulk_wait_read_but_one() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

// Largest s in [lo, hi) with cu_seqlens[s] <= t (skips zero-length survivors), given cu_seqlens[lo] <= t < cu_seqlens[hi].
__device__ __forceinline__ int find_survivor_of(const int64_t* __restrict__ cu_seqlens, int lo, int hi, int64_t t) {
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(cu_seqlens + mid) <= t) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(GB_THREADS, GB_BLOCKS_PER_SM)
gather_rows_bulk_kernel(const int64_t* __restrict__ d_num, const int64_t* __restrict__ cu_seqlens,
                        const int32_t* __restrict__ survivor_idx, const int64_t* __restrict__ src_tok_off,
                        const uint8_t* __restrict__ src_rows, int64_t row_bytes, int64_t capacity, int tile_rows,
                        uint8_t* __restrict__ dst_rows, uint32_t* d_status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)GB_STAGES * GB_TILE_BYTES);   // loads -> storer
    uint64_t* empty = full + GB_STAGES;                                                      // storer -> producer
    volatile uint32_t* abort_flag = reinterpret_cast<uint32_t*>(empty + GB_STAGES);

    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < GB_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        *abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    pdl_wait();
    d_num = pdl_acquire(d_num); cu_seqlens = pdl_acquire(cu_seqlens); survivor_idx = pdl_acquire(survivor_idx);
    src_tok_off = pdl_acquire(src_tok_off); src_rows = pdl_acquire(src_rows);
    __syncthreads();

    const int S = (int)d_num[0];
    const int64_t T = d_num[1];
    if (T > capacity || S <= 0 || T <= 0 || d_status[1]) return;   // overflow / bad index was recorded by the scan kernel
    const int64_t n_tiles = (T + tile_rows - 1) / tile_rows;
    const int64_t per_block = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * per_block;
    const int64_t tile_end = min(n_tiles, tile_begin + per_block);

    if (threadIdx.x == 0 && tile_begin < tile_end) {
        // ---------------- producer ----------------
        int s = find_survivor_of(cu_seqlens, 0, S, tile_begin * tile_rows);
        int64_t s_begin = __ldg(cu_seqlens + s), s_end = __ldg(cu_seqlens + s + 1);
        int64_t s_src = __ldg(src_tok_off + __ldg(survivor_idx + s));
        uint32_t stage = 0, phase = 0, issued = 0;
        bool ok = true;
        for (int64_t tile = tile_begin; tile < tile_end && ok; ++tile) {
            const int64_t t0 = tile * tile_rows;
            const int rows_here = (int)min((int64_t)tile_rows, T - t0);
            if (!mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
            mbar_expect_tx(&full[stage], (uint32_t)(rows_here * row_bytes));
            uint8_t* dst = smem + (size_t)stage * GB_TILE_BYTES;
            int64_t t = t0;
            while (t < t0 + rows_here) {
                while (s_end <= t) {                      // next survivor (zero-length ones fall through)
                    ++s;
                    s_begin = s_end;
                    s_end = __ldg(cu_seqlens + s + 1);
                    s_src = __ldg(src_tok_off + __ldg(survivor_idx + s));
                }
                const int64_t seg = min(s_end, t0 + rows_here) - t;          // rows of this tile inside survivor s
                bulk_load(dst + (t - t0) * row_bytes, src_rows + (s_src + (t - s_begin)) * row_bytes,
                          (uint32_t)(seg * row_bytes), &full[stage]);
                t += seg;
            }
            ++issued;
            if (++stage == GB_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) {   // gave up: let the loads already issued land before shared memory goes away (bounded)
            const uint32_t pending = issued < (uint32_t)GB_STAGES ? issued : (uint32_t)GB_STAGES;
            uint32_t st = stage, ph = phase;
            for (uint32_t i = 0; i < pending; ++i) {
                if (st == 0) { st = GB_STAGES - 1; ph ^= 1u; } else { --st; }
                for (uint32_t it = 0; it < SPIN_LIMIT; ++it)
                    if (mbar_try_wait(&full[st], ph)) break;
            }
        }
    } else if (threadIdx.x == 32 && tile_begin < tile_end) {
        // ---------------- storer ----------------
        uint32_t stage = 0, phase = 0;
        int prev_stage = -1;
        for (int64_t tile = tile_begin; tile < tile_end; ++tile) {
            const int64_t t0 = tile * tile_rows;
            const int rows_here = (int)min((int64_t)tile_rows, T - t0);
            if (!mbar_wait(&full[stage], phase, abort_flag)) break;
            fence_proxy_async_smem();
            bulk_store(dst_rows + t0 * row_bytes, smem + (size_t)stage * GB_TILE_BYTES, (uint32_t)(rows_here * row_bytes));
            bulk_commit_group();
            if (prev_stage >= 0) {                        // the store before this one has read its stage: free it
                bulk_wait_read_but_one();
                mbar_arrive(&empty[prev_stage]);
            }
            prev_stage = (int)stage;
            if (++stage == GB_STAGES) { stage = 0; phase ^= 1u; }
        }
        bulk_wait_all();                                  // stores complete before the block's shared memory goes
    }
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) atomicOr(d_status, ARROL_DEV_WAIT_EXPIRED);
}

}  // namespace

// Moves the survivors' rows with bulk copies.  ARROL_ERR_UNSUPPORTED (nothing launched) for rows that do not fit a
// stage; the caller then takes the load/store kernel.
int arrol_internal_gather_rows_bulk(arrol_ctx* ctx, const int64_t* d_num, const int64_t* cu_seqlens,
                                    const int32_t* survivor_idx, const int64_t* src_tok_off, const void* src_rows,
                                    int64_t row_bytes, int64_t capacity, void* dst_rows, cudaStream_t s) {
    if (row_bytes <= 0 || row_bytes % 16 != 0 || row_bytes > GB_TILE_BYTES) return ARROL_ERR_UNSUPPORTED;
    const int tile_rows = (int)(GB_TILE_BYTES / row_bytes);
    const int64_t max_tiles = (capacity + tile_rows - 1) / tile_rows;
    if (!ctx->gather_bulk_smem_set) {
        ARROL_CUDA_OK(cudaFuncSetAttribute(gather_rows_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                           (int)GB_SMEM));
        // all of the SM's shared memory, so that the three blocks fit side by side
        ARROL_CUDA_OK(cudaFuncSetAttribute(gather_rows_bulk_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                                           (int)cudaSharedmemCarveoutMaxShared));
        ctx->gather_bulk_smem_set = true;
    }
    int64_t blocks = (int64_t)ctx->sm_count * GB_BLOCKS_PER_SM;
    if (blocks > max_tiles) blocks = max_tiles;
    if (blocks < 1) blocks = 1;
    ARROL_CUDA_OK(arrol_launch_pdl(gather_rows_bulk_kernel, dim3((unsigned)blocks), dim3(GB_THREADS), GB_SMEM, s, d_num,
                                   cu_seqlens, survivor_idx, src_tok_off, static_cast<const uint8_t*>(src_rows),
                                   row_bytes, capacity, tile_rows, static_cast<uint8_t*>(dst_rows), ctx->d_status));
    ctx->launches += 1;
    return ARROL_OK;
}
