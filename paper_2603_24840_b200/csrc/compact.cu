// arrol_compact: filter pruned rollouts and re-batch the survivors (Section 4.3 (ii); Algorithm 1), with the
// group-relative advantage evaluated on the survivors (Section 3).
//
// Kernel 1 (one block): stable partition by a block-wide prefix sum over (kept flag, kept length):
//   survivor_idx, cu_seqlens, {S, T}, and per-survivor advantages (fp64 statistics over the kept rollouts of
//   the group, in index order, rounded once to fp32).
// Kernel 2: the per-token outputs (token id, survivor ordinal, advantage), one block per survivor, and, when there is
//   a hidden-row plane, the rows themselves by bulk copies through shared memory (gather_bulk.cu).  Rows too large
//   for a bulk stage take gather_kernel below: one wave of persistent blocks, each owning a contiguous run of
//   destination tiles; one thread per row finds its survivor (binary search once per block, then a forward walk in
//   cu_seqlens), then the block streams the tile's payload with 16-byte loads/stores, eight in flight per thread.
//   T is read from device memory, so there is no host synchronisation between the kernels.
#include "arrol_internal.h"
#include "prune_kernels.cuh"

namespace {

__global__ void __launch_bounds__(SCAN_THREADS)
scan_adv_kernel(const uint8_t* __restrict__ keep, const int32_t* __restrict__ lengths, int N, int G,
                const float* __restrict__ rewards, double eps, int ddof, int64_t capacity,
                int32_t* __restrict__ survivor_idx, int64_t* __restrict__ cu_seqlens, float* __restrict__ adv,
                int64_t* __restrict__ d_num, uint32_t* __restrict__ d_status,
                const int64_t* __restrict__ src_tok_off, int64_t source_rows) {
    pdl_launch_dependents();
    pdl_wait();
    keep = pdl_acquire(keep); lengths = pdl_acquire(lengths); rewards = pdl_acquire(rewards);
    src_tok_off = pdl_acquire(src_tok_off);
    scan_adv_block(keep, lengths, N, G, rewards, eps, ddof, capacity, survivor_idx, cu_seqlens, adv, d_num, d_status,
                   src_tok_off, source_rows);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream(uint4* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

constexpr int GATHER_THREADS = 256;

// Largest s in [lo, hi) with cu_seqlens[s] <= t, given cu_seqlens[lo] <= t < cu_seqlens[hi].  Taking the last
// such s skips zero-length survivors.
__device__ __forceinline__ int find_survivor(const int64_t* __restrict__ cu_seqlens, int lo, int hi, int64_t t) {
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(cu_seqlens + mid) <= t) lo = mid; else hi = mid;
    }
    return lo;
}

constexpr int MAX_TILE_ROWS = 256;
constexpr int BATCH_VECS = 8 * GATHER_THREADS;   // 16-byte vectors a block moves per pass: 32 KB

// tile_rows: destination rows per tile (<= MAX_TILE_ROWS); vec_per_row = row_bytes / 16 (0 without payload).
// Every block owns a contiguous run of tiles: it locates its first row's survivor once by binary search and
// then only walks forward, so the per-tile look-up is a load or two instead of a search.
__global__ void __launch_bounds__(GATHER_THREADS, 5)
gather_kernel(const int64_t* __restrict__ d_num, const int64_t* __restrict__ cu_seqlens,
              const int32_t* __restrict__ survivor_idx, const int64_t* __restrict__ src_tok_off,
              const int32_t* __restrict__ src_tokens, const uint4* __restrict__ src_rows, int vec_per_row,
              const float* __restrict__ adv, int64_t capacity, int tile_rows, int32_t* __restrict__ dst_tokens,
              uint4* __restrict__ dst_rows, float* __restrict__ tok_adv, int32_t* __restrict__ tok_seq,
              const uint32_t* __restrict__ gate) {
    __shared__ int64_t src_row_of[MAX_TILE_ROWS];
    __shared__ int s_first[2];               // survivor of the first row of the current / next tile
    pdl_launch_dependents();
    pdl_wait();
    d_num = pdl_acquire(d_num); cu_seqlens = pdl_acquire(cu_seqlens); survivor_idx = pdl_acquire(survivor_idx);
    src_tok_off = pdl_acquire(src_tok_off); src_tokens = pdl_acquire(src_tokens); src_rows = pdl_acquire(src_rows);
    adv = pdl_acquire(adv); gate = pdl_acquire(gate);
    const int S = (int)d_num[0];
    const int64_t T = d_num[1];
    if (T > capacity || S <= 0 || T <= 0 || *gate) return;   // overflow / bad index was recorded by the scan kernel
    const int64_t n_tiles = (T + tile_rows - 1) / tile_rows;
    const int64_t tiles_per_block = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int64_t tile_begin = (int64_t)blockIdx.x * tiles_per_block;
    const int64_t tile_end = min(n_tiles, tile_begin + tiles_per_block);
    if (tile_begin >= tile_end) return;
    if (threadIdx.x == 0) s_first[0] = find_survivor(cu_seqlens, 0, S, tile_begin * tile_rows);
    __syncthreads();
    int parity = 0;
    for (int64_t tile = tile_begin; tile < tile_end; ++tile, parity ^= 1) {
        const int64_t t0 = tile * tile_rows;
        const int rows_here = (int)min((int64_t)tile_rows, T - t0);
        const int s0 = s_first[parity];
        for (int r = threadIdx.x; r < rows_here; r += GATHER_THREADS) {
            const int64_t t = t0 + r;
            int s = s0;
            for (int steps = 0; __ldg(cu_seqlens + s + 1) <= t; ++steps) {
                if (steps == 8) { s = find_survivor(cu_seqlens, s, S, t); break; }   // many short survivors
                ++s;
            }
            const int64_t src = __ldg(src_tok_off + __ldg(survivor_idx + s)) + (t - __ldg(cu_seqlens + s));
            src_row_of[r] = src;
            if (dst_tokens) dst_tokens[t] = __ldg(src_tokens + src);
            if (tok_seq) tok_seq[t] = s;
            if (tok_adv) tok_adv[t] = __ldg(adv + s);
            if (r == rows_here - 1) s_first[parity ^ 1] = s;
        }
        __syncthreads();
        if (vec_per_row > 0) {
            const int total = rows_here * vec_per_row;
            uint4* dst = dst_rows + t0 * vec_per_row;
            // eight 16-byte loads in flight per thread; the last pass of a tile is predicated
            for (int v0 = 0; v0 < total; v0 += BATCH_VECS) {
                uint4 buf[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int vv = v0 + u * GATHER_THREADS + threadIdx.x;
                    if (vv < total) {
                        const int r = vv / vec_per_row;
                        buf[u] = ld_stream(src_rows + src_row_of[r] * vec_per_row + (vv - r * vec_per_row));
                    }
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int vv = v0 + u * GATHER_THREADS + threadIdx.x;
                    if (vv < total) st_stream(dst + vv, buf[u]);
                }
            }
            __syncthreads();
        }
    }
}

// Per-token outputs without a payload plane (token ids, survivor ordinal, advantage): one block per survivor walks
// its run of tokens with coalesced 4-byte accesses, so nothing has to be searched.  Blocks past S return at once.
constexpr int TOKENS_THREADS = 128;
constexpr int TOKENS_PER_THREAD = 16;   // token ids in flight per thread (4: 28.7 us, 8: 26.4, 16: 24.6 for the Qwen-3-4B-shaped step)
__global__ void __launch_bounds__(TOKENS_THREADS)
gather_tokens_kernel(const int64_t* __restrict__ d_num, const int64_t* __restrict__ cu_seqlens,
                     const int32_t* __restrict__ survivor_idx, const int64_t* __restrict__ src_tok_off,
                     const int32_t* __restrict__ src_tokens, const float* __restrict__ adv, int64_t capacity,
                     int32_t* __restrict__ dst_tokens, float* __restrict__ tok_adv, int32_t* __restrict__ tok_seq,
                     const uint32_t* __restrict__ gate) {
    pdl_launch_dependents();
    pdl_wait();
    d_num = pdl_acquire(d_num); cu_seqlens = pdl_acquire(cu_seqlens); survivor_idx = pdl_acquire(survivor_idx);
    src_tok_off = pdl_acquire(src_tok_off); src_tokens = pdl_acquire(src_tokens); adv = pdl_acquire(adv);
    gate = pdl_acquire(gate);
    const int S = (int)d_num[0];
    if (d_num[1] > capacity || *gate) return;              // overflow / bad index was recorded by the scan kernel
    for (int s = blockIdx.x; s < S; s += gridDim.x) {
        const int64_t c0 = __ldg(cu_seqlens + s);
        const int len = (int)(__ldg(cu_seqlens + s + 1) - c0);
        const int64_t src0 = __ldg(src_tok_off + __ldg(survivor_idx + s));
        const float a = __ldg(adv + s);
        for (int t0 = threadIdx.x; t0 < len; t0 += TOKENS_PER_THREAD * TOKENS_THREADS) {
            int32_t tok[TOKENS_PER_THREAD];
#pragma unroll
            for (int u = 0; u < TOKENS_PER_THREAD; ++u) {
                const int t = t0 + u * TOKENS_THREADS;
                if (dst_tokens && t < len) tok[u] = __ldg(src_tokens + src0 + t);
            }
#pragma unroll
            for (int u = 0; u < TOKENS_PER_THREAD; ++u) {
                const int t = t0 + u * TOKENS_THREADS;
                if (t < len) {
                    if (dst_tokens) dst_tokens[c0 + t] = tok[u];
                    if (tok_seq) tok_seq[c0 + t] = s;
                    if (tok_adv) tok_adv[c0 + t] = a;
                }
            }
        }
    }
}

}  // namespace

// Argument checks of arrol_compact, shared with arrol_prune_step's fused path.
int arrol_internal_check_compact(const uint8_t* keep, const int32_t* lengths, const int64_t* src_tok_off, int32_t N,
                                 int32_t G, const int32_t* src_tokens, const void* src_rows, int32_t row_bytes,
                                 const float* rewards, float eps, int32_t ddof, int64_t dst_capacity_tokens,
                                 const int32_t* dst_tokens, const void* dst_rows, const int64_t* cu_seqlens,
                                 const int32_t* survivor_idx, const float* adv, const int64_t* d_num) {
    if (N < 0 || G < 1 || dst_capacity_tokens < 0 || ddof < 0 || !(eps >= 0.f)) return ARROL_ERR_INVALID_ARG;
    if (!cu_seqlens || !d_num) return ARROL_ERR_INVALID_ARG;
    if (N > 0 && (!keep || !lengths || !src_tok_off || !rewards || !survivor_idx || !adv))
        return ARROL_ERR_INVALID_ARG;
    if (N % G != 0) return ARROL_ERR_INVALID_ARG;
    if ((src_tokens != nullptr) != (dst_tokens != nullptr)) return ARROL_ERR_INVALID_ARG;
    if ((src_rows != nullptr) != (dst_rows != nullptr)) return ARROL_ERR_INVALID_ARG;
    if (src_rows) {
        if (row_bytes <= 0) return ARROL_ERR_INVALID_ARG;
        if (row_bytes % 16 != 0) return ARROL_ERR_UNSUPPORTED;
        if (!arrol_aligned(src_rows, 16) || !arrol_aligned(dst_rows, 16)) return ARROL_ERR_INVALID_ARG;
    }
    return ARROL_OK;
}

// arrol_compact with the scan kernel optional: the fused prune step has already produced the scan outputs.
int arrol_internal_compact(arrol_ctx* ctx, const uint8_t* keep, const int32_t* lengths,
                             const int64_t* src_tok_off, int32_t N, int32_t G, const int32_t* src_tokens,
                             const void* src_rows, int32_t row_bytes, const float* rewards, float eps,
                             int32_t ddof, int64_t dst_capacity_tokens, int32_t* dst_tokens, void* dst_rows,
                             int64_t* cu_seqlens, int32_t* survivor_idx, float* adv, float* tok_adv,
                             int32_t* tok_seq, int64_t* d_num, void* stream, bool scan_done) {
    if (!ctx) return ARROL_ERR_INVALID_ARG;
    {
        const int rc = arrol_internal_check_compact(keep, lengths, src_tok_off, N, G, src_tokens, src_rows, row_bytes,
                                                    rewards, eps, ddof, dst_capacity_tokens, dst_tokens, dst_rows,
                                                    cu_seqlens, survivor_idx, adv, d_num);
        if (rc != ARROL_OK) return rc;
    }
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (!scan_done) {
        ARROL_CUDA_OK(arrol_launch_pdl(scan_adv_kernel, dim3(1), dim3(SCAN_THREADS), 0, s, keep, lengths, N, G, rewards,
                                       (double)eps, ddof, dst_capacity_tokens, survivor_idx, cu_seqlens, adv, d_num,
                                       ctx->d_status, src_tok_off, ctx->source_rows));
        ctx->launches += 1;
    }
    const bool any_token_output = dst_tokens || dst_rows || tok_adv || tok_seq;
    if (N == 0 || dst_capacity_tokens == 0 || !any_token_output) return ARROL_OK;

    const int vec_per_row = src_rows ? row_bytes / 16 : 0;
    // Rows that fit a 32 KB stage go through the bulk-copy kernel; the per-token outputs then come from the
    // survivor-major kernel.  Larger rows take the load/store kernel, which writes both.
    const bool bulk_rows = vec_per_row > 0 && row_bytes <= 32 * 1024;
    if (vec_per_row == 0 || bulk_rows) {
        if (bulk_rows) {
            const int rc = arrol_internal_gather_rows_bulk(ctx, d_num, cu_seqlens, survivor_idx, src_tok_off, src_rows,
                                                           row_bytes, dst_capacity_tokens, dst_rows, s);
            if (rc != ARROL_OK) return rc;
            if (!dst_tokens && !tok_adv && !tok_seq) return ARROL_OK;
        }
        int64_t blocks = N < (int64_t)ctx->sm_count * 16 ? N : (int64_t)ctx->sm_count * 16;
        ARROL_CUDA_OK(arrol_launch_pdl(gather_tokens_kernel, dim3((unsigned)blocks), dim3(TOKENS_THREADS), 0, s, d_num,
                                       cu_seqlens, survivor_idx, src_tok_off, src_tokens, adv, dst_capacity_tokens,
                                       dst_tokens, tok_adv, tok_seq, ctx->d_status + 1));
        ctx->launches += 1;
        return ARROL_OK;
    }
    // as many whole rows as fit one 32 KB pass (rows larger than that take several passes each)
    int tile_rows = BATCH_VECS / vec_per_row;
    if (tile_rows < 1) tile_rows = 1;
    if (tile_rows > MAX_TILE_ROWS) tile_rows = MAX_TILE_ROWS;
    if ((int64_t)tile_rows * vec_per_row > INT32_MAX) return ARROL_ERR_UNSUPPORTED;
    const int64_t max_tiles = (dst_capacity_tokens + tile_rows - 1) / tile_rows;
    // Exactly one wave: every block owns an equal contiguous share of the destination, so a partial second wave
    // would leave SMs idle at the end.
    int resident = 0;
    ARROL_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, gather_kernel, GATHER_THREADS, 0));
    if (resident < 1) resident = 1;
    int64_t blocks = (int64_t)ctx->sm_count * resident;
    if (blocks > max_tiles) blocks = max_tiles;
    if (blocks < 1) blocks = 1;
    ARROL_CUDA_OK(arrol_launch_pdl(gather_kernel, dim3((unsigned)blocks), dim3(GATHER_THREADS), 0, s, d_num, cu_seqlens,
                                   survivor_idx, src_tok_off, src_tokens, static_cast<const uint4*>(src_rows),
                                   vec_per_row, adv, dst_capacity_tokens, tile_rows, dst_tokens,
                                   static_cast<uint4*>(dst_rows), tok_adv, tok_seq, ctx->d_status + 1));
    ctx->launches += 1;
    return ARROL_OK;
}

extern "C" int arrol_compact(arrol_ctx* ctx, const uint8_t* keep, const int32_t* lengths,
                             const int64_t* src_tok_off, int32_t N, int32_t G, const int32_t* src_tokens,
                             const void* src_rows, int32_t row_bytes, const float* rewards, float eps,
                             int32_t ddof, int64_t dst_capacity_tokens, int32_t* dst_tokens, void* dst_rows,
                             int64_t* cu_seqlens, int32_t* survivor_idx, float* adv, float* tok_adv,
                             int32_t* tok_seq, int64_t* d_num, void* stream) {
    return arrol_internal_compact(ctx, keep, lengths, src_tok_off, N, G, src_tokens, src_rows, row_bytes, rewards, eps,
                                  ddof, dst_capacity_tokens, dst_tokens, dst_rows, cu_seqlens, survivor_idx, adv, tok_adv,
                                  tok_seq, d_num, stream, false);
}
