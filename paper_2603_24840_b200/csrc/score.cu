// arrol_score_partial: quality head on the hidden state at the detection length, sigmoid, bin index and
// posterior lookup (Section 4.2; Appendix A.4).
//
// Linear head: HBM-bound row reduction, one warp per rollout, 16-byte loads (eight in flight per lane), shuffle
// reduction, with the
// probability map fused into lane 0's epilogue.
// MLP head: fp32 SIMT register-tiled contraction (64 rollouts x 64 hidden units per block, 8 x 4 per thread,
// next K chunk prefetched into registers) with the bias,
// exact GELU and the w2 dot product fused into the tile epilogue; per-tile partial scores go to the context
// scratch and a finishing kernel adds them in a fixed order and applies the probability map.
#include <cuda_bf16.h>

#include "arrol_internal.h"
#include "prune_kernels.cuh"
#include "score_common.cuh"

namespace {

// CHECK: the row numbers are range-checked against source_rows (arrol_set_source_rows); a separate instantiation, so
// that the unchecked kernel keeps its 80 registers and six blocks per SM (with the check compiled in, 86-88 registers
// and five blocks cost the streamed form of the kernel a tenth of its bandwidth)
template <typename T, bool CHECK>
__global__ void __launch_bounds__(128)
score_linear_kernel(const T* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index, int N,
                    int d, const T* __restrict__ w, const T* __restrict__ bias, int B,
                    const float* __restrict__ q_lut, float* score, float* prob, int32_t* bin, float* q,
                    int64_t source_rows, uint32_t* d_status) {
    constexpr int VN = Vec16<T>::N;
    pdl_launch_dependents();
    pdl_wait();
    hidden = pdl_acquire(hidden); row_index = pdl_acquire(row_index); w = pdl_acquire(w); bias = pdl_acquire(bias);
    q_lut = pdl_acquire(q_lut);
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int64_t row = row_index ? row_index[warp] : (int64_t)warp;
    const T* x = hidden + row * row_stride;
    if constexpr (CHECK) {
        if (row < 0 || row >= source_rows) {   // outside the caller's buffer: never read, scored as zeros
            if (lane == 0) {
                atomicOr(d_status, ARROL_DEV_BAD_INDEX);
                probability_map(bias ? to_f32(bias[0]) : 0.f, warp, B, q_lut, score, prob, bin, q);
            }
            return;
        }
    }
    const int nvec = d / VN;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    // eight independent 16-byte loads of x (and of w) in flight per lane: a 4 KB row is one round trip.  (The fused
    // prune step's linear_row_dot_ws takes the same products and sums in the same order with w in shared memory.)
    for (int c0 = lane; c0 < nvec; c0 += 256) {
        typename Vec16<T>::Raw xr[8], wr[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int c = c0 + 32 * u;
            if (c < nvec) {
                xr[u] = Vec16<T>::load_raw(x + (int64_t)c * VN);
                wr[u] = Vec16<T>::load_raw(w + (int64_t)c * VN);
            }
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (c0 + 32 * u < nvec) acc[u & 3] = Vec16<T>::dot(xr[u], wr[u], acc[u & 3]);
    }
    float s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        if (bias) s += to_f32(bias[0]);
        probability_map(s, warp, B, q_lut, score, prob, bin, q);
    }
}

// ---- MLP head ---------------------------------------------------------------------------------------
// Block tile: TM = 64 rollouts x TH = 64 hidden units, K chunks of 32; 128 threads, 8 x 4 outputs each.
// The next K chunk is fetched from global memory into registers while the current one is multiplied out of
// shared memory (two shared buffers, one barrier per chunk).
constexpr int TM = 64, TH = ARROL_MLP_TH, TK = 32, PAD = 4, MLP_THREADS = 128;

// SPLITK = false: the block contracts the whole of d and finishes its tile (bias, GELU, w2 dot) -> partial [h_tiles][N].
// SPLITK = true:  blockIdx.z picks a K range of k_len columns; the raw partial pre-activations go to
//                 partial [splits][N][h] and score_mlp_splitk_finish_kernel completes them.  More, shorter blocks:
//                 this is what fills the SMs when N x h is only a few hundred tiles.
template <typename T, bool SPLITK>
__global__ void __launch_bounds__(MLP_THREADS)
score_mlp_tile_kernel(const T* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index,
                      int N, int d, int h, const T* __restrict__ W1, const T* __restrict__ b1,
                      const T* __restrict__ w2, float* __restrict__ partial,
                      float* __restrict__ u_out /* [N][h] pre-activations, or NULL */, int k_len,
                      int64_t source_rows, uint32_t* d_status) {
    constexpr int VN = Vec16<T>::N;
    constexpr int VPR = TK / VN;                       // 16-byte vectors per tile row per K chunk
    constexpr int NV = TM * VPR / MLP_THREADS;         // vectors per thread per operand per chunk (2 or 4)
    static_assert(TM == TH && (TM * VPR) % MLP_THREADS == 0, "tile / thread mapping");
    __shared__ __align__(16) float xs[2][TK][TM + PAD];
    __shared__ __align__(16) float ws[2][TK][TH + PAD];

    const int m0 = blockIdx.x * TM, j0 = blockIdx.y * TH;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // tx: 4 hidden units each, ty: 8 rollouts each

    // Global -> register staging.  Vector v of a chunk covers tile row (v % TM), K offset (v / TM) * VN, so that
    // the lanes of a warp write consecutive shared-memory columns (no bank conflicts).
    const T* xrow[NV];
    const T* wrow[NV];
    int kofs[NV], rr[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
        const int v = threadIdx.x + i * MLP_THREADS;
        rr[i] = v % TM;
        kofs[i] = (v / TM) * VN;
        const int m = m0 + rr[i], j = j0 + rr[i];
        xrow[i] = nullptr;
        wrow[i] = nullptr;
        if (m < N) {
            const int64_t row = row_index ? row_index[m] : (int64_t)m;
            if (source_rows > 0 && (row < 0 || row >= source_rows)) atomicOr(d_status, ARROL_DEV_BAD_INDEX);   // read as zeros
            else xrow[i] = hidden + row * row_stride;
        }
        if (j < h) wrow[i] = W1 + (int64_t)j * d;
    }
    const int k_end = SPLITK ? min(d, ((int)blockIdx.z + 1) * k_len) : d;
    float xreg[NV][VN], wreg[NV][VN];
    auto fetch = [&](int k0) {
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const int k = k0 + kofs[i];
            if (xrow[i] && k < k_end) Vec16<T>::load(xrow[i] + k, xreg[i]);
            else {
#pragma unroll
                for (int e = 0; e < VN; ++e) xreg[i][e] = 0.f;
            }
            if (wrow[i] && k < k_end) Vec16<T>::load(wrow[i] + k, wreg[i]);
            else {
#pragma unroll
                for (int e = 0; e < VN; ++e) wreg[i][e] = 0.f;
            }
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int e = 0; e < VN; ++e) {
                xs[buf][kofs[i] + e][rr[i]] = xreg[i][e];
                ws[buf][kofs[i] + e][rr[i]] = wreg[i][e];
            }
    };

    float acc[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    const int k_lo = SPLITK ? (int)blockIdx.z * k_len : 0;
    const int k_hi = SPLITK ? min(d, k_lo + k_len) : d;
    fetch(k_lo);
    stash(0);
    __syncthreads();
    int buf = 0;
    for (int k0 = k_lo; k0 < k_hi; k0 += TK, buf ^= 1) {
        const bool more = k0 + TK < k_hi;
        if (more) fetch(k0 + TK);
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const float4 xa = *reinterpret_cast<const float4*>(&xs[buf][k][ty * 8]);
            const float4 xb = *reinterpret_cast<const float4*>(&xs[buf][k][ty * 8 + 4]);
            const float4 wb = *reinterpret_cast<const float4*>(&ws[buf][k][tx * 4]);
            const float xr[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
            const float wr[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xr[a], wr[b], acc[a][b]);
        }
        if (more) stash(buf ^ 1);      // the other buffer was last read before the previous barrier
        __syncthreads();
    }

    if constexpr (SPLITK) {   // raw partial pre-activations of this K range
        float* out = partial + (int64_t)blockIdx.z * N * h;
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            const int m = m0 + ty * 8 + a, j = j0 + tx * 4;
            if (m < N && j < h)     // h % 4 == 0: a float4 never straddles the edge
                *reinterpret_cast<float4*>(out + (int64_t)m * h + j) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        }
    } else {
    // epilogue: u + b1 -> exact GELU -> dot with w2 over this tile's hidden units
    float part[8];
#pragma unroll
    for (int a = 0; a < 8; ++a) part[a] = 0.f;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int j = j0 + tx * 4 + b;
        if (j < h) {
            const float bj = b1 ? to_f32(b1[j]) : 0.f;
            const float wj = to_f32(w2[j]);
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                const float u = acc[a][b] + bj;
                if (u_out && m0 + ty * 8 + a < N) u_out[(int64_t)(m0 + ty * 8 + a) * h + j] = u;
                const float g = 0.5f * u * (1.0f + erff(u * 0.70710678118654752440f));
                part[a] = fmaf(wj, g, part[a]);
            }
        }
    }
    // the 16 threads that share a group of 8 rollouts are one half-warp: reduce over tx
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) part[a] += __shfl_xor_sync(0xffffffffu, part[a], o, 16);
    if (tx == 0) {
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            const int m = m0 + ty * 8 + a;
            if (m < N) partial[(int64_t)blockIdx.y * N + m] = part[a];
        }
    }
    }
}

template <typename T>
__global__ void score_mlp_finish_kernel(const float* __restrict__ partial, int N, int h_tiles,
                                        const T* __restrict__ b2, int B, const float* __restrict__ q_lut,
                                        float* score, float* prob, int32_t* bin, float* q) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    float s = 0.f;
    for (int t = 0; t < h_tiles; ++t) s += partial[(int64_t)t * N + i];
    if (b2) s += to_f32(b2[0]);
    probability_map(s, i, B, q_lut, score, prob, bin, q);
}

// One warp per rollout: u_j = b1_j + sum over the K splits, s = sum_j w2_j gelu(u_j) + b2 (lanes stride over j, fixed
// shuffle order), then the probability map.
template <typename T>
__global__ void __launch_bounds__(128)
score_mlp_splitk_finish_kernel(const float* __restrict__ upart, int splits, int N, int h, const T* __restrict__ b1,
                               const T* __restrict__ w2, const T* __restrict__ b2, int B,
                               const float* __restrict__ q_lut, float* score, float* prob, int32_t* bin, float* q) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (i >= N) return;
    float s = 0.f;
    for (int j = lane; j < h; j += 32) {
        float u = b1 ? to_f32(b1[j]) : 0.f;
        for (int z = 0; z < splits; ++z) u += upart[((int64_t)z * N + i) * h + j];
        const float g = 0.5f * u * (1.0f + erff(u * 0.70710678118654752440f));
        s = fmaf(to_f32(w2[j]), g, s);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
        if (b2) s += to_f32(b2[0]);
        probability_map(s, i, B, q_lut, score, prob, bin, q);
    }
}

template <typename T>
int launch_score(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index, int N,
                 const arrol_head* head, int B, const float* q_lut, float* score, float* prob, int32_t* bin,
                 float* q, cudaStream_t s) {
    const T* hid = static_cast<const T*>(hidden);
    if (head->h == 0) {
        const int warps_per_block = 4;
        const int blocks = (N + warps_per_block - 1) / warps_per_block;
        auto kernel = ctx->source_rows > 0 ? score_linear_kernel<T, true> : score_linear_kernel<T, false>;
        ARROL_CUDA_OK(arrol_launch_pdl(kernel, dim3(blocks), dim3(32 * warps_per_block), 0, s, hid,
                                       row_stride, row_index, N, head->d, static_cast<const T*>(head->W1),
                                       static_cast<const T*>(head->b1), B, q_lut, score, prob, bin, q,
                                       ctx->source_rows, ctx->d_status));
        ctx->launches += 1;
    } else {
        if constexpr (sizeof(T) == 2) {
            // bf16 head: the first layer is a dense contraction, so the whole head runs on the tensor-core path
            // when the context's buffers hold the problem
            const int rc = arrol_internal_score_mlp_tc(ctx, hidden, row_stride, row_index, N, head, B, q_lut, score,
                                                       prob, bin, q, nullptr, s);
            if (rc != ARROL_ERR_UNSUPPORTED) return rc;
        }
        const int h_tiles = (head->h + TH - 1) / TH;
        const int m_tiles = (N + TM - 1) / TM;
        // split d across blocks until there are about three blocks per SM, as far as the scratch allows
        int splits = (3 * ctx->sm_count + m_tiles * h_tiles - 1) / (m_tiles * h_tiles);
        if (splits > 8) splits = 8;
        const size_t per_split = (size_t)N * (size_t)head->h;
        while (splits > 1 && per_split * splits > ARROL_SCRATCH_FLOATS) --splits;
        int k_len = ((head->d + splits - 1) / splits + TK - 1) / TK * TK;
        splits = (head->d + k_len - 1) / k_len;
        if (per_split * splits <= ARROL_SCRATCH_FLOATS) {
            dim3 grid(m_tiles, h_tiles, splits);
            score_mlp_tile_kernel<T, true><<<grid, MLP_THREADS, 0, s>>>(
                hid, row_stride, row_index, N, head->d, head->h, static_cast<const T*>(head->W1), nullptr, nullptr,
                ctx->d_scratch, nullptr, k_len, ctx->source_rows, ctx->d_status);
            score_mlp_splitk_finish_kernel<T><<<(N + 3) / 4, 128, 0, s>>>(
                ctx->d_scratch, splits, N, head->h, static_cast<const T*>(head->b1), static_cast<const T*>(head->w2),
                static_cast<const T*>(head->b2), B, q_lut, score, prob, bin, q);
        } else {   // N x h too large for the scratch: one block per tile finishes its tile itself
            dim3 grid(m_tiles, h_tiles);
            score_mlp_tile_kernel<T, false><<<grid, MLP_THREADS, 0, s>>>(
                hid, row_stride, row_index, N, head->d, head->h, static_cast<const T*>(head->W1),
                static_cast<const T*>(head->b1), static_cast<const T*>(head->w2), ctx->d_scratch, nullptr, 0,
                ctx->source_rows, ctx->d_status);
            score_mlp_finish_kernel<T><<<(N + 255) / 256, 256, 0, s>>>(ctx->d_scratch, N, h_tiles,
                                                                      static_cast<const T*>(head->b2), B, q_lut,
                                                                      score, prob, bin, q);
        }
        ctx->launches += 2;
    }
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

}  // namespace

// Internal: MLP tile pass that also stores the pre-activations u [N][h] (used by the head training step).
int arrol_internal_mlp_tiles(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index, int N,
                             const arrol_head* head, float* partial, float* u_out, cudaStream_t s) {
    const int h_tiles = (head->h + TH - 1) / TH;
    dim3 grid((N + TM - 1) / TM, h_tiles);
    if (head->dtype == ARROL_F32)
        score_mlp_tile_kernel<float, false><<<grid, MLP_THREADS, 0, s>>>(
            static_cast<const float*>(hidden), row_stride, row_index, N, head->d, head->h,
            static_cast<const float*>(head->W1), static_cast<const float*>(head->b1),
            static_cast<const float*>(head->w2), partial, u_out, 0, ctx->source_rows, ctx->d_status);
    else
        score_mlp_tile_kernel<__nv_bfloat16, false><<<grid, MLP_THREADS, 0, s>>>(
            static_cast<const __nv_bfloat16*>(hidden), row_stride, row_index, N, head->d, head->h,
            static_cast<const __nv_bfloat16*>(head->W1), static_cast<const __nv_bfloat16*>(head->b1),
            static_cast<const __nv_bfloat16*>(head->w2), partial, u_out, 0, ctx->source_rows, ctx->d_status);
    ctx->launches += 1;
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

// Argument checks of arrol_score_partial (N > 0), shared with arrol_prune_step's fused path.
int arrol_internal_check_score(const void* hidden, int64_t row_stride_elems, int32_t N, const arrol_head* head,
                               const arrol_calib* calib, const float* score, const float* prob, const float* q) {
    if (!hidden || !score || !prob || !q || !head->W1) return ARROL_ERR_INVALID_ARG;
    if (head->dtype != ARROL_F32 && head->dtype != ARROL_BF16) return ARROL_ERR_INVALID_ARG;
    if (head->d <= 0 || head->h < 0) return ARROL_ERR_INVALID_ARG;
    if (head->h > 0 && !head->w2) return ARROL_ERR_INVALID_ARG;
    const int esz = head->dtype == ARROL_F32 ? 4 : 2;
    if (head->d % 8 != 0 || head->h % 4 != 0 || head->h > ARROL_MAX_H) return ARROL_ERR_UNSUPPORTED;
    if (head->h > 0 && N > ARROL_MAX_MLP_N) return ARROL_ERR_UNSUPPORTED;
    if (row_stride_elems < head->d) return ARROL_ERR_INVALID_ARG;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(head->W1, 16) || (row_stride_elems * esz) % 16 != 0)
        return ARROL_ERR_INVALID_ARG;
    if (calib && calib->q_lut && calib->B <= 0) return ARROL_ERR_INVALID_ARG;
    return ARROL_OK;
}

extern "C" int arrol_score_partial(arrol_ctx* ctx, const void* hidden, int64_t row_stride_elems,
                                   const int64_t* row_index, int32_t N, const arrol_head* head,
                                   const arrol_calib* calib, float* score, float* prob, int32_t* bin, float* q,
                                   void* stream) {
    if (!ctx || !head || N < 0) return ARROL_ERR_INVALID_ARG;
    if (N == 0) return ARROL_OK;
    {
        const int rc = arrol_internal_check_score(hidden, row_stride_elems, N, head, calib, score, prob, q);
        if (rc != ARROL_OK) return rc;
    }
    if (!hidden || !score || !prob || !q || !head->W1) return ARROL_ERR_INVALID_ARG;
    if (head->dtype != ARROL_F32 && head->dtype != ARROL_BF16) return ARROL_ERR_INVALID_ARG;
    if (head->d <= 0 || head->h < 0) return ARROL_ERR_INVALID_ARG;
    if (head->h > 0 && !head->w2) return ARROL_ERR_INVALID_ARG;
    const int esz = head->dtype == ARROL_F32 ? 4 : 2;
    if (head->d % 8 != 0 || head->h % 4 != 0 || head->h > ARROL_MAX_H) return ARROL_ERR_UNSUPPORTED;
    if (head->h > 0 && N > ARROL_MAX_MLP_N) return ARROL_ERR_UNSUPPORTED;
    if (row_stride_elems < head->d) return ARROL_ERR_INVALID_ARG;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(head->W1, 16) || (row_stride_elems * esz) % 16 != 0)
        return ARROL_ERR_INVALID_ARG;
    int B = 0;
    const float* q_lut = nullptr;
    if (calib) {
        if (calib->q_lut && calib->B <= 0) return ARROL_ERR_INVALID_ARG;
        B = calib->B > 0 ? calib->B : 0;
        q_lut = calib->q_lut;
    }
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (head->dtype == ARROL_F32)
        return launch_score<float>(ctx, hidden, row_stride_elems, row_index, N, head, B, q_lut, score, prob, bin,
                                   q, s);
    return launch_score<__nv_bfloat16>(ctx, hidden, row_stride_elems, row_index, N, head, B, q_lut, score, prob,
                                       bin, q, s);
}

// ---- MLP-head scoring without any allocation --------------------------------------------------------------
// Same kernels as above, but the per-tile partial scores live in a fixed array in device global memory that
// is part of the library image, so this entry point needs neither an arrol_ctx (whose creation allocates)
// nor any other allocation.  Every device that loads the library carries the array until the process exits.
#include <mutex>

constexpr int ARROL_STATIC_MAX_N = 4096;                       // rollouts per call
constexpr int ARROL_STATIC_MAX_H = 512;                        // hidden units of the head
constexpr int ARROL_STATIC_MAX_TILES = ARROL_STATIC_MAX_H / ARROL_MLP_TH;
constexpr int ARROL_STATIC_MAX_DEVICES = 64;

// [h_tiles][N] partial scores, 128 KiB.  In host code this name is only a handle for the runtime; the device
// address is obtained per device with cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_mlp_partial[ARROL_STATIC_MAX_TILES * ARROL_STATIC_MAX_N];

static std::mutex g_static_setup_mutex;
static float* g_static_partial_addr[ARROL_STATIC_MAX_DEVICES] = {nullptr};

extern "C" int arrol_score_partial_static(const void* hidden, int64_t row_stride_elems, const int64_t* row_index,
                                          int32_t N, const arrol_head* head, const arrol_calib* calib,
                                          float* score, float* prob, int32_t* bin, float* q, void* stream) {
    if (!head || N < 0) return ARROL_ERR_INVALID_ARG;
    if (N == 0) return ARROL_OK;
    if (!hidden || !score || !prob || !q || !head->W1 || !head->w2) return ARROL_ERR_INVALID_ARG;
    if (head->dtype != ARROL_F32 && head->dtype != ARROL_BF16) return ARROL_ERR_INVALID_ARG;
    if (head->d <= 0 || head->h <= 0) return ARROL_ERR_INVALID_ARG;      // MLP head only
    if (head->d % 8 != 0 || head->h % 4 != 0) return ARROL_ERR_UNSUPPORTED;
    if (N > ARROL_STATIC_MAX_N || head->h > ARROL_STATIC_MAX_H) return ARROL_ERR_UNSUPPORTED;   // beyond the fixed scratch
    const int esz = head->dtype == ARROL_F32 ? 4 : 2;
    if (row_stride_elems < head->d) return ARROL_ERR_INVALID_ARG;
    if (!arrol_aligned(hidden, 16) || !arrol_aligned(head->W1, 16) || (row_stride_elems * esz) % 16 != 0)
        return ARROL_ERR_INVALID_ARG;
    int B = 0;
    const float* q_lut = nullptr;
    if (calib) {
        if (calib->q_lut && calib->B <= 0) return ARROL_ERR_INVALID_ARG;
        B = calib->B > 0 ? calib->B : 0;
        q_lut = calib->q_lut;
    }

    // One-time set-up per device, on the caller's current device: resolve the array's device address.
    int dev = -1;
    ARROL_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= ARROL_STATIC_MAX_DEVICES) return ARROL_ERR_UNSUPPORTED;
    float* partial = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_setup_mutex);
        if (!g_static_partial_addr[dev]) {
            float* addr = nullptr;
            ARROL_CUDA_OK(cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_static_mlp_partial));
            if (!addr) return ARROL_ERR_CUDA;
            g_static_partial_addr[dev] = addr;
        }
        partial = g_static_partial_addr[dev];
    }

    cudaStream_t s = (cudaStream_t)stream;
    const int h_tiles = (head->h + TH - 1) / TH;
    dim3 grid((N + TM - 1) / TM, h_tiles);
    // The tile kernel writes every entry [tile][i], i < N, that the finishing kernel reads, so nothing left in
    // the array by an earlier call is ever read and nothing needs clearing.
    if (head->dtype == ARROL_F32) {
        score_mlp_tile_kernel<float, false><<<grid, MLP_THREADS, 0, s>>>(
            static_cast<const float*>(hidden), row_stride_elems, row_index, N, head->d, head->h,
            static_cast<const float*>(head->W1), static_cast<const float*>(head->b1),
            static_cast<const float*>(head->w2), partial, nullptr, 0, (int64_t)0, nullptr);
        score_mlp_finish_kernel<float><<<(N + 255) / 256, 256, 0, s>>>(
            partial, N, h_tiles, static_cast<const float*>(head->b2), B, q_lut, score, prob, bin, q);
    } else {
        score_mlp_tile_kernel<__nv_bfloat16, false><<<grid, MLP_THREADS, 0, s>>>(
            static_cast<const __nv_bfloat16*>(hidden), row_stride_elems, row_index, N, head->d, head->h,
            static_cast<const __nv_bfloat16*>(head->W1), static_cast<const __nv_bfloat16*>(head->b1),
            static_cast<const __nv_bfloat16*>(head->w2), partial, nullptr, 0, (int64_t)0, nullptr);
        score_mlp_finish_kernel<__nv_bfloat16><<<(N + 255) / 256, 256, 0, s>>>(
            partial, N, h_tiles, static_cast<const __nv_bfloat16*>(head->b2), B, q_lut, score, prob, bin, q);
    }
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
