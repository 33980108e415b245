// arrol_score_partial: quality head on the hidden state at the detection length, sigmoid, bin index and
// posterior lookup (Section 4.2; Appendix A.4).
//
// Linear head: HBM-bound row reduction, one warp per rollout, 16-byte loads, shuffle reduction, with the
// probability map fused into lane 0's epilogue.
// MLP head: fp32 SIMT register-tiled contraction (64 rollouts x 64 hidden units per block) with the bias,
// exact GELU and the w2 dot product fused into the tile epilogue; per-tile partial scores go to the context
// scratch and a finishing kernel adds them in a fixed order and applies the probability map.
#include <cuda_bf16.h>

#include "arrol_internal.h"

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// 16-byte vector of T -> floats
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    __device__ static __forceinline__ void load(const float* p, float (&out)[4]) {
        float4 v = __ldg(reinterpret_cast<const float4*>(p));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&out)[8]) {
        uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {   // a bf16 is the upper half of a binary32
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};

// s -> s' = sigmoid(s), b = min(B-1, floor(B s')), q = q_lut[b] (Appendix A.4)
__device__ __forceinline__ void probability_map(float s, int i, int B, const float* __restrict__ q_lut,
                                                float* score, float* prob, int32_t* bin, float* q) {
    float sp = 1.0f / (1.0f + expf(-s));
    int b = 0;
    if (B > 0) {
        b = (int)floorf((float)B * sp);
        b = min(max(b, 0), B - 1);
    }
    score[i] = s;
    prob[i] = sp;
    if (bin) bin[i] = b;
    q[i] = (q_lut != nullptr) ? __ldg(q_lut + b) : sp;
}

template <typename T>
__global__ void __launch_bounds__(128)
score_linear_kernel(const T* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index, int N,
                    int d, const T* __restrict__ w, const T* __restrict__ bias, int B,
                    const float* __restrict__ q_lut, float* score, float* prob, int32_t* bin, float* q) {
    constexpr int VN = Vec16<T>::N;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= N) return;
    const int64_t row = row_index ? row_index[warp] : (int64_t)warp;
    const T* x = hidden + row * row_stride;
    const int nvec = d / VN;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    int c = lane;
    // four independent 16-byte loads in flight per lane
    for (; c + 96 < nvec; c += 128) {
        float xv[4][VN], wv[4][VN];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            Vec16<T>::load(x + (int64_t)(c + 32 * u) * VN, xv[u]);
            Vec16<T>::load(w + (int64_t)(c + 32 * u) * VN, wv[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int e = 0; e < VN; ++e) acc[u] = fmaf(xv[u][e], wv[u][e], acc[u]);
    }
    for (; c < nvec; c += 32) {
        float xv[VN], wv[VN];
        Vec16<T>::load(x + (int64_t)c * VN, xv);
        Vec16<T>::load(w + (int64_t)c * VN, wv);
#pragma unroll
        for (int e = 0; e < VN; ++e) acc[0] = fmaf(xv[e], wv[e], acc[0]);
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
// Block tile: TM = 64 rollouts x TH = 64 hidden units, K chunks of 32; 256 threads, 4 x 4 outputs each.
constexpr int TM = 64, TH = ARROL_MLP_TH, TK = 32, PAD = 4;

template <typename T>
__global__ void __launch_bounds__(256)
score_mlp_tile_kernel(const T* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index,
                      int N, int d, int h, const T* __restrict__ W1, const T* __restrict__ b1,
                      const T* __restrict__ w2, float* __restrict__ partial /* [h_tiles][N] */) {
    constexpr int VN = Vec16<T>::N;
    constexpr int VPR = TK / VN;               // 16-byte vectors per tile row per K chunk
    __shared__ __align__(16) float xs[TK][TM + PAD];
    __shared__ __align__(16) float ws[TK][TH + PAD];

    const int m0 = blockIdx.x * TM, j0 = blockIdx.y * TH;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;   // tx: hidden units, ty: rollouts

    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

    for (int k0 = 0; k0 < d; k0 += TK) {
        // stage X[m0..m0+63][k0..k0+31] and W1[j0..j0+63][k0..k0+31] as fp32, k-major
        for (int v = threadIdx.x; v < TM * VPR; v += 256) {
            const int r = v / VPR, cv = v % VPR;
            const int k = k0 + cv * VN;
            float vals[VN];
            const int m = m0 + r;
            if (m < N && k < d) {
                const int64_t row = row_index ? row_index[m] : (int64_t)m;
                Vec16<T>::load(hidden + row * row_stride + k, vals);
            } else {
#pragma unroll
                for (int e = 0; e < VN; ++e) vals[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < VN; ++e) xs[cv * VN + e][r] = vals[e];
        }
        for (int v = threadIdx.x; v < TH * VPR; v += 256) {
            const int r = v / VPR, cv = v % VPR;
            const int k = k0 + cv * VN;
            float vals[VN];
            const int j = j0 + r;
            if (j < h && k < d) {
                Vec16<T>::load(W1 + (int64_t)j * d + k, vals);
            } else {
#pragma unroll
                for (int e = 0; e < VN; ++e) vals[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < VN; ++e) ws[cv * VN + e][r] = vals[e];
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            const float4 xa = *reinterpret_cast<const float4*>(&xs[k][ty * 4]);
            const float4 wb = *reinterpret_cast<const float4*>(&ws[k][tx * 4]);
            const float xr[4] = {xa.x, xa.y, xa.z, xa.w};
            const float wr[4] = {wb.x, wb.y, wb.z, wb.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xr[a], wr[b], acc[a][b]);
        }
        __syncthreads();
    }

    // epilogue: u + b1 -> exact GELU -> dot with w2 over this tile's hidden units
    float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        const int j = j0 + tx * 4 + b;
        if (j < h) {
            const float bj = b1 ? to_f32(b1[j]) : 0.f;
            const float wj = to_f32(w2[j]);
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const float u = acc[a][b] + bj;
                const float g = 0.5f * u * (1.0f + erff(u * 0.70710678118654752440f));
                part[a] = fmaf(wj, g, part[a]);
            }
        }
    }
    // the 16 threads of one rollout quadruple are lanes (ty & 1) * 16 + tx of a warp: reduce over tx
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) part[a] += __shfl_xor_sync(0xffffffffu, part[a], o, 16);
    if (tx == 0) {
#pragma unroll
        for (int a = 0; a < 4; ++a) {
            const int m = m0 + ty * 4 + a;
            if (m < N) partial[(int64_t)blockIdx.y * N + m] = part[a];
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

template <typename T>
int launch_score(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index, int N,
                 const arrol_head* head, int B, const float* q_lut, float* score, float* prob, int32_t* bin,
                 float* q, cudaStream_t s) {
    const T* hid = static_cast<const T*>(hidden);
    if (head->h == 0) {
        const int warps_per_block = 4;
        const int blocks = (N + warps_per_block - 1) / warps_per_block;
        score_linear_kernel<T><<<blocks, 32 * warps_per_block, 0, s>>>(
            hid, row_stride, row_index, N, head->d, static_cast<const T*>(head->W1),
            static_cast<const T*>(head->b1), B, q_lut, score, prob, bin, q);
        ctx->launches += 1;
    } else {
        const int h_tiles = (head->h + TH - 1) / TH;
        dim3 grid((N + TM - 1) / TM, h_tiles);
        score_mlp_tile_kernel<T><<<grid, 256, 0, s>>>(hid, row_stride, row_index, N, head->d, head->h,
                                                     static_cast<const T*>(head->W1),
                                                     static_cast<const T*>(head->b1),
                                                     static_cast<const T*>(head->w2), ctx->d_scratch);
        score_mlp_finish_kernel<T><<<(N + 255) / 256, 256, 0, s>>>(ctx->d_scratch, N, h_tiles,
                                                                  static_cast<const T*>(head->b2), B, q_lut,
                                                                  score, prob, bin, q);
        ctx->launches += 2;
    }
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

}  // namespace

extern "C" int arrol_score_partial(arrol_ctx* ctx, const void* hidden, int64_t row_stride_elems,
                                   const int64_t* row_index, int32_t N, const arrol_head* head,
                                   const arrol_calib* calib, float* score, float* prob, int32_t* bin, float* q,
                                   void* stream) {
    if (!ctx || !head || N < 0) return ARROL_ERR_INVALID_ARG;
    if (N == 0) return ARROL_OK;
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
        score_mlp_tile_kernel<float><<<grid, 256, 0, s>>>(
            static_cast<const float*>(hidden), row_stride_elems, row_index, N, head->d, head->h,
            static_cast<const float*>(head->W1), static_cast<const float*>(head->b1),
            static_cast<const float*>(head->w2), partial);
        score_mlp_finish_kernel<float><<<(N + 255) / 256, 256, 0, s>>>(
            partial, N, h_tiles, static_cast<const float*>(head->b2), B, q_lut, score, prob, bin, q);
    } else {
        score_mlp_tile_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(
            static_cast<const __nv_bfloat16*>(hidden), row_stride_elems, row_index, N, head->d, head->h,
            static_cast<const __nv_bfloat16*>(head->W1), static_cast<const __nv_bfloat16*>(head->b1),
            static_cast<const __nv_bfloat16*>(head->w2), partial);
        score_mlp_finish_kernel<__nv_bfloat16><<<(N + 255) / 256, 256, 0, s>>>(
            partial, N, h_tiles, static_cast<const __nv_bfloat16*>(head->b2), B, q_lut, score, prob, bin, q);
    }
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}
