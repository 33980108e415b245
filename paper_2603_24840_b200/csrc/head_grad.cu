// arrol_head_grad: one training step's gradients for the quality head (Section 4.2: trained on the fly with a
// cross-entropy loss on (score, final reward); Section 4.3 (iii): gradients stop at the head).
//   loss = (1/n) sum_i [log(1 + exp(s_i)) - y_i s_i],  ds_i = (sigmoid(s_i) - y_i) / n  over the masked-in rollouts;
//   linear head:  dw = sum_i ds_i x_i, db = sum_i ds_i
//   MLP head:     dw2_j = sum_i ds_i gelu(u_ij), db2 = sum_i ds_i, du_ij = ds_i w2_j gelu'(u_ij),
//                 dW1 = du^T X, db1_j = sum_i du_ij.
// All reductions run in a fixed order (no atomics), so the gradients are reproducible run to run.
#include <cuda_bf16.h>

#include "arrol_internal.h"

namespace {

constexpr int DS_THREADS = 1024;
constexpr int DU_RUNS = 32;          // row runs of the du kernel on the tensor-core path

__device__ __forceinline__ double block_sum(double v, double* sh /* [32] */) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += sh[w];
    return t;
}

// s_i (given, or assembled from the MLP tile partials), ds_i, loss, sum of ds.  One block.
template <typename T>
__global__ void __launch_bounds__(DS_THREADS)
head_ds_kernel(const float* __restrict__ score, const float* __restrict__ partial, int h_tiles,
               const T* __restrict__ b2_ptr, int N,
               const float* __restrict__ rewards, const uint8_t* __restrict__ mask, float* __restrict__ ds,
               double* __restrict__ loss, float* __restrict__ dbias) {
    __shared__ double sh[32];
    float b2 = 0.f;
    if (b2_ptr) {
        if constexpr (sizeof(T) == 2) b2 = __bfloat162float(b2_ptr[0]); else b2 = b2_ptr[0];
    }
    double cnt = 0.0;
    for (int i = threadIdx.x; i < N; i += DS_THREADS) cnt += (!mask || mask[i]) ? 1.0 : 0.0;
    const double n = block_sum(cnt, sh);
    double l = 0.0, sd = 0.0;
    for (int i = threadIdx.x; i < N; i += DS_THREADS) {
        float v = 0.f;
        if (!mask || mask[i]) {
            float s;
            if (score) s = score[i];
            else {
                s = 0.f;
                for (int t = 0; t < h_tiles; ++t) s += partial[(int64_t)t * N + i];
                s += b2;
            }
            const float y = rewards[i] > 0.5f ? 1.f : 0.f;
            const float softplus = s > 0.f ? s + log1pf(expf(-s)) : log1pf(expf(s));
            l += (double)(softplus - y * s);
            v = (1.0f / (1.0f + expf(-s)) - y) / (float)n;
            sd += (double)v;
        }
        ds[i] = v;
    }
    l = block_sum(l, sh);
    sd = block_sum(sd, sh);
    if (threadIdx.x == 0) {
        *loss = n > 0.0 ? l / n : 0.0;
        *dbias = (float)sd;
    }
}

__device__ __forceinline__ void widen8(const __nv_bfloat16* p, float (&o)[8]) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { o[2 * i] = __uint_as_float(w[i] << 16); o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
__device__ __forceinline__ void widen8(const float* p, float (&o)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
}

// Linear head: partial[c][k] = sum over the rows of row-chunk c of ds_i x_ik.  Thread = 8 consecutive columns.
constexpr int LIN_ROWS = 32;
template <typename T>
__global__ void __launch_bounds__(256)
linear_dw_partial_kernel(const T* __restrict__ hidden, int64_t row_stride, const int64_t* __restrict__ row_index,
                         int N, int d, const float* __restrict__ ds, float* __restrict__ partial) {
    const int k0 = (blockIdx.x * 256 + threadIdx.x) * 8;
    if (k0 >= d) return;
    const int i0 = blockIdx.y * LIN_ROWS, i1 = min(N, i0 + LIN_ROWS);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = i0; i < i1; ++i) {
        const float g = ds[i];
        if (g == 0.f) continue;
        const int64_t row = row_index ? row_index[i] : (int64_t)i;
        float x[8];
        widen8(hidden + row * row_stride + k0, x);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = fmaf(g, x[e], acc[e]);
    }
    float* out = partial + (int64_t)blockIdx.y * d + k0;
#pragma unroll
    for (int e = 0; e < 8; ++e) out[e] = acc[e];
}

__global__ void column_sum_kernel(const float* __restrict__ partial, int chunks, int d, float* __restrict__ out) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= d) return;
    float s = 0.f;
    for (int c = 0; c < chunks; ++c) s += partial[(int64_t)c * d + k];
    out[k] = s;
}

// MLP head: du_ij, and per hidden unit j the sums dw2_j = sum_i ds_i gelu(u_ij), db1_j = sum_i du_ij.
// Block = 32 hidden units x 8 row lanes; rows are walked in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256)
mlp_du_kernel(const float* __restrict__ u, const float* __restrict__ ds, const T* __restrict__ w2, int N, int h,
              float* __restrict__ du, __nv_bfloat16* __restrict__ du_hi, __nv_bfloat16* __restrict__ du_lo,
              float* __restrict__ dw2, float* __restrict__ db1, int rows_per_block) {
    __shared__ float sh_w2[8][33], sh_b1[8][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int j = blockIdx.x * 32 + tx;
    float a_w2 = 0.f, a_b1 = 0.f;
    if (j < h) {
        float wj;
        if constexpr (sizeof(T) == 2) wj = __bfloat162float(w2[j]); else wj = w2[j];
        // blockIdx.y picks a run of rows; its sums go to row blockIdx.y of dw2 / db1 ([gridDim.y][h]), added up in
        // index order by column_sum_kernel when there is more than one run
        const int i_begin = blockIdx.y * rows_per_block, i_end = min(N, i_begin + rows_per_block);
        for (int i = i_begin + ty; i < i_end; i += 8) {
            const float g = ds[i];
            const float a = u[(int64_t)i * h + j];
            const float cdf = 0.5f * (1.0f + erff(a * 0.70710678118654752440f));
            const float pdf = expf(-0.5f * a * a) * 0.39894228040143267794f;
            const float d_u = g * wj * (cdf + a * pdf);
            if (du_hi) {       // du as the sum of two bf16 numbers (error 2^-17 relative): the tensor-core operand
                const __nv_bfloat16 hi = __float2bfloat16_rn(d_u);
                du_hi[(int64_t)i * h + j] = hi;
                du_lo[(int64_t)i * h + j] = __float2bfloat16_rn(d_u - __bfloat162float(hi));
            } else {
                du[(int64_t)i * h + j] = d_u;
            }
            a_w2 = fmaf(g, a * cdf, a_w2);
            a_b1 += d_u;
        }
    }
    sh_w2[ty][tx] = a_w2;
    sh_b1[ty][tx] = a_b1;
    __syncthreads();
    if (ty == 0 && j < h) {
        float s1 = 0.f, s2 = 0.f;
        for (int r = 0; r < 8; ++r) { s1 += sh_w2[r][tx]; s2 += sh_b1[r][tx]; }
        dw2[(int64_t)blockIdx.y * h + j] = s1;
        db1[(int64_t)blockIdx.y * h + j] = s2;
    }
}

// dW1[j][k] = sum_i du[i][j] x[i][k]: 64 x 64 output tile per block, 8 x 4 per thread, rollouts in chunks of 32.
constexpr int GT = 64, GK = 32, GPAD = 4;
template <typename T>
__global__ void __launch_bounds__(128)
mlp_dw1_kernel(const float* __restrict__ du, const T* __restrict__ hidden, int64_t row_stride,
               const int64_t* __restrict__ row_index, int N, int d, int h, float* __restrict__ dW1) {
    __shared__ __align__(16) float as[GK][GT + GPAD];   // du rows
    __shared__ __align__(16) float bs[GK][GT + GPAD];   // x rows
    const int j0 = blockIdx.y * GT, c0 = blockIdx.x * GT;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[8][4];
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
    for (int i0 = 0; i0 < N; i0 += GK) {
        // du tile: 32 rows x 64 floats = 512 float4, 4 per thread
        for (int v = threadIdx.x; v < GK * (GT / 4); v += 128) {
            const int r = v / (GT / 4), c4 = v % (GT / 4);
            float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
            const int i = i0 + r, j = j0 + c4 * 4;
            if (i < N && j < h) val = __ldg(reinterpret_cast<const float4*>(du + (int64_t)i * h + j));   // h % 4 == 0
            *reinterpret_cast<float4*>(&as[r][c4 * 4]) = val;
        }
        // x tile: 32 rows x 64 columns, 8 columns per load
        for (int v = threadIdx.x; v < GK * (GT / 8); v += 128) {
            const int r = v / (GT / 8), c8 = v % (GT / 8);
            float x[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            const int i = i0 + r, k = c0 + c8 * 8;
            if (i < N && k < d) {
                const int64_t row = row_index ? row_index[i] : (int64_t)i;
                widen8(hidden + row * row_stride + k, x);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) bs[r][c8 * 8 + e] = x[e];
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < GK; ++kk) {
            const float4 a0 = *reinterpret_cast<const float4*>(&as[kk][ty * 8]);
            const float4 a1 = *reinterpret_cast<const float4*>(&as[kk][ty * 8 + 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&bs[kk][tx * 4]);
            const float ar[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float br[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(ar[a], br[b], acc[a][b]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        const int j = j0 + ty * 8 + a, k = c0 + tx * 4;
        if (j < h && k < d)     // d % 8 == 0: a float4 never straddles the edge
            *reinterpret_cast<float4*>(dW1 + (int64_t)j * d + k) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
    }
}

struct GradLayout {
    size_t tmp3, ds, u, du, partial, total;   // byte offsets
    size_t du_plane;                          // bytes of one bf16 plane of du (hi at du, lo at du + du_plane)
};
GradLayout grad_layout(int N, int d, int h) {
    GradLayout L;
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    size_t o = 0;
    L.tmp3 = o; o = up(o + sizeof(float) * 3 * (size_t)N);
    L.ds = o; o = up(o + sizeof(float) * (size_t)N);
    L.u = o; o = up(o + sizeof(float) * (size_t)N * (size_t)(h > 0 ? h : 0));
    const size_t plane = up(sizeof(uint16_t) * (size_t)N * (size_t)(h > 0 ? h : 0));   // one bf16 plane of du
    L.du = o; o = up(o + (sizeof(float) * (size_t)N * (size_t)(h > 0 ? h : 0) > 2 * plane
                              ? sizeof(float) * (size_t)N * (size_t)(h > 0 ? h : 0) : 2 * plane));
    L.du_plane = plane;
    const size_t chunks = ((size_t)N + LIN_ROWS - 1) / LIN_ROWS;
    const size_t tiles = (size_t)((h > 0 ? h : 0) + ARROL_MLP_TH - 1) / ARROL_MLP_TH;
    size_t part = h > 0 ? tiles * (size_t)N : chunks * (size_t)d;
    if (h > 0 && part < 2 * (size_t)DU_RUNS * (size_t)h) part = 2 * (size_t)DU_RUNS * (size_t)h;   // dw2 / db1 per row run
    L.partial = o; o = up(o + sizeof(float) * part);
    L.total = o;
    return L;
}

template <typename T>
int run_head_grad(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index, int N,
                  const arrol_head* head, const float* rewards, const uint8_t* mask, float* dW1, float* db1,
                  float* dw2, float* db2, double* loss, uint8_t* ws, const GradLayout& L, cudaStream_t s) {
    const T* hid = static_cast<const T*>(hidden);
    float* ds = reinterpret_cast<float*>(ws + L.ds);
    float* partial = reinterpret_cast<float*>(ws + L.partial);
    const int d = head->d, h = head->h;
    if (h == 0) {
        float* tmp = reinterpret_cast<float*>(ws + L.tmp3);
        const int rc = arrol_score_partial(ctx, hidden, row_stride, row_index, N, head, nullptr, tmp, tmp + N, nullptr,
                                           tmp + 2 * (size_t)N, s);
        if (rc != ARROL_OK) return rc;
        head_ds_kernel<T><<<1, DS_THREADS, 0, s>>>(tmp, nullptr, 0, nullptr, N, rewards, mask, ds, loss, db1);
        const int chunks = (N + LIN_ROWS - 1) / LIN_ROWS;
        dim3 grid((d / 8 + 255) / 256, chunks);
        linear_dw_partial_kernel<T><<<grid, 256, 0, s>>>(hid, row_stride, row_index, N, d, ds, partial);
        column_sum_kernel<<<(d + 255) / 256, 256, 0, s>>>(partial, chunks, d, dW1);
        ctx->launches += 3;
    } else {
        float* u = reinterpret_cast<float*>(ws + L.u);
        float* du = reinterpret_cast<float*>(ws + L.du);
        if constexpr (sizeof(T) == 2) {
            // bf16 head: both contractions on the tensor cores.  Forward with the pre-activations kept, du split into
            // two bf16 planes, dW1 = du_hi^T X + du_lo^T X with X the packed rows (or the rows in place).
            if (h % 8 == 0) {
                float* tmp = reinterpret_cast<float*>(ws + L.tmp3);
                const int rc = arrol_internal_score_mlp_tc(ctx, hidden, row_stride, row_index, N, head, 0, nullptr, tmp,
                                                           tmp + N, nullptr, tmp + 2 * (size_t)N, u, s);
                if (rc == ARROL_OK) {
                    __nv_bfloat16* du_hi = reinterpret_cast<__nv_bfloat16*>(ws + L.du);
                    __nv_bfloat16* du_lo = reinterpret_cast<__nv_bfloat16*>(ws + L.du + L.du_plane);
                    head_ds_kernel<T><<<1, DS_THREADS, 0, s>>>(tmp, nullptr, 0, nullptr, N, rewards, mask, ds, loss, db2);
                    // the tile partials are consumed by now: the region holds the per-run sums of dw2 and db1
                    const int rows_per = ((N + DU_RUNS - 1) / DU_RUNS + 7) / 8 * 8;
                    const int runs = (N + rows_per - 1) / rows_per;
                    float* dw2_runs = partial;
                    float* db1_runs = partial + (size_t)DU_RUNS * h;
                    mlp_du_kernel<T><<<dim3((h + 31) / 32, runs), 256, 0, s>>>(u, ds, static_cast<const T*>(head->w2), N, h,
                                                                               nullptr, du_hi, du_lo, dw2_runs, db1_runs,
                                                                               rows_per);
                    column_sum_kernel<<<(h + 255) / 256, 256, 0, s>>>(dw2_runs, runs, h, dw2);
                    column_sum_kernel<<<(h + 255) / 256, 256, 0, s>>>(db1_runs, runs, h, db1);
                    ctx->launches += 4;
                    ARROL_CUDA_OK(cudaGetLastError());
                    const void* x = row_index ? ctx->d_pack : hidden;
                    const int64_t ldx = row_index ? d : row_stride;
                    int rg = arrol_internal_gemm_tn(ctx, du_hi, h, x, ldx, h, d, N, dW1, d, 0, s);
                    if (rg == ARROL_OK) rg = arrol_internal_gemm_tn(ctx, du_lo, h, x, ldx, h, d, N, dW1, d, 1, s);
                    return rg;
                }
                if (rc != ARROL_ERR_UNSUPPORTED) return rc;
            }
        }
        const int rc = arrol_internal_mlp_tiles(ctx, hidden, row_stride, row_index, N, head, partial, u, s);
        if (rc != ARROL_OK) return rc;
        const int h_tiles = (h + ARROL_MLP_TH - 1) / ARROL_MLP_TH;
        head_ds_kernel<T><<<1, DS_THREADS, 0, s>>>(nullptr, partial, h_tiles, static_cast<const T*>(head->b2), N,
                                                   rewards, mask, ds, loss, db2);
        mlp_du_kernel<T><<<(h + 31) / 32, 256, 0, s>>>(u, ds, static_cast<const T*>(head->w2), N, h, du, nullptr,
                                                       nullptr, dw2, db1, N);
        dim3 grid((d + GT - 1) / GT, (h + GT - 1) / GT);
        mlp_dw1_kernel<T><<<grid, 128, 0, s>>>(du, hid, row_stride, row_index, N, d, h, dW1);
        ctx->launches += 3;
    }
    ARROL_CUDA_OK(cudaGetLastError());
    return ARROL_OK;
}

}  // namespace

extern "C" size_t arrol_head_grad_workspace(arrol_ctx* ctx, int32_t N, int32_t d, int32_t h) {
    if (!ctx || N <= 0 || d <= 0 || h < 0) return 0;
    return grad_layout(N, d, h).total;
}

extern "C" int arrol_head_grad(arrol_ctx* ctx, const void* hidden, int64_t row_stride_elems, const int64_t* row_index,
                               int32_t N, const arrol_head* head, const float* rewards, const uint8_t* mask,
                               float* dW1, float* db1, float* dw2, float* db2, double* loss, void* workspace,
                               size_t workspace_bytes, void* stream) {
    if (!ctx || !head || N < 0) return ARROL_ERR_INVALID_ARG;
    if (!loss || !dW1 || !db1) return ARROL_ERR_INVALID_ARG;
    if (head->h > 0 && (!dw2 || !db2 || !head->w2)) return ARROL_ERR_INVALID_ARG;
    if (head->dtype != ARROL_F32 && head->dtype != ARROL_BF16) return ARROL_ERR_INVALID_ARG;
    if (head->d <= 0 || head->h < 0 || !head->W1) return ARROL_ERR_INVALID_ARG;
    if (head->d % 8 != 0 || head->h % 4 != 0 || head->h > ARROL_MAX_H) return ARROL_ERR_UNSUPPORTED;
    if (N > ARROL_MAX_MLP_N) return ARROL_ERR_UNSUPPORTED;
    if (N > 0 && (!hidden || !rewards)) return ARROL_ERR_INVALID_ARG;
    const int esz = head->dtype == ARROL_F32 ? 4 : 2;
    if (N > 0 && (row_stride_elems < head->d || (row_stride_elems * esz) % 16 != 0 || !arrol_aligned(hidden, 16)))
        return ARROL_ERR_INVALID_ARG;
    if (!arrol_aligned(dW1, 16)) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (N == 0) {   // nothing to learn from: zero loss and gradients
        const size_t hh = head->h > 0 ? (size_t)head->h : 1;
        ARROL_CUDA_OK(cudaMemsetAsync(loss, 0, sizeof(double), s));
        ARROL_CUDA_OK(cudaMemsetAsync(dW1, 0, sizeof(float) * hh * head->d, s));
        ARROL_CUDA_OK(cudaMemsetAsync(db1, 0, sizeof(float) * hh, s));
        if (head->h > 0) {
            ARROL_CUDA_OK(cudaMemsetAsync(dw2, 0, sizeof(float) * hh, s));
            ARROL_CUDA_OK(cudaMemsetAsync(db2, 0, sizeof(float), s));
        }
        return ARROL_OK;
    }
    const GradLayout L = grad_layout(N, head->d, head->h);
    if (!workspace || workspace_bytes < L.total || !arrol_aligned(workspace, 256)) return ARROL_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    if (head->dtype == ARROL_F32)
        return run_head_grad<float>(ctx, hidden, row_stride_elems, row_index, N, head, rewards, mask, dW1, db1, dw2,
                                    db2, loss, ws, L, s);
    return run_head_grad<__nv_bfloat16>(ctx, hidden, row_stride_elems, row_index, N, head, rewards, mask, dW1, db1,
                                        dw2, db2, loss, ws, L, s);
}
