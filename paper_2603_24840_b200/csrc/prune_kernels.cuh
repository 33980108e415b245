// Device functions shared by the kernels of the prune step (score -> select -> scan), so that the separate kernels
// behind arrol_score_partial / arrol_select / arrol_compact and the fused kernel behind arrol_prune_step run the
// same arithmetic in the same order and give bit-identical results.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "arrol_internal.h"
#include "score_common.cuh"

namespace {

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// 16-byte vector of T -> floats
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    using Raw = float4;
    __device__ static __forceinline__ Raw load_raw(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
    __device__ static __forceinline__ float dot(const Raw& a, const Raw& b, float acc) {
        acc = fmaf(a.x, b.x, acc); acc = fmaf(a.y, b.y, acc); acc = fmaf(a.z, b.z, acc); return fmaf(a.w, b.w, acc);
    }
    __device__ static __forceinline__ void load(const float* p, float (&out)[4]) {
        float4 v = __ldg(reinterpret_cast<const float4*>(p));
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    using Raw = uint4;
    __device__ static __forceinline__ Raw load_raw(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
    __device__ static __forceinline__ float dot(const Raw& a, const Raw& b, float acc) {
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {   // a bf16 is the upper half of a binary32
            acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
            acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
        }
        return acc;
    }
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

// Dot product of one hidden row with the linear head's weights by one warp (Section 4.2) with the weights staged in
// shared memory (w_s: the d / VN 16-byte vectors of w): 16-byte loads, eight of the row in flight per lane (a 4 KB row
// is one round trip), four accumulators per lane, shuffle reduction; every lane returns the row's sum (without the
// bias); nvec = d / Vec16<T>::N, or 0 to skip the row (sum 0).  Products and sums are taken in exactly the order of
// score_linear_kernel, which keeps w's vectors in registers beside the row's, so the two give the same bits.
template <typename T>
__device__ __forceinline__ float linear_row_dot_ws(const T* __restrict__ x, const typename Vec16<T>::Raw* w_s, int nvec,
                                                   int lane) {
    constexpr int VN = Vec16<T>::N;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int c0 = lane; c0 < nvec; c0 += 256) {
        typename Vec16<T>::Raw xr[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int c = c0 + 32 * u;
            if (c < nvec) xr[u] = Vec16<T>::load_raw(x + (int64_t)c * VN);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (c0 + 32 * u < nvec) acc[u & 3] = Vec16<T>::dot(xr[u], w_s[c0 + 32 * u], acc[u & 3]);
    }
    float s = (acc[0] + acc[1]) + (acc[2] + acc[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    return s;
}

__device__ __forceinline__ double shfl_double(double v, int src_lane, int width) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_sync(0xffffffffu, lo, src_lane, width);
    hi = __shfl_sync(0xffffffffu, hi, src_lane, width);
    return __hiloint2double(hi, lo);
}

__device__ __forceinline__ double shfl_xor_double(double v, int mask, int width) {
    int lo = __double2loint(v), hi = __double2hiint(v);
    lo = __shfl_xor_sync(0xffffffffu, lo, mask, width);
    hi = __shfl_xor_sync(0xffffffffu, hi, mask, width);
    return __hiloint2double(hi, lo);
}

// Per-group correctness-balancing selection (Section 4.1; Theorem 1's rule j^ = argmin_j |mu_{-j} - rho| applied
// G - K times) for the groups held by one warp: a group occupies a segment of `seg` = next power of two >= G lanes,
// lane j of the segment holds rollout j's q in double (`member` false for padding lanes and groups past the end).
// Each round: tau = Sigma - rho (n - 1) (one rounding per operation, no fused multiply-add), key = |q - tau|, a
// segmented shuffle arg-min on (key, index) where of equal keys the higher index wins, then the winner leaves the
// group and Sigma -= q_winner.  Sigma starts as the index-order sum, built with broadcasts so that every lane of the
// segment adds the same values in the same order.  All 32 lanes must call this.  Returns whether the lane's rollout
// is kept.
__device__ __forceinline__ bool select_lanes(double qj, bool member, int j, int G, int K, double rho, int seg) {
    bool alive = member;
    double sigma = 0.0;
    for (int i = 0; i < G; ++i) sigma = __dadd_rn(sigma, shfl_double(qj, i, seg));
    for (int n = G; n > K; --n) {
        const double tau = __dsub_rn(sigma, __dmul_rn(rho, (double)(n - 1)));
        double key = alive ? fabs(__dsub_rn(qj, tau)) : __longlong_as_double(0x7ff0000000000000LL);
        int idx = alive ? j : -1;
        // segmented arg-min; ties -> the higher index
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            if (o < seg) {
                const double okey = shfl_xor_double(key, o, seg);
                const int oidx = __shfl_xor_sync(0xffffffffu, idx, o, seg);
                if (okey < key || (okey == key && oidx > idx)) { key = okey; idx = oidx; }
            }
        }
        const double q_removed = shfl_double(qj, idx < 0 ? 0 : idx, seg);
        if (idx == j) alive = false;
        sigma = __dsub_rn(sigma, q_removed);
    }
    return alive;
}

// Statistics of one group over its kept rollouts r in [g0, g1) (Section 3, on the survivors): mean and
// 1 / (std + eps) in fp64, sums in index order.  flag(r) / rew(r) give rollout r's keep flag and reward; adding 0.0 for
// a pruned rollout changes nothing.  A double-precision division or square root costs a one-block kernel about half a
// microsecond each, so the reciprocals of the small counts come from the table inv_count[c] = 1 / c (c < SCAN_INV) and
// sqrt / reciprocal are Newton steps from single-precision seeds (relative error below 1e-15 after two steps); values
// outside the single-precision range take the plain operations.  inv_den = 0 (advantage exactly 0) when fewer than
// ddof + 1 rollouts are kept or all kept rewards are equal.
constexpr int SCAN_INV = 65;
template <typename Flag, typename Rew>
__device__ __forceinline__ void group_statistics(int g0, int g1, int ddof, double eps, const double* inv_count, Flag flag,
                                                 Rew rew, double& mean, double& inv_den) {
    int n = 0;
    double sum = 0.0;
    float first = 0.f;
    bool all_equal = true;
#pragma unroll 4
    for (int r = g0; r < g1; ++r) {
        const bool k = flag(r);
        const float v = rew(r);
        if (k && n == 0) first = v;
        all_equal = all_equal && (!k || v == first);
        sum += k ? (double)v : 0.0;
        n += k ? 1 : 0;
    }
    auto recip_count = [&](int c) { return c < SCAN_INV ? inv_count[c] : 1.0 / (double)c; };
    mean = n > 0 ? sum * recip_count(n) : 0.0;
    double ss = 0.0;
#pragma unroll 4
    for (int r = g0; r < g1; ++r) {
        const bool k = flag(r);
        const double dv = (double)rew(r) - mean;
        ss += k ? dv * dv : 0.0;
    }
    inv_den = 0.0;
    if (n - ddof > 0 && !all_equal) {
        const double var = ss * recip_count(n - ddof);
        double sd;
        const float varf = (float)var;
        if (varf > 1e-30f && varf < 1e30f) {
            double y = (double)rsqrtf(varf);
            y = y * (1.5 - 0.5 * var * y * y);
            y = y * (1.5 - 0.5 * var * y * y);
            sd = var * y;
        } else {
            sd = sqrt(var);
        }
        const double den = sd + eps;
        const float denf = (float)den;
        if (denf > 1e-30f && denf < 1e30f) {
            double x = (double)(1.0f / denf);
            x = x * (2.0 - den * x);
            x = x * (2.0 - den * x);
            inv_den = x;
        } else {
            inv_den = 1.0 / den;
        }
    }
}

constexpr int SCAN_THREADS = 1024;
constexpr int SCAN_ITEMS = 4;      // consecutive rollouts per thread and pass: N <= 4096 is one pass
constexpr int SCAN_GROUPS = SCAN_THREADS * SCAN_ITEMS / 4 + 2;   // groups of size >= 4 that one pass can touch

// Survivor scan and advantages of arrol_compact (Section 4.3 (ii); Section 3) by ONE block of SCAN_THREADS threads.
// `keep` may have been written earlier in the same kernel by other blocks (the fused prune step): it is read with
// L2-coherent loads, never through the read-only path.
__device__ __forceinline__ void scan_adv_block(const uint8_t* keep, const int32_t* __restrict__ lengths, int N, int G,
                const float* __restrict__ rewards, double eps, int ddof, int64_t capacity,
                int32_t* __restrict__ survivor_idx, int64_t* __restrict__ cu_seqlens, float* __restrict__ adv,
                int64_t* __restrict__ d_num, uint32_t* __restrict__ d_status,
                const int64_t* __restrict__ src_tok_off, int64_t source_rows) {
    __shared__ int32_t warp_cnt[32];
    __shared__ int64_t warp_tok[32];
    // per-group statistics of the groups a pass touches (G >= 4: at most SCAN_GROUPS of them)
    __shared__ double g_mean[SCAN_GROUPS], g_den[SCAN_GROUPS];     // mean, 1 / (std + eps)
    // the pass's keep flags and rewards, staged once so that the statistics and the advantages read shared memory
    __shared__ float s_rew[SCAN_THREADS * SCAN_ITEMS];
    __shared__ uint8_t s_keep[SCAN_THREADS * SCAN_ITEMS];
    __shared__ double s_inv[SCAN_INV];             // 1 / count for the small counts
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const bool shared_stats = G >= 4;
    if (threadIdx.x == 0) cu_seqlens[0] = 0;
    bool bad_index = false;          // a kept rollout whose source rows leave the caller's buffer (checked on request)
    int32_t carry_c = 0;             // survivors / tokens of the passes so far (the same in every thread)
    int64_t carry_t = 0;

    // statistics over the kept rollouts of a group (Section 3, on survivors): sums in index order, fp64
    constexpr int PASS = SCAN_THREADS * SCAN_ITEMS;
    // Statistics of group g over its kept rollouts: mean and 1 / (std + eps), in fp64.  A double-precision division
    // or square root costs this one-block kernel about half a microsecond each, so the reciprocals of the small
    // counts come from a table and sqrt / reciprocal are Newton steps from single-precision seeds (relative error
    // below 1e-15 after two steps); values outside the single-precision range take the plain operations.
    // inv_den = 0 (advantage exactly 0) when fewer than ddof + 1 rollouts are kept or all kept rewards are equal.
    auto group_stats = [&](int g, int base, double& mean, double& inv_den) {
        const int g0 = g * G;
        const int g1 = min(g0 + G, N);
        // members inside the staged pass come from shared memory, a group that straddles its edge reads the rest
        // from global memory; the loads do not depend on the flags, so they overlap
        auto flag = [&](int r) { return (unsigned)(r - base) < (unsigned)PASS ? s_keep[r - base] != 0 : __ldcg(keep + r) != 0; };
        auto rew = [&](int r) { return (unsigned)(r - base) < (unsigned)PASS ? s_rew[r - base] : rewards[r]; };
        group_statistics(g0, g1, ddof, eps, s_inv, flag, rew, mean, inv_den);
    };

    if (threadIdx.x >= 1 && threadIdx.x < SCAN_INV) s_inv[threadIdx.x] = 1.0 / (double)threadIdx.x;   // before the first barrier below

    for (int base = 0; base < N; base += PASS) {
        const int i0 = base + threadIdx.x * SCAN_ITEMS;
        bool kept[SCAN_ITEMS];
        int64_t len[SCAN_ITEMS];
        int32_t c = 0;
        int64_t t = 0;
        // one round of coalesced loads: flags and rewards of the pass into shared memory, lengths into registers
        for (int e = threadIdx.x; e < PASS; e += SCAN_THREADS) {
            const int i = base + e;
            s_keep[e] = i < N ? __ldcg(keep + i) : (uint8_t)0;
            s_rew[e] = i < N ? rewards[i] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < SCAN_ITEMS; ++u) len[u] = (i0 + u < N) ? (int64_t)max(lengths[i0 + u], 0) : 0;
        __syncthreads();
#pragma unroll
        for (int u = 0; u < SCAN_ITEMS; ++u) {
            kept[u] = s_keep[threadIdx.x * SCAN_ITEMS + u] != 0;
            if (!kept[u]) len[u] = 0;
            else if (source_rows > 0) {
                const int64_t o = src_tok_off[i0 + u];
                bad_index = bad_index || o < 0 || o + len[u] > source_rows;
            }
        }
        const int g_lo = base / G;
        if (shared_stats) {          // one thread per group of this pass; visible after the scan's first barrier
            const int g_hi = (min(N, base + PASS) - 1) / G;
            for (int gi = threadIdx.x; gi <= g_hi - g_lo; gi += SCAN_THREADS)
                group_stats(g_lo + gi, base, g_mean[gi], g_den[gi]);
        }
#pragma unroll
        for (int u = 0; u < SCAN_ITEMS; ++u) { c += kept[u] ? 1 : 0; t += len[u]; }
        const int32_t own_c = c;
        const int64_t own_t = t;
        // inclusive scan of the per-thread totals inside the warp
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t oc = __shfl_up_sync(0xffffffffu, c, o);
            const int64_t ot = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) { c += oc; t += ot; }
        }
        if (lane == 31) { warp_cnt[wid] = c; warp_tok[wid] = t; }
        __syncthreads();
        // every warp scans the 32 warp totals itself (no second barrier, no single-warp phase)
        int32_t wc = warp_cnt[lane];
        int64_t wt = warp_tok[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t oc = __shfl_up_sync(0xffffffffu, wc, o);
            const int64_t ot = __shfl_up_sync(0xffffffffu, wt, o);
            if (lane >= o) { wc += oc; wt += ot; }
        }
        const int32_t pass_cnt = __shfl_sync(0xffffffffu, wc, 31);          // totals of the pass
        const int64_t pass_tok = __shfl_sync(0xffffffffu, wt, 31);
        const int32_t before_c = __shfl_sync(0xffffffffu, wc, wid ? wid - 1 : 0);
        const int64_t before_t = __shfl_sync(0xffffffffu, wt, wid ? wid - 1 : 0);
        int32_t pos = carry_c + (wid ? before_c : 0) + (c - own_c);   // survivors before this thread's items
        int64_t tok = carry_t + (wid ? before_t : 0) + (t - own_t);
#pragma unroll
        for (int u = 0; u < SCAN_ITEMS; ++u) {
            if (!kept[u]) continue;
            const int i = i0 + u;
            tok += len[u];
            survivor_idx[pos] = i;
            cu_seqlens[pos + 1] = tok;
            double mean, den;
            if (shared_stats) { mean = g_mean[i / G - g_lo]; den = g_den[i / G - g_lo]; }
            else group_stats(i / G, base, mean, den);
            const double a = ((double)s_rew[i - base] - mean) * den;      // den holds 1 / (std + eps), or 0
            adv[pos] = (float)a;
            ++pos;
        }
        carry_c += pass_cnt;
        carry_t += pass_tok;
        __syncthreads();                 // the staging arrays and warp totals are rewritten by the next pass
    }
    const int any_bad = __syncthreads_or(bad_index ? 1 : 0);
    if (threadIdx.x == 0) {
        d_num[0] = carry_c;
        d_num[1] = carry_t;
        if (carry_t > capacity) atomicOr(d_status, ARROL_DEV_CAPACITY);
        if (any_bad) atomicOr(d_status, ARROL_DEV_BAD_INDEX);
        d_status[1] = any_bad ? 1u : 0u;       // gate word: the gather kernels of this call copy nothing when it is set
    }
}

}  // namespace
