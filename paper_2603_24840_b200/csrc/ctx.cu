// Context life-cycle, status reporting and the host-side calibration-table helpers.
#include <cmath>
#include <new>

#include "arrol_internal.h"

extern "C" int arrol_version(void) { return 100; }

extern "C" const char* arrol_status_string(int status) {
    switch (status) {
        case ARROL_OK: return "ok";
        case ARROL_ERR_INVALID_ARG: return "invalid argument";
        case ARROL_ERR_UNSUPPORTED: return "unsupported size or configuration";
        case ARROL_ERR_WORKSPACE: return "workspace missing or too small";
        case ARROL_ERR_CAPACITY: return "destination capacity exceeded (detected on the device)";
        case ARROL_ERR_CUDA: return "a CUDA call failed";
        case ARROL_ERR_DEVICE_STATUS: return "device-detected error (bad target id, expired wait, bad state or index)";
        case ARROL_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
        default: return "unknown status";
    }
}

extern "C" int arrol_create(arrol_ctx** out, int device) {
    if (!out) return ARROL_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0) {
        (void)cudaGetLastError();
        return ARROL_ERR_NO_DEVICE;
    }
    if (device < 0 || device >= count) return ARROL_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    ARROL_CUDA_OK(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return ARROL_ERR_NO_DEVICE;  // the kernels are built for sm_100a only
    ArrolDeviceGuard guard(device);
    if (!guard.ok) return ARROL_ERR_CUDA;

    arrol_ctx* ctx = new (std::nothrow) arrol_ctx();
    if (!ctx) return ARROL_ERR_CUDA;
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->d_status = nullptr;
    ctx->h_status = nullptr;
    ctx->d_scratch = nullptr;
    ctx->d_pack = nullptr;
    ctx->d_tile_counters = nullptr;
    ctx->d_chain = nullptr;
    ctx->score_tc_smem_set = false;
    ctx->gather_bulk_smem_set = false;
    ctx->test_spin_limit = 0;
    ctx->test_mute_producer = 0;
    ctx->logprob_pair = 2;
    for (int i = 0; i < 3; ++i) ctx->pair_max_clusters[i] = 0;
    ctx->logprob_splits = 0;
    ctx->logprob_timing = nullptr;
    ctx->logprob_timing_items = 0;
    ctx->encode_tiled = nullptr;
    ctx->launches = 0;
    ctx->copy_stream = nullptr;
    ctx->h_keep = nullptr;
    ctx->h_stage = nullptr;
    ctx->source_rows = 0;
    for (int i = 0; i < ARROL_COPY_EVENTS; ++i) ctx->copy_events[i] = nullptr;
    bool ok = cudaMalloc(&ctx->d_status, 256) == cudaSuccess &&
              cudaMemset(ctx->d_status, 0, 256) == cudaSuccess &&
              cudaMallocHost(&ctx->h_status, 64) == cudaSuccess &&
              cudaMalloc(&ctx->d_scratch, ARROL_SCRATCH_FLOATS * sizeof(float)) == cudaSuccess &&
              cudaMalloc(&ctx->d_pack, ARROL_PACK_BYTES) == cudaSuccess &&
              cudaMalloc(&ctx->d_tile_counters, ARROL_TILE_COUNTERS * sizeof(uint32_t)) == cudaSuccess &&
              cudaMemset(ctx->d_tile_counters, 0, ARROL_TILE_COUNTERS * sizeof(uint32_t)) == cudaSuccess &&
              cudaMalloc(&ctx->d_chain, (2 + 2 * ARROL_CHAIN_BLOCKS) * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMemset(ctx->d_chain, 0, (2 + 2 * ARROL_CHAIN_BLOCKS) * sizeof(unsigned long long)) == cudaSuccess &&
              cudaMallocHost(&ctx->h_keep, ARROL_MAX_HOST_N) == cudaSuccess &&
              cudaMallocHost(&ctx->h_stage, ARROL_STAGE_BYTES) == cudaSuccess &&
              cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; ok && i < ARROL_COPY_EVENTS; ++i)
        ok = cudaEventCreateWithFlags(&ctx->copy_events[i], cudaEventDisableTiming) == cudaSuccess;
    if (ok) {
        cudaDriverEntryPointQueryResult qres;
        void* fn = nullptr;
        ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
             qres == cudaDriverEntryPointSuccess && fn != nullptr;
        ctx->encode_tiled = fn;
    }
    if (!ok) {
        (void)cudaGetLastError();
        arrol_destroy(ctx);
        return ARROL_ERR_CUDA;
    }
    *out = ctx;
    return ARROL_OK;
}

extern "C" int arrol_destroy(arrol_ctx* ctx) {
    if (!ctx) return ARROL_OK;
    ArrolDeviceGuard guard(ctx->device);
    if (ctx->d_status) (void)cudaFree(ctx->d_status);
    if (ctx->h_status) (void)cudaFreeHost(ctx->h_status);
    if (ctx->d_scratch) (void)cudaFree(ctx->d_scratch);
    if (ctx->d_pack) (void)cudaFree(ctx->d_pack);
    if (ctx->d_tile_counters) (void)cudaFree(ctx->d_tile_counters);
    if (ctx->d_chain) (void)cudaFree(ctx->d_chain);
    if (ctx->h_keep) (void)cudaFreeHost(ctx->h_keep);
    if (ctx->h_stage) (void)cudaFreeHost(ctx->h_stage);
    for (int i = 0; i < ARROL_COPY_EVENTS; ++i)
        if (ctx->copy_events[i]) (void)cudaEventDestroy(ctx->copy_events[i]);
    if (ctx->copy_stream) (void)cudaStreamDestroy(ctx->copy_stream);
    delete ctx;
    return ARROL_OK;
}

extern "C" int arrol_set_source_rows(arrol_ctx* ctx, int64_t source_rows) {
    if (!ctx || source_rows < 0) return ARROL_ERR_INVALID_ARG;
    ctx->source_rows = source_rows;
    return ARROL_OK;
}

extern "C" int64_t arrol_launch_count(arrol_ctx* ctx) { return ctx ? (int64_t)ctx->launches : -1; }

extern "C" int arrol_test_hook(arrol_ctx* ctx, int32_t key, int64_t value) {
    if (!ctx) return ARROL_ERR_INVALID_ARG;
    switch (key) {
        case ARROL_HOOK_SPIN_LIMIT:
            if (value < 0 || value > (int64_t)1 << 26) return ARROL_ERR_INVALID_ARG;
            ctx->test_spin_limit = (uint32_t)value;
            return ARROL_OK;
        case ARROL_HOOK_MUTE_LOGPROB_PRODUCER:
            ctx->test_mute_producer = value != 0;
            return ARROL_OK;
        case ARROL_HOOK_LOGPROB_SPLITS:
            if (value < 0 || value > 64) return ARROL_ERR_INVALID_ARG;
            ctx->logprob_splits = (int)value;
            return ARROL_OK;
        case ARROL_HOOK_LOGPROB_PAIR:
            if (value < 0 || value > 2) return ARROL_ERR_INVALID_ARG;
            ctx->logprob_pair = (int)value;
            return ARROL_OK;
        case ARROL_HOOK_LOGPROB_TIMING_BUFFER:
            ctx->logprob_timing = reinterpret_cast<unsigned long long*>((uintptr_t)value);
            if (!value) ctx->logprob_timing_items = 0;
            return ARROL_OK;
        case ARROL_HOOK_LOGPROB_TIMING_ITEMS:
            if (value < 0) return ARROL_ERR_INVALID_ARG;
            ctx->logprob_timing_items = value;
            return ARROL_OK;
        default:
            return ARROL_ERR_INVALID_ARG;
    }
}

extern "C" int arrol_poll_status(arrol_ctx* ctx, void* stream, uint32_t* dev_status_bits) {
    if (!ctx) return ARROL_ERR_INVALID_ARG;
    ArrolDeviceGuard guard(ctx->device);
    if (!guard.ok) return ARROL_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    ARROL_CUDA_OK(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    ARROL_CUDA_OK(cudaMemsetAsync(ctx->d_status, 0, sizeof(uint32_t), s));
    ARROL_CUDA_OK(cudaStreamSynchronize(s));
    uint32_t bits = *ctx->h_status;
    if (dev_status_bits) *dev_status_bits = bits;
    if (bits == 0) return ARROL_OK;
    if (bits & (ARROL_DEV_BAD_TARGET | ARROL_DEV_WAIT_EXPIRED | ARROL_DEV_BAD_STATE | ARROL_DEV_BAD_INDEX))
        return ARROL_ERR_DEVICE_STATUS;
    return ARROL_ERR_CAPACITY;
}

// ---- Binned posterior table (Appendix A.4), host side ----------------------------------------------

extern "C" int arrol_calib_counts(const double* sprime, const uint8_t* y, int64_t n, int B, int64_t* cpos,
                                  int64_t* cneg) {
    if (B <= 0 || n < 0 || !cpos || !cneg || (n > 0 && (!sprime || !y))) return ARROL_ERR_INVALID_ARG;
    for (int b = 0; b < B; ++b) { cpos[b] = 0; cneg[b] = 0; }
    for (int64_t k = 0; k < n; ++k) {
        double scaled = std::floor(sprime[k] * (double)B);
        int b = scaled >= (double)(B - 1) ? B - 1 : (scaled <= 0.0 ? 0 : (int)scaled);
        (y[k] ? cpos : cneg)[b] += 1;
    }
    return ARROL_OK;
}

extern "C" int arrol_build_q_lut(const int64_t* cpos, const int64_t* cneg, int B, double alpha, float* q_lut) {
    if (B <= 0 || !cpos || !cneg || !q_lut || !(alpha >= 0.0)) return ARROL_ERR_INVALID_ARG;
    double n_pos = 0.0, n_neg = 0.0;
    for (int b = 0; b < B; ++b) {
        if (cpos[b] < 0 || cneg[b] < 0) return ARROL_ERR_INVALID_ARG;
        n_pos += (double)cpos[b];
        n_neg += (double)cneg[b];
    }
    const double prior = (n_pos + n_neg) > 0.0 ? n_pos / (n_pos + n_neg) : 0.5;
    const double den_pos = n_pos + alpha * B, den_neg = n_neg + alpha * B;
    for (int b = 0; b < B; ++b) {
        double like_pos = den_pos > 0.0 ? ((double)cpos[b] + alpha) / den_pos : 0.0;
        double like_neg = den_neg > 0.0 ? ((double)cneg[b] + alpha) / den_neg : 0.0;
        double num = prior * like_pos;
        double den = num + (1.0 - prior) * like_neg;
        q_lut[b] = den > 0.0 ? (float)(num / den) : (float)prior;  // an empty bin with alpha = 0 falls back to pi
    }
    return ARROL_OK;
}
