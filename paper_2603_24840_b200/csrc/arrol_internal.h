// Internal declarations shared by the library's translation units (not part of the public ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "arrol.h"

constexpr int ARROL_COPY_EVENTS = 64;
constexpr int ARROL_MAX_HOST_N = 1 << 20;   // rollouts per arrol_prune_rebatch_host call
constexpr size_t ARROL_STAGE_BYTES = (size_t)64 << 20;

struct arrol_ctx {
    int device;
    int sm_count;
    uint32_t* d_status;        // device status word (bits ARROL_DEV_*)
    uint32_t* h_status;        // pinned host mirror used by arrol_poll_status
    float* d_scratch;          // MLP-head partial sums: [ARROL_SCRATCH_FLOATS]
    void* d_pack;              // MLP head on the tensor cores: the scored rows packed as bf16 [N][d], ARROL_PACK_BYTES
    uint32_t* d_tile_counters; // MLP head on the tensor cores: finished blocks per row tile, zero between calls
    unsigned long long* d_chain;   // fused prune step: finished blocks, index-check flag, per-block totals; zero between calls
    bool score_tc_smem_set;    // the scoring kernel's dynamic shared-memory limit has been raised on this device
    bool gather_bulk_smem_set; // likewise for the bulk-copy gather kernel
    uint32_t test_spin_limit;  // arrol_test_hook: tries per pipeline wait of the log-prob kernel, 0 = the normal limit
    unsigned long long* logprob_timing;   // arrol_test_hook: device buffer for per-work-item time stamps of the log-prob kernel
    int64_t logprob_timing_items;         // its capacity in work items (4 words each)
    int logprob_splits;        // arrol_test_hook: vocabulary splits of the log-prob kernel, 0 = chosen from the sizes
    int logprob_pair;          // form of the log-prob kernel: 2 = pairs of blocks (cta_group::2) where they need no more splits (default), 1 = pairs, 0 = single blocks
    int pair_max_clusters[3];  // pairs of that kernel that are resident at once (plain, with confidence, rows in place); 0 = not asked yet
    int test_mute_producer;    // arrol_test_hook: the log-prob kernel's producer issues no copies (its waits run out)
    void* encode_tiled;        // cuTensorMapEncodeTiled, resolved once through the runtime
    unsigned long long launches;   // kernels launched through this context (host-side count)
    cudaStream_t copy_stream;      // second stream of the host-buffer step: uploads overlap the log-prob kernel
    cudaEvent_t copy_events[ARROL_COPY_EVENTS];
    uint8_t* h_keep;               // pinned, ARROL_MAX_HOST_N bytes: the keep mask read back by the host-buffer step
    int64_t source_rows;           // arrol_set_source_rows: rows of the caller's source buffers, 0 = indices unchecked
    uint8_t* h_stage;              // pinned, ARROL_STAGE_BYTES: the scored rows of the host-buffer step, packed for one copy
};

constexpr int ARROL_MAX_MLP_N = 65536;       // rollouts per arrol_score_partial call with an MLP head
constexpr int ARROL_MLP_TH = 64;             // hidden units per MLP thread-block tile
constexpr int ARROL_MAX_H = 4096;
constexpr size_t ARROL_SCRATCH_FLOATS = (size_t)ARROL_MAX_MLP_N * (ARROL_MAX_H / ARROL_MLP_TH);
constexpr size_t ARROL_PACK_BYTES = (size_t)64 << 20;
constexpr int ARROL_TILE_COUNTERS = 1024;   // [0, 1020) row tiles of the MLP head, [1023] log-prob waves
constexpr int ARROL_SCORE_ROW_TILES = 1020;
constexpr int ARROL_CHAIN_BLOCKS = 510;      // blocks of the fused prune step's chained scan (2 + 2 * 510 words = 8 KB)

#define ARROL_CUDA_OK(expr)                      \
    do {                                         \
        cudaError_t e__ = (expr);                \
        if (e__ != cudaSuccess) {                \
            (void)cudaGetLastError();            \
            return ARROL_ERR_CUDA;               \
        }                                        \
    } while (0)

static inline bool arrol_aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

// Device guard: makes the context's device current for the duration of a call.
struct ArrolDeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit ArrolDeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        cur = dev;
    }
    ~ArrolDeviceGuard() {
        if (prev >= 0 && prev != cur) (void)cudaSetDevice(prev);
    }
    int cur = -1;
};

#ifdef __CUDACC__
// Programmatic dependent launch for the short kernels of the prune step (score -> select -> scan -> gather), which
// run back to back on one stream and last a few microseconds each: a kernel launched with arrol_launch_pdl may
// start while its predecessor is still running, sets up (shared memory, barriers, tensor-map prefetch) and then
// blocks in pdl_wait() until the predecessor has completed and its writes are visible.  Every such kernel calls
// pdl_launch_dependents() at its top and touches global memory only after pdl_wait(), through pointers passed
// through pdl_acquire().
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// A kernel that may start before its predecessor has finished must not load the predecessor's results early.  The
// compiler is free to hoist loads through `const __restrict__` pointers (read-only data by contract) above the wait,
// so every pointer to data an earlier kernel may have written is passed through this after pdl_wait(): the loads
// then depend on a value produced after the wait.
template <typename T>
__device__ __forceinline__ T* pdl_acquire(T* p) {
    asm volatile("" : "+l"(p) :: "memory");
    return p;
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t arrol_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                             Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Argument checks of the three prune-step calls (score.cu, select.cu, compact.cu) and arrol_compact with the scan
// kernel left out (the fused prune step has produced its outputs already).
int arrol_internal_check_score(const void* hidden, int64_t row_stride_elems, int32_t N, const arrol_head* head,
                               const arrol_calib* calib, const float* score, const float* prob, const float* q);
int arrol_internal_check_select(const float* q, int32_t P, int32_t G, int32_t K, double rho, int32_t mode,
                                const uint8_t* keep);
int arrol_internal_compact(arrol_ctx* ctx, const uint8_t* keep, const int32_t* lengths, const int64_t* src_tok_off,
                           int32_t N, int32_t G, const int32_t* src_tokens, const void* src_rows, int32_t row_bytes,
                           const float* rewards, float eps, int32_t ddof, int64_t dst_capacity_tokens,
                           int32_t* dst_tokens, void* dst_rows, int64_t* cu_seqlens, int32_t* survivor_idx, float* adv,
                           float* tok_adv, int32_t* tok_seq, int64_t* d_num, void* stream, bool scan_done);
int arrol_internal_check_compact(const uint8_t* keep, const int32_t* lengths, const int64_t* src_tok_off, int32_t N,
                                 int32_t G, const int32_t* src_tokens, const void* src_rows, int32_t row_bytes,
                                 const float* rewards, float eps, int32_t ddof, int64_t dst_capacity_tokens,
                                 const int32_t* dst_tokens, const void* dst_rows, const int64_t* cu_seqlens,
                                 const int32_t* survivor_idx, const float* adv, const int64_t* d_num);

// score.cu: MLP tile pass with optional pre-activation output; partial is [ceil(h / ARROL_MLP_TH)][N].
int arrol_internal_mlp_tiles(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index, int N,
                             const arrol_head* head, float* partial, float* u_out, cudaStream_t s);

// score_tc.cu: scores of a bf16 MLP head on the tensor cores (pack, contraction, GELU, w2 dot, probability map).
// ARROL_ERR_UNSUPPORTED (nothing launched) when the sizes do not fit the context's buffers.
int arrol_internal_score_mlp_tc(arrol_ctx* ctx, const void* hidden, int64_t row_stride, const int64_t* row_index,
                                int N, const arrol_head* head, int B, const float* q_lut, float* score, float* prob,
                                int32_t* bin, float* q, float* u_out /* [N][h] pre-activations, or NULL */,
                                cudaStream_t s);

// gather_bulk.cu: the survivors' rows moved by bulk copies through shared memory.  ARROL_ERR_UNSUPPORTED (nothing
// launched) when a row does not fit a 32 KB stage.
int arrol_internal_gather_rows_bulk(arrol_ctx* ctx, const int64_t* d_num, const int64_t* cu_seqlens,
                                    const int32_t* survivor_idx, const int64_t* src_tok_off, const void* src_rows,
                                    int64_t row_bytes, int64_t capacity, void* dst_rows, cudaStream_t s);

// lm_head_backward.cu: C[M,N] (+)= A^T B on the tensor cores, A stored [K, M] and B stored [K, N] row-major bf16
// (rows lda / ldb elements apart, multiples of 8), C fp32 with rows ldc apart.  Rows past K read as zero.
int arrol_internal_gemm_tn(arrol_ctx* ctx, const void* A, int64_t lda, const void* B, int64_t ldb, int M, int N, int K,
                           float* C, int64_t ldc, int accumulate, cudaStream_t s);
