// Shared host-side declarations of the library: the context, error handling
// and the launch helpers that the entry points in api.cu use.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <atomic>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

// the library is built with hidden visibility; only the C ABI is exported
#pragma GCC visibility push(default)
#include "../../include/adloco.h"
#pragma GCC visibility pop

namespace adloco {

constexpr int kMaxInstances = 64;     // K of the outer step / merge (pointers travel as kernel arguments)
constexpr int kSchedCounters = 1024;   // launches of the grouped kernel that may be in flight at once
constexpr int64_t kMaxBatchRows = 4096;  // B of one materialised (micro-)batch (per-warp rows live in shared memory)

// Staging buffers for the host-memory entry points (allocated on first use).
struct HostStaging {
    void* dev[2] = {nullptr, nullptr};
    size_t bytes = 0;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t filled[2] = {nullptr, nullptr};
    cudaEvent_t drained[2] = {nullptr, nullptr};
    cudaEvent_t out_done[2] = {nullptr, nullptr};
};

}  // namespace adloco

struct adloco_ctx {
    int device = 0;
    int sm_count = 0;
    int64_t launches = 0;
    char cuda_err[256] = {0};

    // workspace of the streaming reductions
    float* n_partials = nullptr;   // [grid][B] per-block partial row sums of squares
    size_t n_partials_elems = 0;
    double* blk_scalars = nullptr; // [max_grid][4]
    unsigned* ticket = nullptr;    // "last block done" counter, left at zero by every kernel
    int max_grid = 0;
    adloco_test_sums* scratch_sums = nullptr;  // used when the caller passes no sums_dev
    int* gemm_status = nullptr;                // device status word of the tensor-core kernels
    uint64_t wait_limit_ns = 2000000000ull;    // bound of every in-kernel wait: 2 s, far beyond any legitimate wait
    float* n_scratch = nullptr;                // [kMaxBatchRows] per-sample norms when the caller wants none
    void* tensor_maps = nullptr;               // cache of encoded tensor maps (gram_kernels.cu owns the type)
    int pair_ok = -1;                          // CTA-pair launches possible on this device: -1 not asked yet
    int* sched_counters = nullptr;             // [kSchedCounters] work counters of the grouped tensor-core kernel
    std::atomic<unsigned> sched_next{0};       // next counter to hand to a launch

    adloco::HostStaging staging;
};

struct adloco_accum {
    adloco_ctx* ctx = nullptr;
    int32_t n_bufs = 0;
    float** bufs_host = nullptr;       // host copy of the S pointers
    int64_t* sizes_host = nullptr;
    float** bufs_dev = nullptr;        // device copies, for the squared-norm reduction
    int64_t* chunk_prefix_dev = nullptr;  // [n_bufs + 1] prefix sums of 4096-element chunks
    int64_t* sizes_dev = nullptr;
    int64_t total_chunks = 0;
    adloco_test_sums* state = nullptr; // device: Q, ||S||^2, centred ss, count
    bool sqnorm_current = true;        // state->sum_sq_gsum already equals ||S||^2 (kept by the materialised form)
};

namespace adloco {

inline int set_cuda_error(adloco_ctx* ctx, cudaError_t e, const char* where) {
    if (ctx) snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "%s: %s", where, cudaGetErrorString(e));
    return ADLOCO_ERR_CUDA;
}

#define ADLOCO_CUDA_TRY(ctx, expr)                                        \
    do {                                                                  \
        cudaError_t e__ = (expr);                                         \
        if (e__ != cudaSuccess) return adloco::set_cuda_error((ctx), e__, #expr); \
    } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int check_params(const adloco_test_params* p) {
    if (!p) return ADLOCO_ERR_INVALID_ARG;
    if (!(p->eta > 0.0) || !(p->eta < 1.0e300)) return ADLOCO_ERR_INVALID_ARG;  // also rejects NaN
    if (p->ddof < 0 || p->switch_n < 1 || p->b_max < 1 || p->b_cur < 0 || p->b_cap < 0) return ADLOCO_ERR_INVALID_ARG;
    return ADLOCO_OK;
}

// ---- launchers implemented in stream_kernels.cu --------------------------------
enum NtMode { NT_ONESHOT = 0, NT_PANEL = 1, NT_MICRO = 2 };

struct NtLaunch {
    const float* G = nullptr;     // rows of float, or of bfloat16 when bf16 != 0
    int bf16 = 0;
    int64_t B = 0, P = 0, stride = 0;
    float* n_out = nullptr;       // [B], may be null
    int n_accum = 0;              // n_out[i] += instead of =
    float* S = nullptr;           // [P]: written (ONESHOT/PANEL) or read-modify-written (MICRO); may be null unless MICRO
    adloco_test_sums* sums = nullptr;    // required (ctx scratch if the caller has none)
    adloco_test_result* result = nullptr;  // decision written by the last block when non-null
    adloco_test_result* result_mirror = nullptr;  // device-side address of a page-locked host copy of it, or null
    adloco_test_params params{};
    int mode = NT_ONESHOT;
    int first_panel = 1;          // PANEL: overwrite the sums on the first panel, add afterwards
};
int launch_norm_test(adloco_ctx* ctx, const NtLaunch& l, cudaStream_t st);
int launch_decide(adloco_ctx* ctx, const adloco_test_sums* sums, const adloco_test_params& p,
                  adloco_test_result* result, adloco_test_result* mirror, cudaStream_t st);

struct IpLaunch {
    const float* G = nullptr;
    int bf16 = 0;
    const float* S = nullptr;
    int64_t B = 0, P = 0, stride = 0;
    const adloco_test_sums* sums = nullptr;
    adloco_ip_params params{};
    float* dots_out = nullptr;
    adloco_ip_result* result = nullptr;
    adloco_ip_result* result_mirror = nullptr;
};
int launch_inner_product(adloco_ctx* ctx, const IpLaunch& l, cudaStream_t st);

int launch_vec_param(adloco_ctx* ctx, const void* D, const void* X, int64_t B, int64_t T, int64_t d, float* n,
                     int accumulate_norms, float* S, int accumulate_sum, cudaStream_t st);

struct OuterLaunch {
    const void* inst[kMaxInstances];
    void* wb[kMaxInstances];
    int K = 0;
    int has_wb = 0;
    int bf16 = 0;
    int64_t P = 0;
    const float* th_in = nullptr;
    float* th_out = nullptr;
    const float* v_in = nullptr;
    float* v_out = nullptr;
    float lr = 0, mu = 0;
    int nesterov = 1;
};
int launch_outer_step(adloco_ctx* ctx, const OuterLaunch& l, cudaStream_t st);

int launch_pseudo_grad(adloco_ctx* ctx, const float* theta, const void* inst, int bf16, float* g, int64_t P, cudaStream_t st);
int launch_outer_apply(adloco_ctx* ctx, const float* g_sum, int K, int64_t P, const float* th_in, float* th_out,
                       const float* v_in, float* v_out, float lr, float mu, int nesterov, cudaStream_t st);
int launch_refresh(adloco_ctx* ctx, const float* theta, void* inst, int bf16, int64_t P, cudaStream_t st);

struct MergeLaunch {
    const void* x[kMaxInstances];
    float coef[kMaxInstances];
    int K = 0;
    int bf16 = 0;
    int64_t P = 0;
    void* out = nullptr;
};
int launch_merge(adloco_ctx* ctx, const MergeLaunch& l, cudaStream_t st);

// sum over all S buffers of an accumulator of ||S||^2 -> state->sum_sq_gsum, then
// state->sum_sqnorm += sum(n[0..b)) and the count (form (b) of adloco_accumulate)
int launch_accum_add_norms(adloco_ctx* ctx, adloco_accum* acc, const float* n, int64_t b, cudaStream_t st);
int launch_accum_sqnorm(adloco_ctx* ctx, adloco_accum* acc, cudaStream_t st);
int launch_accum_zero(adloco_ctx* ctx, adloco_accum* acc, cudaStream_t st);

// ---- tensor-core path, implemented in gram_kernels.cu ---------------------------
int launch_gram_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                       int64_t d_out, float* n, int accumulate_norms, cudaStream_t st);
int launch_gram_pair(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                     int64_t d_out, float* n, int accumulate_norms, cudaStream_t st);
int launch_mean_grad(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                     int64_t d_out, float* S, int accumulate_sum, cudaStream_t st);
int launch_embedding(adloco_ctx* ctx, const int* ids, const void* D, int64_t B, int64_t T, int64_t d, int64_t V,
                     float* n, int accumulate_norms, float* S, int accumulate_sum, cudaStream_t st);
int launch_direct_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                         int64_t d_out, float* n, int accumulate_norms, float* S, int accumulate_sum, int pair,
                         cudaStream_t st);
int launch_direct_group(adloco_ctx* ctx, const adloco_linear_layer* layers, int n_layers, int64_t B, int64_t T,
                        float* n, int accumulate_norms, int accumulate_sum, int pair, cudaStream_t st);
void free_tensor_map_cache(adloco_ctx* ctx);

}  // namespace adloco
