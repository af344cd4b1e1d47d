// C ABI of the library: argument validation, context and accumulator life
// cycle, and dispatch to the kernels.  Nothing here computes on the host.
#include <algorithm>
#include <new>
#include <vector>

#include "common.cuh"

using namespace adloco;

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int ensure_staging(adloco_ctx* ctx, size_t bytes_each) {
    HostStaging& s = ctx->staging;
    if (!s.copy_stream) {
        ADLOCO_CUDA_TRY(ctx, cudaStreamCreateWithFlags(&s.copy_stream, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            ADLOCO_CUDA_TRY(ctx, cudaEventCreateWithFlags(&s.filled[i], cudaEventDisableTiming));
            ADLOCO_CUDA_TRY(ctx, cudaEventCreateWithFlags(&s.drained[i], cudaEventDisableTiming));
            ADLOCO_CUDA_TRY(ctx, cudaEventCreateWithFlags(&s.out_done[i], cudaEventDisableTiming));
        }
    }
    if (bytes_each > s.bytes) {
        for (int i = 0; i < 2; ++i) {
            if (s.dev[i]) ADLOCO_CUDA_TRY(ctx, cudaFree(s.dev[i]));
            s.dev[i] = nullptr;
        }
        s.bytes = 0;
        for (int i = 0; i < 2; ++i) ADLOCO_CUDA_TRY(ctx, cudaMalloc(&s.dev[i], bytes_each));
        s.bytes = bytes_each;
    }
    return ADLOCO_OK;
}

constexpr size_t kPanelBytes = 64u << 20;  // staging panel of the host-memory entry points

// The device-side address of a caller's host buffer when the GPU can store to it directly (page-locked
// memory under unified addressing), else null: a result struct then goes there from the deciding thread
// itself and the stream is spared a device-to-host copy between two kernels.  Pageable memory gets the copy.
static void* device_address_of_pinned(void* host) {
    if (!host) return nullptr;
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        cudaGetLastError();
        return nullptr;
    }
    return at.type == cudaMemoryTypeHost ? at.devicePointer : nullptr;
}

// thread-block clusters of two CTAs need compute capability 9.0 or later and the launch attribute
bool pair_launch_ok(adloco_ctx* ctx) {
    if (ctx->pair_ok < 0) {
        int v = 0;
        ctx->pair_ok = (cudaDeviceGetAttribute(&v, cudaDevAttrClusterLaunch, ctx->device) == cudaSuccess && v != 0) ? 1 : 0;
    }
    return ctx->pair_ok == 1;
}

}  // namespace

extern "C" {

const char* adloco_status_string(int status) {
    switch (status) {
        case ADLOCO_OK: return "ok";
        case ADLOCO_ERR_INVALID_ARG: return "invalid argument";
        case ADLOCO_ERR_UNSUPPORTED: return "unsupported shape or type";
        case ADLOCO_ERR_ALIGNMENT: return "pointer or pitch not 16-byte aligned";
        case ADLOCO_ERR_CUDA: return "CUDA error";
        case ADLOCO_ERR_WORKSPACE: return "workspace error";
        case ADLOCO_ERR_TIMEOUT: return "bounded wait ran out on the device";
        default: return "unknown status";
    }
}

const char* adloco_last_cuda_error(const adloco_ctx* ctx) { return ctx ? ctx->cuda_err : ""; }
int64_t adloco_launch_count(const adloco_ctx* ctx) { return ctx ? ctx->launches : 0; }

int adloco_create(adloco_ctx** out, int device) {
    if (!out) return ADLOCO_ERR_INVALID_ARG;
    *out = nullptr;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return ADLOCO_ERR_CUDA;
    adloco_ctx* ctx = new (std::nothrow) adloco_ctx();
    if (!ctx) return ADLOCO_ERR_WORKSPACE;
    ctx->device = device;
    DeviceGuard g(device);
    cudaDeviceProp prop;
    cudaError_t e = g.ok ? cudaGetDeviceProperties(&prop, device) : cudaErrorInvalidDevice;
    if (e != cudaSuccess) { delete ctx; return ADLOCO_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_grid = ctx->sm_count * 8;
    bool ok = true;
    ok = ok && cudaMalloc(&ctx->blk_scalars, (size_t)ctx->max_grid * 4 * sizeof(double)) == cudaSuccess;
    // per-block partial row sums for the largest launch: at most 4 resident blocks per SM, kMaxBatchRows rows
    ctx->n_partials_elems = (size_t)ctx->sm_count * 4 * (size_t)kMaxBatchRows;
    ok = ok && cudaMalloc(&ctx->n_partials, ctx->n_partials_elems * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->ticket, 64) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->scratch_sums, sizeof(adloco_test_sums)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->gemm_status, 64) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->n_scratch, kMaxBatchRows * sizeof(float)) == cudaSuccess;
    ok = ok && cudaMalloc(&ctx->sched_counters, kSchedCounters * sizeof(int)) == cudaSuccess;
    ok = ok && cudaMemset(ctx->ticket, 0, 64) == cudaSuccess;
    ok = ok && cudaMemset(ctx->gemm_status, 0, 64) == cudaSuccess;
    ok = ok && cudaMemset(ctx->scratch_sums, 0, sizeof(adloco_test_sums)) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) { adloco_destroy(ctx); return ADLOCO_ERR_CUDA; }
    *out = ctx;
    return ADLOCO_OK;
}

int adloco_destroy(adloco_ctx* ctx) {
    if (!ctx) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaFree(ctx->n_partials);
    cudaFree(ctx->blk_scalars);
    cudaFree(ctx->ticket);
    cudaFree(ctx->scratch_sums);
    cudaFree(ctx->gemm_status);
    cudaFree(ctx->n_scratch);
    cudaFree(ctx->sched_counters);
    free_tensor_map_cache(ctx);
    HostStaging& s = ctx->staging;
    for (int i = 0; i < 2; ++i) {
        cudaFree(s.dev[i]);
        if (s.filled[i]) cudaEventDestroy(s.filled[i]);
        if (s.drained[i]) cudaEventDestroy(s.drained[i]);
        if (s.out_done[i]) cudaEventDestroy(s.out_done[i]);
    }
    if (s.copy_stream) cudaStreamDestroy(s.copy_stream);
    delete ctx;
    return ADLOCO_OK;
}

int adloco_set_wait_limit(adloco_ctx* ctx, uint64_t limit_ns) {
    if (!ctx) return ADLOCO_ERR_INVALID_ARG;
    ctx->wait_limit_ns = limit_ns;
    return ADLOCO_OK;
}

int adloco_device_status(adloco_ctx* ctx, int32_t* status_host, int clear, void* stream) {
    if (!ctx || !status_host) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int v = 0;
    ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(&v, ctx->gemm_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    if (clear) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(ctx->gemm_status, 0, sizeof(int), st));
    ADLOCO_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    *status_host = v;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// norm test
// ---------------------------------------------------------------------------------
static int check_grads(const void* grads, adloco_dtype dtype, int64_t B, int64_t P, int64_t row_stride) {
    if (!grads || B < 1 || P < 1 || row_stride < P) return ADLOCO_ERR_INVALID_ARG;
    if (dtype != ADLOCO_F32 && dtype != ADLOCO_BF16) return ADLOCO_ERR_UNSUPPORTED;
    if (B > kMaxBatchRows) return ADLOCO_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(grads) & (dtype == ADLOCO_BF16 ? 1u : 3u)) != 0) return ADLOCO_ERR_ALIGNMENT;
    return ADLOCO_OK;
}

int adloco_norm_test(adloco_ctx* ctx, const void* grads, adloco_dtype dtype, int64_t B, int64_t P,
                     int64_t row_stride, const adloco_test_params* params, float* per_sample_sqnorm,
                     float* grad_sum, adloco_test_sums* sums_dev, adloco_test_result* result_dev,
                     adloco_test_result* result_host, void* stream) {
    if (!ctx || !result_dev) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_params(params);
    if (rc != ADLOCO_OK) return rc;
    rc = check_grads(grads, dtype, B, P, row_stride);
    if (rc != ADLOCO_OK) return rc;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    NtLaunch l;
    l.G = static_cast<const float*>(grads);
    l.bf16 = (dtype == ADLOCO_BF16);
    l.B = B; l.P = P; l.stride = row_stride;
    l.n_out = per_sample_sqnorm; l.S = grad_sum;
    l.sums = sums_dev ? sums_dev : ctx->scratch_sums;
    l.result = result_dev; l.params = *params; l.mode = NT_ONESHOT;
    l.result_mirror = static_cast<adloco_test_result*>(device_address_of_pinned(result_host));
    rc = launch_norm_test(ctx, l, st);
    if (rc != ADLOCO_OK) return rc;
    if (result_host && !l.result_mirror)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(result_host, result_dev, sizeof(adloco_test_result), cudaMemcpyDeviceToHost, st));
    return ADLOCO_OK;
}

int adloco_test_decide(adloco_ctx* ctx, const adloco_test_sums* sums_dev, const adloco_test_params* params,
                       adloco_test_result* result_dev, adloco_test_result* result_host, void* stream) {
    if (!ctx || !sums_dev || !result_dev) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_params(params);
    if (rc != ADLOCO_OK) return rc;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    adloco_test_result* mirror = static_cast<adloco_test_result*>(device_address_of_pinned(result_host));
    rc = launch_decide(ctx, sums_dev, *params, result_dev, mirror, st);
    if (rc != ADLOCO_OK) return rc;
    if (result_host && !mirror)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(result_host, result_dev, sizeof(adloco_test_result), cudaMemcpyDeviceToHost, st));
    return ADLOCO_OK;
}

int adloco_norm_test_host(adloco_ctx* ctx, const float* grads_host, int64_t B, int64_t P, int64_t row_stride,
                          const adloco_test_params* params, float* per_sample_sqnorm_host,
                          adloco_test_result* result_host, void* stream) {
    if (!ctx || !result_host) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_params(params);
    if (rc != ADLOCO_OK) return rc;
    if (!grads_host || B < 1 || P < 1 || row_stride < P) return ADLOCO_ERR_INVALID_ARG;
    if (B > kMaxBatchRows) return ADLOCO_ERR_UNSUPPORTED;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // column panels of width w (a multiple of 1024), about kPanelBytes each
    int64_t w = (int64_t)(kPanelBytes / sizeof(float)) / B;
    w = std::max<int64_t>(1024, (w / 1024) * 1024);
    if (w > P) w = ((P + 3) / 4) * 4;
    const size_t panel_bytes = (size_t)B * (size_t)w * sizeof(float);
    const size_t tail = 256 + sizeof(adloco_test_sums) + sizeof(adloco_test_result);
    rc = ensure_staging(ctx, panel_bytes + tail);
    if (rc != ADLOCO_OK) return rc;
    HostStaging& s = ctx->staging;
    // result and sums live behind the first panel buffer
    char* tail0 = static_cast<char*>(s.dev[0]) + ((panel_bytes + 255) / 256) * 256;
    adloco_test_sums* sums = reinterpret_cast<adloco_test_sums*>(tail0);
    adloco_test_result* result = reinterpret_cast<adloco_test_result*>(tail0 + sizeof(adloco_test_sums));

    const int64_t npanels = (P + w - 1) / w;
    // the caller's stream must be done with the staging buffers' previous use
    ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.drained[0], st));
    ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.drained[1], st));
    for (int64_t p = 0; p < npanels; ++p) {
        const int b = (int)(p & 1);
        const int64_t col0 = p * w;
        const int64_t wp = std::min<int64_t>(w, P - col0);
        ADLOCO_CUDA_TRY(ctx, cudaStreamWaitEvent(s.copy_stream, s.drained[b], 0));
        ADLOCO_CUDA_TRY(ctx, cudaMemcpy2DAsync(s.dev[b], (size_t)w * sizeof(float), grads_host + col0,
                                               (size_t)row_stride * sizeof(float), (size_t)wp * sizeof(float),
                                               (size_t)B, cudaMemcpyHostToDevice, s.copy_stream));
        ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.filled[b], s.copy_stream));
        ADLOCO_CUDA_TRY(ctx, cudaStreamWaitEvent(st, s.filled[b], 0));
        NtLaunch l;
        l.G = static_cast<const float*>(s.dev[b]);
        l.B = B; l.P = wp; l.stride = w;
        l.n_out = ctx->n_scratch; l.n_accum = (p > 0);
        l.sums = sums; l.params = *params; l.mode = NT_PANEL; l.first_panel = (p == 0);
        l.result = (p == npanels - 1) ? result : nullptr;
        rc = launch_norm_test(ctx, l, st);
        if (rc != ADLOCO_OK) return rc;
        ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.drained[b], st));
    }
    ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(result_host, result, sizeof(adloco_test_result), cudaMemcpyDeviceToHost, st));
    if (per_sample_sqnorm_host)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(per_sample_sqnorm_host, ctx->n_scratch, (size_t)B * sizeof(float),
                                             cudaMemcpyDeviceToHost, st));
    ADLOCO_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    return ADLOCO_OK;
}

int adloco_inner_product_test(adloco_ctx* ctx, const void* grads, adloco_dtype dtype, int64_t B, int64_t P,
                              int64_t row_stride, const adloco_ip_params* params, const float* grad_sum,
                              const adloco_test_sums* sums_dev, float* inner_products,
                              adloco_ip_result* result_dev, adloco_ip_result* result_host, void* stream) {
    if (!ctx || !params || !grad_sum || !sums_dev || !result_dev) return ADLOCO_ERR_INVALID_ARG;
    if (!(params->theta > 0.0) || !(params->theta < 1.0e300) || !(params->nu > 0.0) || !(params->nu < 1.0e300))
        return ADLOCO_ERR_INVALID_ARG;
    if (params->ddof < 0 || params->b_cur < 0 || params->b_cap < 0) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_grads(grads, dtype, B, P, row_stride);
    if (rc != ADLOCO_OK) return rc;
    if ((reinterpret_cast<uintptr_t>(grad_sum) & 3u) != 0) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    IpLaunch l;
    l.G = static_cast<const float*>(grads);
    l.bf16 = (dtype == ADLOCO_BF16);
    l.S = grad_sum; l.B = B; l.P = P; l.stride = row_stride; l.sums = sums_dev; l.params = *params;
    l.dots_out = inner_products; l.result = result_dev;
    l.result_mirror = static_cast<adloco_ip_result*>(device_address_of_pinned(result_host));
    rc = launch_inner_product(ctx, l, st);
    if (rc != ADLOCO_OK) return rc;
    if (result_host && !l.result_mirror)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(result_host, result_dev, sizeof(adloco_ip_result), cudaMemcpyDeviceToHost, st));
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// Gram path
// ---------------------------------------------------------------------------------
// variant: 0 = the one-CTA Gram kernel, 1 = the CTA-pair Gram kernel, -1 = whichever suits the shape
static int gram_route(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                      int64_t d_out, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                      int accumulate_sum, int variant, void* stream) {
    if (!ctx || !X || !D || !per_sample_sqnorm) return ADLOCO_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d_in < 1 || d_out < 1) return ADLOCO_ERR_INVALID_ARG;
    if ((d_in % 8) != 0 || (d_out % 8) != 0) return ADLOCO_ERR_UNSUPPORTED;
    if (B > (1 << 30) || T > (1 << 30) || d_in > (1 << 30) || d_out > (1 << 30)) return ADLOCO_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(D)) return ADLOCO_ERR_ALIGNMENT;
    if (grad_sum && !aligned16(grad_sum)) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (variant == 1 && !pair_launch_ok(ctx)) return ADLOCO_ERR_UNSUPPORTED;
    if (variant < 0) variant = 0;
    int rc = variant == 1 ? launch_gram_pair(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, st)
                          : launch_gram_sqnorm(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, st);
    if (rc != ADLOCO_OK) return rc;
    if (grad_sum) rc = launch_mean_grad(ctx, X, D, B, T, d_in, d_out, grad_sum, accumulate_sum, st);
    return rc;
}

int adloco_gram_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                       int64_t d_out, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                       int accumulate_sum, void* stream) {
    return gram_route(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, grad_sum, accumulate_sum, -1,
                      stream);
}

int adloco_vector_param_sqnorm(adloco_ctx* ctx, const void* D, const void* X, int64_t B, int64_t T, int64_t d,
                               float* per_sample_sqnorm, int accumulate_norms, float* grad_sum, int accumulate_sum,
                               void* stream) {
    if (!ctx || !D || !per_sample_sqnorm) return ADLOCO_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d < 1) return ADLOCO_ERR_INVALID_ARG;
    if ((d % 8) != 0 || B > 65535) return ADLOCO_ERR_UNSUPPORTED;
    if (!aligned16(D) || (X && !aligned16(X))) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    return launch_vec_param(ctx, D, X, B, T, d, per_sample_sqnorm, accumulate_norms, grad_sum, accumulate_sum,
                            static_cast<cudaStream_t>(stream));
}

int adloco_embedding_sqnorm(adloco_ctx* ctx, const int32_t* token_ids, const void* D, int64_t B, int64_t T, int64_t d,
                            int64_t V, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                            int accumulate_sum, void* stream) {
    if (!ctx || !token_ids || !D || !per_sample_sqnorm) return ADLOCO_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d < 1 || V < 1) return ADLOCO_ERR_INVALID_ARG;
    if ((d % 8) != 0 || B > (1 << 30) || T > (1 << 30) || d > (1 << 30) || V > 0x7fffffff) return ADLOCO_ERR_UNSUPPORTED;
    if (!aligned16(D) || (reinterpret_cast<uintptr_t>(token_ids) & 3u) != 0) return ADLOCO_ERR_ALIGNMENT;
    if (grad_sum && !aligned16(grad_sum)) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    return launch_embedding(ctx, token_ids, D, B, T, d, V, per_sample_sqnorm, accumulate_norms, grad_sum, accumulate_sum,
                            static_cast<cudaStream_t>(stream));
}

int adloco_linear_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                         int64_t d_out, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                         int accumulate_sum, int method, void* stream) {
    if (method != ADLOCO_LINEAR_AUTO && method != ADLOCO_LINEAR_GRAM && method != ADLOCO_LINEAR_DIRECT &&
        method != ADLOCO_LINEAR_DIRECT_PAIR && method != ADLOCO_LINEAR_GRAM_ONE_CTA && method != ADLOCO_LINEAR_GRAM_PAIR)
        return ADLOCO_ERR_INVALID_ARG;
    if (!ctx || !X || !D || !per_sample_sqnorm) return ADLOCO_ERR_INVALID_ARG;
    if (B < 1 || T < 1 || d_in < 1 || d_out < 1) return ADLOCO_ERR_INVALID_ARG;
    if (method == ADLOCO_LINEAR_GRAM_ONE_CTA || method == ADLOCO_LINEAR_GRAM_PAIR)
        return gram_route(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, grad_sum, accumulate_sum,
                          method == ADLOCO_LINEAR_GRAM_PAIR ? 1 : 0, stream);
    const bool was_auto = (method == ADLOCO_LINEAR_AUTO);
    if (method == ADLOCO_LINEAR_AUTO) {
        // tensor work of the two routes at the granularity the kernels execute, divided by
        // the share of the SMs their work items can occupy (few tokens give the Gram kernel
        // fewer items than there are SMs; the direct kernel then wins despite more flops)
        const double sms = (double)ctx->sm_count;
        const double nt = (double)((T + 127) / 128);
        const double gram_items = (double)B * ((nt * (nt + 1) / 2 + 1) / 2);           // about one item per two blocks
        const double dir_items = (double)((d_out + 127) / 128) * (double)((d_in + 255) / 256) * (double)B;
        const double gemm = 2.0 * (double)B * (double)T * (double)d_in * (double)d_out;
        const double gram_util = gram_items < sms ? gram_items / sms : 1.0;
        const double dir_util = dir_items < sms ? dir_items / sms : 1.0;
        const double gram = 2.0 * (double)B * (nt * (nt + 1) / 2) * 128.0 * 128.0 * (double)(d_in + d_out) / gram_util +
                            (grad_sum ? gemm / dir_util : 0.0);
        const double direct = gemm / dir_util;
        method = direct <= gram ? ADLOCO_LINEAR_DIRECT : ADLOCO_LINEAR_GRAM;
    }
    if (method == ADLOCO_LINEAR_GRAM)
        return adloco_gram_sqnorm(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, grad_sum,
                                  accumulate_sum, stream);
    if ((d_in % 8) != 0 || (d_out % 8) != 0) return ADLOCO_ERR_UNSUPPORTED;
    if (B > (1 << 30) || T > (1 << 30) || d_in > (1 << 30) || d_out > (1 << 30)) return ADLOCO_ERR_UNSUPPORTED;
    if (!aligned16(X) || !aligned16(D)) return ADLOCO_ERR_ALIGNMENT;
    if (grad_sum && !aligned16(grad_sum)) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    // the automatic route takes the CTA-pair form of the direct kernel where clusters can be launched
    // and the tile is at least one pair's worth of rows
    if (was_auto && method == ADLOCO_LINEAR_DIRECT && d_out > 128 && pair_launch_ok(ctx)) method = ADLOCO_LINEAR_DIRECT_PAIR;
    if (method == ADLOCO_LINEAR_DIRECT_PAIR && !pair_launch_ok(ctx)) return ADLOCO_ERR_UNSUPPORTED;
    return launch_direct_sqnorm(ctx, X, D, B, T, d_in, d_out, per_sample_sqnorm, accumulate_norms, grad_sum,
                                accumulate_sum, method == ADLOCO_LINEAR_DIRECT_PAIR, static_cast<cudaStream_t>(stream));
}

int adloco_linear_sqnorm_group(adloco_ctx* ctx, const adloco_linear_layer* layers, int32_t n_layers, int64_t B,
                               int64_t T, float* per_sample_sqnorm, int accumulate_norms, int accumulate_sum,
                               int method, void* stream) {
    if (method != ADLOCO_LINEAR_AUTO && method != ADLOCO_LINEAR_DIRECT && method != ADLOCO_LINEAR_DIRECT_PAIR)
        return ADLOCO_ERR_INVALID_ARG;
    if (!ctx || !layers || n_layers < 1 || !per_sample_sqnorm || B < 1 || T < 1) return ADLOCO_ERR_INVALID_ARG;
    if (B > (1 << 30) || T > (1 << 30) || n_layers > (1 << 20)) return ADLOCO_ERR_UNSUPPORTED;
    for (int l = 0; l < n_layers; ++l) {
        const adloco_linear_layer& L = layers[l];
        if (!L.X || !L.D || L.d_in < 1 || L.d_out < 1) return ADLOCO_ERR_INVALID_ARG;
        if ((L.d_in % 8) != 0 || (L.d_out % 8) != 0 || L.d_in > (1 << 30) || L.d_out > (1 << 30)) return ADLOCO_ERR_UNSUPPORTED;
        if (!aligned16(L.X) || !aligned16(L.D) || (L.grad_sum && !aligned16(L.grad_sum))) return ADLOCO_ERR_ALIGNMENT;
    }
    DeviceGuard g(ctx->device);
    int pair = 0;
    if (method == ADLOCO_LINEAR_DIRECT_PAIR) {
        if (!pair_launch_ok(ctx)) return ADLOCO_ERR_UNSUPPORTED;
        pair = 1;
    } else if (method == ADLOCO_LINEAR_AUTO) {
        pair = pair_launch_ok(ctx) ? 1 : 0;
    }
    return launch_direct_group(ctx, layers, n_layers, B, T, per_sample_sqnorm, accumulate_norms, accumulate_sum, pair,
                               static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------
// switch-mode accumulator
// ---------------------------------------------------------------------------------
int adloco_accum_create(adloco_ctx* ctx, adloco_accum** out, float* const* sum_bufs, const int64_t* sum_sizes,
                        int32_t n_bufs) {
    if (!out) return ADLOCO_ERR_INVALID_ARG;
    *out = nullptr;
    if (!ctx || !sum_bufs || !sum_sizes || n_bufs < 1 || n_bufs > 4096) return ADLOCO_ERR_INVALID_ARG;
    for (int i = 0; i < n_bufs; ++i) {
        if (!sum_bufs[i] || sum_sizes[i] < 1) return ADLOCO_ERR_INVALID_ARG;
        if (!aligned16(sum_bufs[i])) return ADLOCO_ERR_ALIGNMENT;
    }
    DeviceGuard g(ctx->device);
    adloco_accum* a = new (std::nothrow) adloco_accum();
    if (!a) return ADLOCO_ERR_WORKSPACE;
    a->ctx = ctx;
    a->n_bufs = n_bufs;
    a->bufs_host = new float*[n_bufs];
    a->sizes_host = new int64_t[n_bufs];
    std::vector<int64_t> prefix(n_bufs + 1, 0);
    for (int i = 0; i < n_bufs; ++i) {
        a->bufs_host[i] = sum_bufs[i];
        a->sizes_host[i] = sum_sizes[i];
        prefix[i + 1] = prefix[i] + (sum_sizes[i] + 4095) / 4096;
    }
    a->total_chunks = prefix[n_bufs];
    bool ok = true;
    ok = ok && cudaMalloc(&a->bufs_dev, n_bufs * sizeof(float*)) == cudaSuccess;
    ok = ok && cudaMalloc(&a->sizes_dev, n_bufs * sizeof(int64_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&a->chunk_prefix_dev, (n_bufs + 1) * sizeof(int64_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&a->state, sizeof(adloco_test_sums)) == cudaSuccess;
    ok = ok && cudaMemcpy(a->bufs_dev, a->bufs_host, n_bufs * sizeof(float*), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(a->sizes_dev, a->sizes_host, n_bufs * sizeof(int64_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(a->chunk_prefix_dev, prefix.data(), (n_bufs + 1) * sizeof(int64_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemset(a->state, 0, sizeof(adloco_test_sums)) == cudaSuccess;
    if (!ok) { adloco_accum_destroy(a); return set_cuda_error(ctx, cudaGetLastError(), "adloco_accum_create"); }
    *out = a;
    return ADLOCO_OK;
}

int adloco_accum_destroy(adloco_accum* a) {
    if (!a) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(a->ctx->device);
    cudaFree(a->bufs_dev);
    cudaFree(a->sizes_dev);
    cudaFree(a->chunk_prefix_dev);
    cudaFree(a->state);
    delete[] a->bufs_host;
    delete[] a->sizes_host;
    delete a;
    return ADLOCO_OK;
}

int adloco_accum_reset(adloco_ctx* ctx, adloco_accum* a, void* stream) {
    if (!ctx || !a || a->ctx != ctx) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int rc = launch_accum_zero(ctx, a, st);     // every S buffer and the state, one launch
    if (rc != ADLOCO_OK) return rc;
    a->sqnorm_current = true;
    return ADLOCO_OK;
}

int adloco_accumulate(adloco_ctx* ctx, adloco_accum* a, const void* grads, adloco_dtype dtype, int64_t b_micro,
                      int64_t P, int64_t row_stride, float* per_sample_sqnorm, void* stream) {
    if (!ctx || !a || a->ctx != ctx || b_micro < 1) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (grads == nullptr) {
        if (!per_sample_sqnorm) return ADLOCO_ERR_INVALID_ARG;
        a->sqnorm_current = false;   // the caller has changed the S buffers itself
        return launch_accum_add_norms(ctx, a, per_sample_sqnorm, b_micro, st);
    }
    int rc = check_grads(grads, dtype, b_micro, P, row_stride);
    if (rc != ADLOCO_OK) return rc;
    if (a->n_bufs != 1 || a->sizes_host[0] != P) return ADLOCO_ERR_INVALID_ARG;
    NtLaunch l;
    l.G = static_cast<const float*>(grads);
    l.bf16 = (dtype == ADLOCO_BF16);
    l.B = b_micro; l.P = P; l.stride = row_stride;
    l.n_out = per_sample_sqnorm; l.S = a->bufs_host[0];
    l.sums = a->state; l.result = nullptr; l.mode = NT_MICRO;
    // this pass rewrites all of S and leaves ||S||^2 in the state
    a->sqnorm_current = true;
    return launch_norm_test(ctx, l, st);
}

int adloco_accum_finalize(adloco_ctx* ctx, adloco_accum* a, const adloco_test_params* params,
                          adloco_test_sums* sums_dev, adloco_test_result* result_dev,
                          adloco_test_result* result_host, void* stream) {
    if (!ctx || !a || a->ctx != ctx || !result_dev) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_params(params);
    if (rc != ADLOCO_OK) return rc;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // ||S||^2 over every buffer, unless the last materialised micro-batch left it current
    if (!a->sqnorm_current) {
        rc = launch_accum_sqnorm(ctx, a, st);
        if (rc != ADLOCO_OK) return rc;
        a->sqnorm_current = true;
    }
    adloco_test_result* mirror = static_cast<adloco_test_result*>(device_address_of_pinned(result_host));
    rc = launch_decide(ctx, a->state, *params, result_dev, mirror, st);
    if (rc != ADLOCO_OK) return rc;
    if (sums_dev)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(sums_dev, a->state, sizeof(adloco_test_sums), cudaMemcpyDeviceToDevice, st));
    if (result_host && !mirror)
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(result_host, result_dev, sizeof(adloco_test_result), cudaMemcpyDeviceToHost, st));
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// outer step
// ---------------------------------------------------------------------------------
int adloco_outer_step(adloco_ctx* ctx, const void* const* inst_params, adloco_dtype inst_dtype, int32_t K,
                      int64_t P, const float* theta_in, float* theta_out, const float* mom_in, float* mom_out,
                      float lr, float momentum, int nesterov, void* const* inst_writeback, void* stream) {
    if (!ctx || !inst_params || !theta_in || !theta_out || !mom_in || !mom_out) return ADLOCO_ERR_INVALID_ARG;
    if (K < 1 || P < 1) return ADLOCO_ERR_INVALID_ARG;
    if (K > kMaxInstances) return ADLOCO_ERR_UNSUPPORTED;
    if (inst_dtype != ADLOCO_F32 && inst_dtype != ADLOCO_BF16) return ADLOCO_ERR_INVALID_ARG;
    if (!(lr == lr) || !(momentum == momentum)) return ADLOCO_ERR_INVALID_ARG;
    if (!aligned16(theta_in) || !aligned16(theta_out) || !aligned16(mom_in) || !aligned16(mom_out)) return ADLOCO_ERR_ALIGNMENT;
    OuterLaunch l;
    for (int k = 0; k < K; ++k) {
        if (!inst_params[k]) return ADLOCO_ERR_INVALID_ARG;
        if (!aligned16(inst_params[k])) return ADLOCO_ERR_ALIGNMENT;
        l.inst[k] = inst_params[k];
        l.wb[k] = nullptr;
        if (inst_writeback && inst_writeback[k]) {
            if (!aligned16(inst_writeback[k])) return ADLOCO_ERR_ALIGNMENT;
            l.wb[k] = inst_writeback[k];
            l.has_wb = 1;
        }
    }
    l.K = K; l.bf16 = (inst_dtype == ADLOCO_BF16); l.P = P;
    l.th_in = theta_in; l.th_out = theta_out; l.v_in = mom_in; l.v_out = mom_out;
    l.lr = lr; l.mu = momentum; l.nesterov = nesterov ? 1 : 0;
    DeviceGuard g(ctx->device);
    return launch_outer_step(ctx, l, static_cast<cudaStream_t>(stream));
}

int adloco_outer_step_host(adloco_ctx* ctx, const void* const* inst_params_host, adloco_dtype inst_dtype,
                           int32_t K, int64_t P, float* theta_host, float* mom_host, float lr, float momentum,
                           int nesterov, void* stream) {
    if (!ctx || !inst_params_host || !theta_host || !mom_host) return ADLOCO_ERR_INVALID_ARG;
    if (K < 1 || P < 1) return ADLOCO_ERR_INVALID_ARG;
    if (K > kMaxInstances) return ADLOCO_ERR_UNSUPPORTED;
    if (inst_dtype != ADLOCO_F32 && inst_dtype != ADLOCO_BF16) return ADLOCO_ERR_INVALID_ARG;
    for (int k = 0; k < K; ++k) if (!inst_params_host[k]) return ADLOCO_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t es = inst_dtype == ADLOCO_BF16 ? 2 : 4;
    const size_t per_elem = 8 + (size_t)K * es;
    // panel of L elements (a multiple of 1024): theta | mom | K instance slices
    int64_t L = (int64_t)(kPanelBytes / per_elem);
    L = std::max<int64_t>(1024, (L / 1024) * 1024);
    if (L > P) L = ((P + 1023) / 1024) * 1024;
    int rc = ensure_staging(ctx, (size_t)L * per_elem);
    if (rc != ADLOCO_OK) return rc;
    HostStaging& s = ctx->staging;
    const int64_t npanels = (P + L - 1) / L;
    ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.out_done[0], st));
    ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.out_done[1], st));
    for (int64_t p = 0; p < npanels; ++p) {
        const int b = (int)(p & 1);
        const int64_t e0 = p * L;
        const int64_t n = std::min<int64_t>(L, P - e0);
        char* base = static_cast<char*>(s.dev[b]);
        float* th = reinterpret_cast<float*>(base);
        float* mv = reinterpret_cast<float*>(base + (size_t)L * 4);
        char* inst0 = base + (size_t)L * 8;
        // fill: after the previous results of this buffer have left it
        ADLOCO_CUDA_TRY(ctx, cudaStreamWaitEvent(s.copy_stream, s.out_done[b], 0));
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(th, theta_host + e0, (size_t)n * 4, cudaMemcpyHostToDevice, s.copy_stream));
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(mv, mom_host + e0, (size_t)n * 4, cudaMemcpyHostToDevice, s.copy_stream));
        OuterLaunch l;
        for (int k = 0; k < K; ++k) {
            char* dst = inst0 + (size_t)k * (size_t)L * es;
            ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(dst, static_cast<const char*>(inst_params_host[k]) + (size_t)e0 * es,
                                                 (size_t)n * es, cudaMemcpyHostToDevice, s.copy_stream));
            l.inst[k] = dst;
            l.wb[k] = nullptr;
        }
        ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.filled[b], s.copy_stream));
        ADLOCO_CUDA_TRY(ctx, cudaStreamWaitEvent(st, s.filled[b], 0));
        l.K = K; l.bf16 = (inst_dtype == ADLOCO_BF16); l.P = n;
        l.th_in = th; l.th_out = th; l.v_in = mv; l.v_out = mv;
        l.lr = lr; l.mu = momentum; l.nesterov = nesterov ? 1 : 0;
        rc = launch_outer_step(ctx, l, st);
        if (rc != ADLOCO_OK) return rc;
        // results go back on the caller's stream, overlapping the next panel's fill
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(theta_host + e0, th, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
        ADLOCO_CUDA_TRY(ctx, cudaMemcpyAsync(mom_host + e0, mv, (size_t)n * 4, cudaMemcpyDeviceToHost, st));
        ADLOCO_CUDA_TRY(ctx, cudaEventRecord(s.out_done[b], st));
    }
    ADLOCO_CUDA_TRY(ctx, cudaStreamSynchronize(st));
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// outer step split around an exchange of pseudo-gradients
// ---------------------------------------------------------------------------------
int adloco_pseudo_gradient(adloco_ctx* ctx, const float* theta, const void* inst_params, adloco_dtype inst_dtype,
                           int64_t P, float* pseudo_grad, void* stream) {
    if (!ctx || !theta || !inst_params || !pseudo_grad || P < 1) return ADLOCO_ERR_INVALID_ARG;
    if (inst_dtype != ADLOCO_F32 && inst_dtype != ADLOCO_BF16) return ADLOCO_ERR_INVALID_ARG;
    if (!aligned16(theta) || !aligned16(inst_params) || !aligned16(pseudo_grad)) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    return launch_pseudo_grad(ctx, theta, inst_params, inst_dtype == ADLOCO_BF16, pseudo_grad, P,
                              static_cast<cudaStream_t>(stream));
}

int adloco_outer_apply(adloco_ctx* ctx, const float* pseudo_grad_sum, int32_t K, int64_t P, const float* theta_in,
                       float* theta_out, const float* mom_in, float* mom_out, float lr, float momentum, int nesterov,
                       void* stream) {
    if (!ctx || !pseudo_grad_sum || !theta_in || !theta_out || !mom_in || !mom_out || K < 1 || P < 1)
        return ADLOCO_ERR_INVALID_ARG;
    if (!(lr == lr) || !(momentum == momentum)) return ADLOCO_ERR_INVALID_ARG;
    if (!aligned16(pseudo_grad_sum) || !aligned16(theta_in) || !aligned16(theta_out) || !aligned16(mom_in) ||
        !aligned16(mom_out))
        return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    return launch_outer_apply(ctx, pseudo_grad_sum, K, P, theta_in, theta_out, mom_in, mom_out, lr, momentum,
                              nesterov ? 1 : 0, static_cast<cudaStream_t>(stream));
}

int adloco_refresh_instance(adloco_ctx* ctx, const float* theta, void* inst_params, adloco_dtype inst_dtype, int64_t P,
                            void* stream) {
    if (!ctx || !theta || !inst_params || P < 1) return ADLOCO_ERR_INVALID_ARG;
    if (inst_dtype != ADLOCO_F32 && inst_dtype != ADLOCO_BF16) return ADLOCO_ERR_INVALID_ARG;
    if (!aligned16(theta) || !aligned16(inst_params)) return ADLOCO_ERR_ALIGNMENT;
    DeviceGuard g(ctx->device);
    return launch_refresh(ctx, theta, inst_params, inst_dtype == ADLOCO_BF16, P, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------
// trainer merge
// ---------------------------------------------------------------------------------
int adloco_check_merge(const int64_t* b_req, int32_t k, int32_t w, int32_t* merge_idx) {
    if (k < 0 || w < 0 || (k > 0 && !b_req)) return ADLOCO_ERR_INVALID_ARG;
    if (w == 0 || k <= 1 || w > k) return 0;
    if (!merge_idx) return ADLOCO_ERR_INVALID_ARG;
    std::vector<int32_t> order(k);
    for (int32_t i = 0; i < k; ++i) order[i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return b_req[x] < b_req[y]; });
    for (int32_t i = 0; i < w; ++i) merge_idx[i] = order[i];
    return w;
}

int adloco_merge(adloco_ctx* ctx, const void* const* members, const int64_t* weights, adloco_dtype dtype,
                 int32_t K, int64_t P, void* out, int32_t* rep, void* stream) {
    if (!ctx || !members || !weights || !out || K < 1 || P < 1) return ADLOCO_ERR_INVALID_ARG;
    if (K > kMaxInstances) return ADLOCO_ERR_UNSUPPORTED;
    if (dtype != ADLOCO_F32 && dtype != ADLOCO_BF16) return ADLOCO_ERR_INVALID_ARG;
    if (!aligned16(out)) return ADLOCO_ERR_ALIGNMENT;
    long double wsum = 0;
    int32_t best = 0;
    for (int k = 0; k < K; ++k) {
        if (!members[k] || weights[k] <= 0) return ADLOCO_ERR_INVALID_ARG;
        if (!aligned16(members[k])) return ADLOCO_ERR_ALIGNMENT;
        wsum += (long double)weights[k];
        if (weights[k] > weights[best]) best = k;
    }
    MergeLaunch l;
    for (int k = 0; k < K; ++k) {
        l.x[k] = members[k];
        l.coef[k] = (float)((long double)weights[k] / wsum);
    }
    l.K = K; l.bf16 = (dtype == ADLOCO_BF16); l.P = P; l.out = out;
    if (rep) *rep = best;
    DeviceGuard g(ctx->device);
    return launch_merge(ctx, l, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
