/*
 * adloco.h -- C ABI of the AdLoCo hot path on one B200 (sm_100a).
 *
 * The library computes, with hand-written CUDA kernels,
 *   - the approximate norm test that sizes the next local batch
 *     (paper, Section "Norm test": sigma^2_B, the batch rule b_{k+1}),
 *   - switch mode's accumulation of the test sums over micro-batches
 *     (Section "Mode switching"; first branch of Algorithm 3),
 *   - the outer step over K model instances (last loop of Algorithm 3),
 *   - the trainer merge (Algorithms 1 and 2).
 *
 * Conventions for every entry point
 *   - Returns an adloco_status (0 = ok, negative = error).  No exception, abort
 *     or trap crosses this boundary.  Argument errors are found on the host
 *     before anything is launched.
 *   - "dev" pointers are device memory owned by the caller; "host" pointers are
 *     host memory owned by the caller.  Base pointers of vector data must be
 *     16-byte aligned unless an entry point says otherwise (ADLOCO_ERR_ALIGNMENT
 *     if not).  The library owns only the workspace inside an adloco_ctx.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream) and is asynchronous unless stated.  The streaming
 *     entry points (norm test, accumulate, finalize, inner-product test, host
 *     variants) share the ctx workspace: do not run two of them at the same
 *     time on one ctx.  The per-layer entry points (adloco_gram_sqnorm,
 *     adloco_linear_sqnorm, adloco_linear_sqnorm_group, adloco_embedding_sqnorm,
 *     adloco_vector_param_sqnorm), adloco_outer_step and adloco_merge use none of it and may be issued on
 *     several streams at once -- the layers of one micro-batch only add into
 *     n and into their own S, and alternating them on two streams overlaps
 *     one kernel's tail with the next one's start.
 *   - Sizes are int64_t element counts; all byte offsets are 64-bit inside.
 *   - There is no CPU fallback: without a usable CUDA device the calls fail
 *     with ADLOCO_ERR_CUDA.
 */
#ifndef ADLOCO_H
#define ADLOCO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adloco_ctx adloco_ctx;     /* device id and workspace */
typedef struct adloco_accum adloco_accum; /* switch-mode accumulator state */

typedef enum {
    ADLOCO_OK = 0,
    ADLOCO_ERR_INVALID_ARG = -1,
    ADLOCO_ERR_UNSUPPORTED = -2, /* a shape the kernels do not take; never a silent fallback */
    ADLOCO_ERR_ALIGNMENT = -3,
    ADLOCO_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed; see adloco_last_cuda_error */
    ADLOCO_ERR_WORKSPACE = -5,
    ADLOCO_ERR_TIMEOUT = -6      /* a bounded wait inside a kernel ran out (device status word) */
} adloco_status;

typedef enum { ADLOCO_F32 = 0, ADLOCO_BF16 = 1 } adloco_dtype;

enum {
    ADLOCO_FLAG_GROW = 1,       /* b_req > b_cur */
    ADLOCO_FLAG_ACCUMULATE = 2, /* switch mode: b_req > switch_n * b_max */
    ADLOCO_FLAG_UNDEFINED = 4,  /* batch_count - ddof <= 0: no variance; b_req = max(1, b_cur) */
    ADLOCO_FLAG_ZERO_MEAN = 8,  /* ||gbar||^2 == 0: stat = +inf, b_req = b_cap or INT64_MAX */
    ADLOCO_FLAG_NONFINITE = 16  /* a sum is Inf or NaN (an overflowed gradient): variance = stat = 0
                                   are placeholders, b_req = max(1, b_cur); checked before the others */
};

/* Parameters of the batch rule and of switch mode.
 *   eta      threshold of the norm test, > 0 and finite
 *   ddof     variance normaliser is (b - ddof); 1 = unbiased sample variance
 *   b_cur    current batch size (only for the GROW flag and the UNDEFINED case)
 *   b_max    largest micro-batch the hardware holds (max_batch), >= 1
 *   b_cap    upper clamp on b_req, 0 = none
 *   switch_n switch multiplier n (the paper uses 2), >= 1 */
typedef struct {
    double eta;
    int32_t ddof;
    int32_t switch_n;
    int64_t b_cur;
    int64_t b_max;
    int64_t b_cap;
} adloco_test_params;

/* Sufficient statistics of one test (device memory, written by the kernels).
 *   sum_sqnorm  Q   = sum_i ||g_i||^2
 *   sum_sq_gsum      ||sum_i g_i||^2  (so ||gbar||^2 = sum_sq_gsum / b^2)
 *   centred_ss       sum_i ||g_i - gbar||^2 computed column-centred; valid iff has_centred
 *   batch_count b */
typedef struct {
    double sum_sqnorm;
    double sum_sq_gsum;
    double centred_ss;
    int64_t batch_count;
    int32_t has_centred;
    int32_t device_status; /* 0, or an adloco_status raised on the device */
} adloco_test_sums;

/* Outcome of the test.  mean_sqnorm = ||gbar||^2, variance = sigma^2_B,
 * stat = variance / (eta^2 mean_sqnorm), b_req = max(1, ceil(stat)) clamped by b_cap;
 * accum_steps / b_micro are the switch-mode plan. */
typedef struct {
    double sum_sqnorm;
    double mean_sqnorm;
    double variance;
    double stat;
    int64_t batch_count;
    int64_t b_req;
    int64_t accum_steps;
    int64_t b_micro;
    uint32_t flags;
    int32_t device_status;
} adloco_test_result;

/* ---- context ------------------------------------------------------------ */

/* Creates a context on CUDA device `device` (allocates about 10 MB of workspace, sized
 * for the largest batch the streaming entry points take, so that none of them allocates
 * or synchronises later; synchronous).  *out is NULL on failure. */
int adloco_create(adloco_ctx** out, int device);
/* Frees the workspace.  The caller must have synchronised every stream that used it. */
int adloco_destroy(adloco_ctx* ctx);
const char* adloco_status_string(int status);
/* Text of the last CUDA error seen by this ctx ("" if none); valid until the next call. */
const char* adloco_last_cuda_error(const adloco_ctx* ctx);
/* Number of kernel launches this ctx has enqueued so far. */
int64_t adloco_launch_count(const adloco_ctx* ctx);

/* The tensor-core kernels wait on hardware barriers (tile arrived, accumulator
 * drained).  Every such wait is bounded: when `limit_ns` of wall time pass the
 * kernel stops waiting, lets its copies in flight land, frees its tensor memory,
 * returns, and raises the context's device status word to ADLOCO_ERR_TIMEOUT; the
 * outputs of that call are then undefined but the context stays usable.  Default
 * 2 s.  adloco_device_status reads the word (synchronises `stream`) and
 * optionally clears it. */
int adloco_set_wait_limit(adloco_ctx* ctx, uint64_t limit_ns);
int adloco_device_status(adloco_ctx* ctx, int32_t* status_host, int clear, void* stream);

/* ---- norm test on materialised per-sample gradients ---------------------- */

/* Section "Norm test" (Eq. 1, sigma^2_B, b_{k+1}) followed by the switch-mode
 * plan (Section "Mode switching").
 *   grads              dev, [B, P] row-major, row i = g_i, row pitch `row_stride`
 *                      elements (>= P), dtype F32 or BF16 (widened exactly, fp32 arithmetic).
 *                      Vector loads are used when the base is 16-byte (F32) / 8-byte (BF16)
 *                      aligned and the pitch is a multiple of 4 (and grad_sum, if given, is
 *                      16-byte aligned); otherwise a slower element-wise path runs.
 *                      1 <= B <= 4096.
 *   per_sample_sqnorm  dev [B] float, receives n_i = ||g_i||^2; may be NULL
 *   grad_sum           dev [P] float, receives S = sum_i g_i; may be NULL
 *   sums_dev           dev, receives the sufficient statistics; may be NULL
 *   result_dev         dev, receives the decision; required
 *   result_host        host copy of the decision, valid after `stream` is synchronised; may be NULL.
 *                      Page-locked memory (cudaHostAlloc, cudaHostRegister) is written by the kernel
 *                      itself, which keeps a copy engine out of the stream (about 11 us per call);
 *                      pageable memory is filled by an async copy on `stream`.  The same holds for
 *                      every result_host of this library.
 * One pass over G: per-row sum of squares, per-column sum and column-centred
 * sum of squares, fp32 inside a thread, fp64 across threads and blocks (fixed
 * order: results are run-to-run deterministic).  B >= 1, P >= 1. */
int adloco_norm_test(adloco_ctx* ctx, const void* grads, adloco_dtype dtype, int64_t B, int64_t P,
                     int64_t row_stride, const adloco_test_params* params, float* per_sample_sqnorm,
                     float* grad_sum, adloco_test_sums* sums_dev, adloco_test_result* result_dev,
                     adloco_test_result* result_host, void* stream);

/* The batch rule and switch plan alone, from sufficient statistics already on
 * the device (e.g. to sweep eta without re-reading the gradients). */
int adloco_test_decide(adloco_ctx* ctx, const adloco_test_sums* sums_dev, const adloco_test_params* params,
                       adloco_test_result* result_dev, adloco_test_result* result_host, void* stream);

/* Same as adloco_norm_test with `grads_host` in HOST memory ([B, P], pitch
 * row_stride): the library stages column panels through device buffers it owns,
 * overlapping the copies with the reduction.  Synchronous: on return
 * *result_host (required) and the optional host outputs per_sample_sqnorm_host
 * [B] are valid. */
int adloco_norm_test_host(adloco_ctx* ctx, const float* grads_host, int64_t B, int64_t P, int64_t row_stride,
                          const adloco_test_params* params, float* per_sample_sqnorm_host,
                          adloco_test_result* result_host, void* stream);

/* Norm test for callers that must not allocate.  The paper has no counterpart:
 * this is adloco_norm_test (same kernel, same results) with the reduction
 * scratch in a device array built into the library (about 290 KB per GPU, held
 * from library load to process exit) instead of an adloco_ctx, for callers that
 * cannot call cudaMalloc where the test runs -- e.g. inside a step whose
 * allocator pool is frozen, or with the device-memory budget already spent.
 * It calls no cudaMalloc/cudaFree and no allocating library routine.
 *   - runs on the CURRENT device, on `stream`; grads/per_sample_sqnorm (may be
 *     NULL)/result_dev are caller-owned dev memory, result_host (may be NULL) is
 *     filled by an async copy as in adloco_norm_test
 *   - limit: B <= 64 rows (ADLOCO_ERR_UNSUPPORTED beyond); any P >= 1
 *   - the first call on each device looks up the array's device address; make
 *     that first call before any stream capture
 *   - every call shares the one array: calls that overlap on the GPU (different
 *     streams, or different threads) race and give wrong results; calls on one
 *     stream are safe back to back. */
int adloco_norm_test_noalloc(const float* grads, int64_t B, int64_t P, int64_t row_stride,
                             const adloco_test_params* params, float* per_sample_sqnorm,
                             adloco_test_result* result_dev, adloco_test_result* result_host, void* stream);

/* ---- inner-product test and augmented inner-product test ------------------ */

/* Parameters: theta and nu are the thresholds of the two tests (> 0, finite);
 * ddof, b_cur, b_cap as in adloco_test_params. */
typedef struct {
    double theta;
    double nu;
    int32_t ddof;
    int32_t reserved;
    int64_t b_cur;
    int64_t b_cap;
} adloco_ip_params;

/* var_ip = Var_i <g_i, gbar>, stat_ip = var_ip / (theta^2 ||gbar||^4), b_ip = max(1, ceil(stat_ip));
 * var_orth = Var_i (g_i - (<g_i, gbar> / ||gbar||^2) gbar), stat_orth = var_orth / (nu^2 ||gbar||^2),
 * b_aug = max(b_ip, ceil(stat_orth)).  Flags GROW (b_aug > b_cur), UNDEFINED, ZERO_MEAN, NONFINITE as for the
 * norm test. */
typedef struct {
    double var_ip;
    double stat_ip;
    double var_orth;
    double stat_orth;
    double mean_sqnorm;
    int64_t batch_count;
    int64_t b_ip;
    int64_t b_aug;
    uint32_t flags;
    int32_t device_status;
} adloco_ip_result;

/* Section "Inner product test": both batch rules for the batch whose norm test
 * has just run.  A second pass over G:
 *   grads, B, P, row_stride   as in adloco_norm_test (the same G)
 *   grad_sum                  dev [P] float: S = sum_i g_i, the grad_sum output of that norm test (required)
 *   sums_dev                  dev: the sums_dev output of that norm test (required)
 *   inner_products            dev [B] float, receives <g_i, gbar>; may be NULL
 *   result_dev / result_host  as in adloco_norm_test
 * Algorithmic traffic 4 B P + 4 P bytes. */
int adloco_inner_product_test(adloco_ctx* ctx, const void* grads, adloco_dtype dtype, int64_t B, int64_t P,
                              int64_t row_stride, const adloco_ip_params* params, const float* grad_sum,
                              const adloco_test_sums* sums_dev, float* inner_products,
                              adloco_ip_result* result_dev, adloco_ip_result* result_host, void* stream);

/* ---- per-sample norms of a linear layer via the Gram identity ------------ */

/* For a linear layer y = W x and a batch of B sequences of T tokens, sample i
 * has weight gradient G_i = sum_t delta_{i,t} x_{i,t}^T (Eq. 1 applied to W).
 * This call computes, on the tensor cores,
 *   n_i = ||G_i||_F^2 = sum_{t,s} (x_t . x_s)(delta_t . delta_s)     (Gram identity)
 *   S   = sum_i G_i = Delta^T X  ([d_out, d_in], fp32 accumulate)     (optional)
 *   X  dev bf16 [B, T, d_in]  row-major (features contiguous)
 *   D  dev bf16 [B, T, d_out] row-major
 *   per_sample_sqnorm  dev [B] float; overwritten, or += when accumulate_norms != 0
 *   grad_sum           dev [d_out, d_in] float, may be NULL; overwritten, or += when
 *                      accumulate_sum != 0
 * d_in and d_out must be multiples of 8 (ADLOCO_ERR_UNSUPPORTED otherwise); any
 * B, T >= 1.  bf16 x bf16 products are exact in fp32; accumulation is fp32. */
int adloco_gram_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                       int64_t d_out, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                       int accumulate_sum, void* stream);

/* Same outputs as adloco_gram_sqnorm (n_i and, optionally, S; same argument
 * meaning and limits) with a choice of route:
 *   ADLOCO_LINEAR_GRAM    the Gram identity (adloco_gram_sqnorm)
 *   ADLOCO_LINEAR_DIRECT  each sample's gradient tile G_i = D_i^T X_i (Eq. 1 applied to
 *                         W, before the mean) is formed in tensor memory, squared and
 *                         summed into n_i and added into S on chip; G_i never reaches HBM.
 *                         One GEMM of 2 B T d_in d_out flops gives both outputs.
 *   ADLOCO_LINEAR_DIRECT_PAIR  the direct route with 256 x 256 tiles, each shared by the two
 *                         SMs of a thread-block cluster (each loads half of the operands);
 *                         ADLOCO_ERR_UNSUPPORTED where cluster launches are not available.
 *   ADLOCO_LINEAR_GRAM_ONE_CTA / ADLOCO_LINEAR_GRAM_PAIR  the Gram identity by a named kernel: one CTA
 *                         per 128 x 256-token tile (what ADLOCO_LINEAR_GRAM and adloco_gram_sqnorm run), or
 *                         256 x 256-token tiles shared by the two SMs of a cluster (same result; a third less
 *                         traffic into shared memory and one read of the operands from HBM, for one unused
 *                         128 x 128 sub-block per diagonal tile; measured as fast as the one-CTA kernel at
 *                         T = 1024; ADLOCO_ERR_UNSUPPORTED where cluster launches are not available).
 *   ADLOCO_LINEAR_AUTO    whichever executes fewer tensor-core flops for the shape
 *                         (direct wins when T exceeds about d_in d_out / (d_in + d_out));
 *                         the direct route then runs in its pair form where available. */
enum { ADLOCO_LINEAR_AUTO = 0, ADLOCO_LINEAR_GRAM = 1, ADLOCO_LINEAR_DIRECT = 2, ADLOCO_LINEAR_DIRECT_PAIR = 3,
       ADLOCO_LINEAR_GRAM_ONE_CTA = 4, ADLOCO_LINEAR_GRAM_PAIR = 5 };
int adloco_linear_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                         int64_t d_out, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                         int accumulate_sum, int method, void* stream);

/* One linear layer of a group: X dev bf16 [B, T, d_in], D dev bf16 [B, T, d_out],
 * grad_sum dev float [d_out, d_in] or NULL; d_in, d_out multiples of 8. */
typedef struct {
    const void* X;
    const void* D;
    int64_t d_in;
    int64_t d_out;
    float* grad_sum;
} adloco_linear_layer;

/* All linear layers of one (micro-)batch in one call (Eq. 1 applied per weight matrix; a
 * sample's gradient is the concatenation over the layers, so its squared norm adds up):
 *   per_sample_sqnorm[i] (+)= sum over the layers of ||D_i^T X_i||_F^2,
 *   layers[l].grad_sum   (+)= sum_i D_i^T X_i   for every layer that gives a buffer.
 *   layers   HOST array of n_layers entries (read during the call); all layers share B and T
 *   method   ADLOCO_LINEAR_DIRECT, ADLOCO_LINEAR_DIRECT_PAIR or ADLOCO_LINEAR_AUTO (the pair
 *            kernel where available, else the direct one)
 * The direct route runs the whole group as one persistent launch per 48 layers: the work
 * items of all layers are dealt to the SMs from one list, so small layers pay no launch of
 * their own and layers whose tile count does not divide the SM count leave no SM idle.
 * accumulate_norms / accumulate_sum as in adloco_gram_sqnorm, applied to every layer. */
int adloco_linear_sqnorm_group(adloco_ctx* ctx, const adloco_linear_layer* layers, int32_t n_layers, int64_t B,
                               int64_t T, float* per_sample_sqnorm, int accumulate_norms, int accumulate_sum,
                               int method, void* stream);

/* Per-sample gradient norms of a vector parameter of width d that acts at every
 * token (Eq. 1 applied to that parameter): a bias, g_i = sum_t delta_{i,t} (X = NULL),
 * or an elementwise gain such as LayerNorm's, g_i = sum_t delta_{i,t} * x_{i,t}
 * (X = the normalised input).  n_i = ||g_i||^2 and, optionally, S = sum_i g_i.
 *   D, X               dev bf16 [B, T, d] row-major; d a multiple of 8, B <= 65535
 *   per_sample_sqnorm  dev [B] float; overwritten, or += when accumulate_norms != 0
 *   grad_sum           dev [d] float, may be NULL; overwritten, or += when accumulate_sum != 0
 * One streaming pass (2 B T d bytes per operand), fp32 accumulation. */
int adloco_vector_param_sqnorm(adloco_ctx* ctx, const void* D, const void* X, int64_t B, int64_t T, int64_t d,
                               float* per_sample_sqnorm, int accumulate_norms, float* grad_sum, int accumulate_sum,
                               void* stream);

/* Per-sample gradient norms of an embedding table E [V, d] looked up at every token
 * (Eq. 1 applied to E): row v of sample i's gradient is the sum of delta_{i,t} over the
 * tokens with token_ids[i, t] = v, and n_i = sum_v || sum_{t: id_t = v} delta_t ||^2.
 * Up to T = 4096 the tokens of a sample are grouped by id on chip and every delta row is
 * read once (a streaming pass; ids that occur once contribute their row's squared norm,
 * repeated ids the squared norm of their rows' sum); longer sequences take the equivalent
 * n_i = sum_{t,s} [id_t == id_s] (delta_t . delta_s) -- the Gram identity with a
 * token-equality mask in place of X X^T -- on the tensor cores.
 * With position indices as ids it covers a learned positional embedding.
 *   token_ids          dev int32 [B, T], values in [0, V) (others match nothing and are skipped)
 *   D                  dev bf16 [B, T, d]: gradient of the loss w.r.t. the looked-up rows; d % 8 == 0
 *   per_sample_sqnorm  dev [B] float; overwritten, or += when accumulate_norms != 0
 *   grad_sum           dev [V, d] float, may be NULL: S = sum_i G_i (scatter-add); overwritten
 *                      (V d floats are cleared first), or += when accumulate_sum != 0 */
int adloco_embedding_sqnorm(adloco_ctx* ctx, const int32_t* token_ids, const void* D, int64_t B, int64_t T, int64_t d,
                            int64_t V, float* per_sample_sqnorm, int accumulate_norms, float* grad_sum,
                            int accumulate_sum, void* stream);

/* ---- switch-mode accumulation -------------------------------------------- */

/* Accumulator of the test sums over the micro-batches of one large batch:
 * Q = sum n_i, the batch count, and the gradient-sum buffers S (one per
 * parameter buffer; caller-owned dev float arrays that the accumulator borrows).
 * adloco_accum_create copies the n_bufs pointers/sizes (host arrays) and
 * allocates a small device state; synchronous. */
int adloco_accum_create(adloco_ctx* ctx, adloco_accum** out, float* const* sum_bufs, const int64_t* sum_sizes,
                        int32_t n_bufs);
/* Zeroes Q, the count and every S buffer (async on stream). */
int adloco_accum_reset(adloco_ctx* ctx, adloco_accum* acc, void* stream);
int adloco_accum_destroy(adloco_accum* acc);   /* before its ctx is destroyed */

/* Adds one micro-batch (Algorithm 3's g <- g + grad L(x; B), applied to the
 * test sums).  Two forms:
 *  (a) grads != NULL: materialised micro-batch [b_micro, P] float (pitch row_stride),
 *      P == sum_sizes[0] and n_bufs == 1.  One pass adds sum_i g_i into S, sum_i n_i
 *      into Q, and keeps the centred sum of squares exact across micro-batches by
 *      the pairwise update  css += css_mb + (c b/(c+b)) ||mean_mb - mean_so_far||^2.
 *      per_sample_sqnorm (dev [b_micro], may be NULL) receives this micro-batch's n_i.
 *  (b) grads == NULL: the caller has already added this micro-batch's gradient sums
 *      into the S buffers (adloco_gram_sqnorm with accumulate_sum) and passes its
 *      n_i in per_sample_sqnorm (dev [b_micro], required); only Q and the count move. */
int adloco_accumulate(adloco_ctx* ctx, adloco_accum* acc, const void* grads, adloco_dtype dtype,
                      int64_t b_micro, int64_t P, int64_t row_stride, float* per_sample_sqnorm, void* stream);

/* One test on everything accumulated: N = sum_bufs ||S/b||^2,
 * V = centred_ss/(b-ddof) when every micro-batch was materialised, otherwise
 * V = (Q - b N)/(b - ddof); then the batch rule and switch plan.  ||S||^2 is taken
 * from the last form-(a) call when that was the last change to S (the caller must
 * not modify S behind a form-(a) accumulation), else reduced here. */
int adloco_accum_finalize(adloco_ctx* ctx, adloco_accum* acc, const adloco_test_params* params,
                          adloco_test_sums* sums_dev, adloco_test_result* result_dev,
                          adloco_test_result* result_host, void* stream);

/* ---- outer step ----------------------------------------------------------- */

/* Last loop of Algorithm 3 for one trainer, fused in one pass:
 *   d      = (1/K) sum_k (theta - theta_k)
 *   v'     = momentum v + d
 *   u      = d + momentum v' (nesterov != 0)  |  v'
 *   theta' = theta - lr u
 *   inst_params  HOST array of K dev pointers, each [P] in inst_dtype (F32 or BF16),
 *                separate allocations allowed; 1 <= K <= 64
 *   theta_in/out, mom_in/out  dev [P] float; out may be the same pointer as in
 *                (exact aliasing only); instances must not overlap theta or mom
 *   inst_writeback  HOST array of K dev pointers (may be NULL, entries may be NULL):
 *                each receives theta' rounded to inst_dtype (Algorithm 3 resets every
 *                worker to the trainer's parameters at the next outer step)
 * The K differences (each exact in fp64) are summed in fp64 in the order k = 0..K-1 and the
 * update is carried in fp64; every output element is rounded to fp32 once. */
int adloco_outer_step(adloco_ctx* ctx, const void* const* inst_params, adloco_dtype inst_dtype, int32_t K,
                      int64_t P, const float* theta_in, float* theta_out, const float* mom_in, float* mom_out,
                      float lr, float momentum, int nesterov, void* const* inst_writeback, void* stream);

/* Same update with every buffer in HOST memory (inst_params_host: K host
 * pointers; theta_host and mom_host are updated in place): panels are staged
 * through device buffers the library owns, copies overlapped with the kernel.
 * Synchronous. */
int adloco_outer_step_host(adloco_ctx* ctx, const void* const* inst_params_host, adloco_dtype inst_dtype,
                           int32_t K, int64_t P, float* theta_host, float* mom_host, float lr, float momentum,
                           int nesterov, void* stream);

/* The outer step when every GPU holds ONE whole instance (and the shared starting point
 * theta) but only a slice of the momentum: the K pseudo-gradients are summed across the
 * GPUs by one reduce-scatter -- the single communication of the method (last loop of
 * Algorithm 3: the workers' differences are gathered and averaged) -- which the caller
 * performs between these calls, with whatever collective library it uses:
 *   1. adloco_pseudo_gradient    pseudo_grad = theta - theta_k, fp32 [P]      (every rank)
 *   2. reduce-scatter (sum) of pseudo_grad over the K ranks -> pseudo_grad_sum, this rank's slice
 *   3. adloco_outer_apply        d = pseudo_grad_sum / K; v' = momentum v + d;
 *                                u = d + momentum v' | v'; theta' = theta - lr u   (on the slice)
 *   4. all-gather of the theta' slices, then adloco_refresh_instance: theta_k = theta'
 *      rounded to the instance type (Algorithm 3 restarts every worker from theta).
 * All pointers dev, 16-byte aligned; theta/mom in and out may alias exactly.  The update is
 * carried in fp64 and rounded once, as in adloco_outer_step.  The K terms cross the exchange
 * as fp32 and are summed by the collective in fp32: against adloco_outer_step (which sums
 * them in fp64) the sum can be off by up to (K - 1/2) ulp of sum_k |theta - theta_k|, which
 * shows where the terms cancel and the update itself is small. */
int adloco_pseudo_gradient(adloco_ctx* ctx, const float* theta, const void* inst_params, adloco_dtype inst_dtype,
                           int64_t P, float* pseudo_grad, void* stream);
int adloco_outer_apply(adloco_ctx* ctx, const float* pseudo_grad_sum, int32_t K, int64_t P, const float* theta_in,
                       float* theta_out, const float* mom_in, float* mom_out, float lr, float momentum, int nesterov,
                       void* stream);
int adloco_refresh_instance(adloco_ctx* ctx, const float* theta, void* inst_params, adloco_dtype inst_dtype, int64_t P,
                            void* stream);

/* ---- trainer merge --------------------------------------------------------- */

/* CheckMerge (Algorithm 1), host only: writes into merge_idx (host, capacity >= w)
 * the indices of the w trainers with the smallest b_req (ties: lower index first)
 * and returns their number; 0 when w == 0, k <= 1 or w > k; negative status on
 * bad arguments. */
int adloco_check_merge(const int64_t* b_req, int32_t k, int32_t w, int32_t* merge_idx);

/* DoMerge (Algorithm 2): x_merge = sum_j b_j x_j / sum_j b_j over the K members
 * (HOST array of dev pointers, [P] each in `dtype`; weights HOST int64 > 0),
 * written to `out` (dev [P] in `dtype`; may be one of the members, exactly).
 * *rep (host, may be NULL) receives the member with the largest weight (lowest
 * index on ties), the trainer that is kept. 1 <= K <= 64. */
int adloco_merge(adloco_ctx* ctx, const void* const* members, const int64_t* weights, adloco_dtype dtype,
                 int32_t K, int64_t P, void* out, int32_t* rep, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ADLOCO_H */
