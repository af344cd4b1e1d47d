// HBM-streaming kernels: the one-pass norm test over materialised per-sample
// gradients (also the switch-mode accumulation step), the batch rule, the fused
// K-way pseudo-gradient average + momentum outer step, the weighted merge and
// the squared-norm reduction over gradient-sum buffers.
//
// All of them move each input byte from HBM once with 128-bit accesses; the
// arithmetic per byte is far below the machine balance, so grids are sized to
// a multiple of the SM count and the only tuning that matters is bytes in
// flight per SM.
#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace adloco {

constexpr int NT_THREADS = 256;
constexpr int NT_WARPS = NT_THREADS / 32;
constexpr int NT_CHUNK = 8;  // rows loaded back to back before they are consumed (4 and 16 measured slower)

// ---------------------------------------------------------------------------------
// small device helpers
// ---------------------------------------------------------------------------------
__device__ __forceinline__ float4 ld_stream4(const float* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}

// the two bfloat16 halves of a 32-bit word, widened exactly
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// up to four consecutive floats starting at p; lanes >= nvalid read as zero.
// VEC = false is the path for rows that do not start on a 16-byte boundary.
template <bool VEC = true>
__device__ __forceinline__ float4 load4(const float* p, int nvalid) {
    if (VEC && nvalid >= 4) return ld_stream4(p);
    if (!VEC && nvalid >= 4) return make_float4(__ldcs(p), __ldcs(p + 1), __ldcs(p + 2), __ldcs(p + 3));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (nvalid > 0) r.x = __ldcs(p);
    if (nvalid > 1) r.y = __ldcs(p + 1);
    if (nvalid > 2) r.z = __ldcs(p + 2);
    return r;
}

// the same for a row of bfloat16: 64-bit load when VEC (rows start on 8-byte boundaries)
template <bool VEC = true>
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p, int nvalid) {
    if (VEC && nvalid >= 4) {
        const uint2 w = __ldcs(reinterpret_cast<const uint2*>(p));
        return make_float4(bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y));
    }
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    const unsigned short* q = reinterpret_cast<const unsigned short*>(p);
    if (nvalid > 0) r.x = __uint_as_float((uint32_t)__ldcs(q) << 16);
    if (nvalid > 1) r.y = __uint_as_float((uint32_t)__ldcs(q + 1) << 16);
    if (nvalid > 2) r.z = __uint_as_float((uint32_t)__ldcs(q + 2) << 16);
    if (nvalid > 3) r.w = __uint_as_float((uint32_t)__ldcs(q + 3) << 16);
    return r;
}

template <bool VEC = true>
__device__ __forceinline__ void store4(float* p, float4 v, int nvalid) {
    if (VEC && nvalid >= 4) {
        *reinterpret_cast<float4*>(p) = v;
    } else if (nvalid >= 4) {
        p[0] = v.x; p[1] = v.y; p[2] = v.z; p[3] = v.w;
    } else {
        if (nvalid > 0) p[0] = v.x;
        if (nvalid > 1) p[1] = v.y;
        if (nvalid > 2) p[2] = v.z;
    }
}

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum of v over the block, fixed tree (deterministic); result valid in thread 0.
__device__ double block_sum(double v, double* smem /* >= 32 doubles */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        for (int w = 0; w < nw; ++w) t += smem[w];
    }
    return t;
}

// Reduces RB per-row accumulators across the 32 lanes of a warp with a halving
// exchange (about RB shuffles instead of 5*RB): at each step a lane keeps the
// half of its values selected by one bit of its lane index and receives the
// partner's sums for that half.
template <int RB, int STEP>
__device__ __forceinline__ void fold_step(float (&v)[RB], int lane) {
    if constexpr (STEP < 5) {
        constexpr int o = 16 >> STEP;
        constexpr int c = RB >> STEP;  // values a lane still holds before this step
        const bool upper = (lane & o) != 0;
        if constexpr (c >= 2) {
            constexpr int h = c / 2;
#pragma unroll
            for (int k = 0; k < h; ++k) {
                const float send = upper ? v[k] : v[k + h];
                const float keep = upper ? v[k + h] : v[k];
                v[k] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
        } else {
            v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
        }
        fold_step<RB, STEP + 1>(v, lane);
    }
}

// Adds the warp totals of the RB rows into dst[0..RB).  After the fold, lane l
// holds rows l*RB/32 .. (RB >= 32), or row l/(32/RB) shared by 32/RB lanes.
template <int RB>
__device__ __forceinline__ void warp_rows_flush(float (&v)[RB], float* dst, int lane) {
    fold_step<RB, 0>(v, lane);
    if constexpr (RB >= 32) {
        constexpr int per = RB / 32;
#pragma unroll
        for (int j = 0; j < per; ++j) dst[lane * per + j] += v[j];
    } else {
        constexpr int share = 32 / RB;
        if ((lane % share) == 0) dst[lane / share] += v[0];
    }
}

// ---------------------------------------------------------------------------------
// batch rule + switch plan (Section "Norm test", Section "Mode switching")
// ---------------------------------------------------------------------------------
// `mirror`, when given, is the caller's page-locked host copy of the result: the deciding thread stores
// there too, which spares the stream a device-to-host copy between two kernels (about 11 us per call).
__device__ void decide_device(const adloco_test_sums& s, const adloco_test_params& p, adloco_test_result* out,
                              adloco_test_result* mirror = nullptr) {
    adloco_test_result r;
    const int64_t b = s.batch_count;
    const double bd = (double)b;
    r.sum_sqnorm = s.sum_sqnorm;
    r.mean_sqnorm = (b > 0) ? s.sum_sq_gsum / (bd * bd) : 0.0;
    r.batch_count = b;
    r.flags = 0;
    r.device_status = s.device_status;
    const int64_t i64max = 0x7fffffffffffffffLL;
    // an overflowed or NaN gradient anywhere poisons every sum: no statistic, the batch stays
    const bool finite = isfinite(s.sum_sqnorm) && isfinite(s.sum_sq_gsum) && (!s.has_centred || isfinite(s.centred_ss));
    if (!finite) {
        r.flags |= ADLOCO_FLAG_NONFINITE;
        r.variance = 0.0;
        r.stat = 0.0;
        r.b_req = p.b_cur > 1 ? p.b_cur : 1;
    } else if (b - p.ddof <= 0) {
        r.flags |= ADLOCO_FLAG_UNDEFINED;
        r.variance = 0.0;
        r.stat = 0.0;
        r.b_req = p.b_cur > 1 ? p.b_cur : 1;
    } else {
        const double denom = (double)(b - p.ddof);
        r.variance = s.has_centred ? s.centred_ss / denom : (s.sum_sqnorm - bd * r.mean_sqnorm) / denom;
        if (r.mean_sqnorm == 0.0) {
            r.flags |= ADLOCO_FLAG_ZERO_MEAN;
            r.stat = __longlong_as_double(0x7ff0000000000000LL);
            r.b_req = p.b_cap > 0 ? p.b_cap : i64max;
        } else {
            r.stat = r.variance / (p.eta * p.eta * r.mean_sqnorm);
            if (r.stat < 9.0e18) {
                const int64_t c = (int64_t)ceil(r.stat);
                r.b_req = c > 1 ? c : 1;
            } else {
                r.b_req = i64max;
            }
        }
    }
    if (p.b_cap > 0 && r.b_req > p.b_cap) r.b_req = p.b_cap;
    if (r.b_req > p.b_cur) r.flags |= ADLOCO_FLAG_GROW;
    // switch mode: accumulate only beyond switch_n * b_max (compare by division: no overflow)
    if (r.b_req / p.b_max > p.switch_n || (r.b_req / p.b_max == p.switch_n && r.b_req % p.b_max != 0)) {
        r.flags |= ADLOCO_FLAG_ACCUMULATE;
        r.accum_steps = r.b_req / p.b_max + (r.b_req % p.b_max != 0 ? 1 : 0);
        r.b_micro = p.b_max;
    } else {
        r.accum_steps = 1;
        r.b_micro = r.b_req < p.b_max ? r.b_req : p.b_max;
    }
    *out = r;
    if (mirror != nullptr) {
        *mirror = r;
        __threadfence_system();
    }
}

__global__ void decide_kernel(const adloco_test_sums* sums, adloco_test_params p, adloco_test_result* out,
                              adloco_test_result* mirror) {
    if (threadIdx.x == 0 && blockIdx.x == 0) decide_device(*sums, p, out, mirror);
}

// Last block of a reduction: the total over all blocks of the per-block partial sums of 32
// rows, rows i0 .. i0 + 31.  Warp w adds up blocks w, w + 8, ... for row i0 + lane -- its loads
// are independent and in flight together, where one thread walking all blocks of a row took
// a tenth of a 100 us launch -- and the eight warp sums are added in warp order: the order is
// fixed, so the result is the same on every run.  Called by all threads of the block;
// returns the total of row i0 + lane in warp 0 (garbage elsewhere and for rows >= B).
__device__ __forceinline__ double combine_rows32(const float* partials, int64_t B, unsigned nblk, int64_t i0,
                                                 double (&comb)[NT_WARPS][32]) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t i = i0 + lane;
    double t = 0.0;
    if (i < B) {
        unsigned blk = warp;
        for (; blk + 7 * NT_WARPS < nblk; blk += 8 * NT_WARPS) {
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = __ldcg(partials + (int64_t)(blk + u * NT_WARPS) * B + i);
#pragma unroll
            for (int u = 0; u < 8; ++u) t += (double)v[u];
        }
        for (; blk < nblk; blk += NT_WARPS) t += (double)__ldcg(partials + (int64_t)blk * B + i);
    }
    comb[warp][lane] = t;
    __syncthreads();
    double r = 0.0;
    if (warp == 0) {
#pragma unroll
        for (int w = 0; w < NT_WARPS; ++w) r += comb[w][lane];
    }
    __syncthreads();
    return r;
}

// ---------------------------------------------------------------------------------
// one-pass norm test
// ---------------------------------------------------------------------------------
struct NtArgs {
    const float* G;
    int64_t B, P, stride;
    float* n_out;
    float* S;
    adloco_test_sums* sums;
    adloco_test_result* result;
    adloco_test_result* result_mirror;   // page-locked host copy the last block also writes, or null
    adloco_test_params params;
    float* n_partials;
    double* blk_scalars;
    unsigned* ticket;
    int mode, n_accum, first_panel, iters;
};

// One tile of RB rows of a thread's four columns: CH rows are loaded back to back, then
// consumed.  CHECKED = false is the path of a full tile of full column groups -- plain
// vector loads and straight-line arithmetic, nothing predicated: with the row and column
// guards in the loop the compiler cannot keep the CH loads of a chunk in flight together,
// which costs a tenth of the bandwidth at full clock and a quarter at a power-capped one.
template <int RB, int CH, bool VEC, bool CHECKED, typename elem_t>
__device__ __forceinline__ void nt_row_tile(const elem_t* rowp, int64_t stride, int64_t rows_left, int nvalid, bool first_tile,
                                            float4& c, float4& sd, float4& sdd, float (&acc)[RB]) {
#pragma unroll
    for (int r0 = 0; r0 < RB; r0 += CH) {
        float4 x[CH];
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            if (CHECKED) x[u] = load4<VEC>(rowp + (int64_t)(r0 + u) * stride, (r0 + u) < rows_left ? nvalid : 0);
            else x[u] = load4<VEC>(rowp + (int64_t)(r0 + u) * stride, 4);
        }
        if (r0 == 0 && first_tile) c = x[0];
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            if (!CHECKED || (r0 + u) < rows_left) {
                const float4 v = x[u];
                float q = v.x * v.x;
                q = fmaf(v.y, v.y, q);
                q = fmaf(v.z, v.z, q);
                q = fmaf(v.w, v.w, q);
                acc[r0 + u] += q;
                const float dx = v.x - c.x, dy = v.y - c.y, dz = v.z - c.z, dw = v.w - c.w;
                sd.x += dx; sd.y += dy; sd.z += dz; sd.w += dw;
                sdd.x = fmaf(dx, dx, sdd.x); sdd.y = fmaf(dy, dy, sdd.y);
                sdd.z = fmaf(dz, dz, sdd.z); sdd.w = fmaf(dw, dw, sdd.w);
            }
        }
    }
}

// Thread t of a block owns one group of four adjacent columns per iteration and
// walks down all B rows of it: per column it keeps the sum and the sum of
// squares of (G_ij - G_0j) -- shifting by the first row removes the mean before
// squaring, so the centred sum of squares comes out without cancellation -- and
// per row the running sum of squares (RB registers, rows tiled by RB).
// MICRO = switch-mode accumulation (a.mode == NT_MICRO), an instantiation of its own: the running sums it
// fetches and the term of the pairwise update cost registers that the one-shot form, at 64 rows per thread,
// does not have (with them in, the row loop spilled and ran 9 % slower, 14 % under the power cap).
template <int RB, bool VEC, bool BF16 = false, bool MICRO = false>
__global__ void __launch_bounds__(NT_THREADS, RB <= 8 ? 4 : 2) norm_test_kernel(const __grid_constant__ NtArgs a) {
    using elem_t = typename std::conditional<BF16, __nv_bfloat16, float>::type;
    constexpr int CH = RB < NT_CHUNK ? RB : NT_CHUNK;   // rows loaded back to back
    extern __shared__ float smem_rows[];  // [NT_WARPS][Bpad]
    __shared__ double smem_red[32];
    __shared__ int smem_is_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t B = a.B;
    const int Bpad = (int)(((B + RB - 1) / RB) * RB);
    for (int i = tid; i < NT_WARPS * Bpad; i += NT_THREADS) smem_rows[i] = 0.f;
    __syncthreads();
    float* my_rows = smem_rows + warp * Bpad;

    const int64_t ngroups = (a.P + 3) >> 2;
    const bool single_tile = (B <= RB);
    const float Bf = (float)B;
    const float invB = 1.0f / Bf;
    // switch-mode accumulation: samples already accumulated before this micro-batch
    const double c_prev_d = MICRO ? (double)a.sums->batch_count : 0.0;
    const float inv_cprev = c_prev_d > 0.0 ? (float)(1.0 / c_prev_d) : 0.f;

    float acc[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) acc[r] = 0.f;

    // per-thread fp64 running sums live in shared memory (touched once per 16 column groups): as registers
    // they pushed the 64-row instantiation into spilling inside the row loop
    __shared__ double smem_run[3][NT_THREADS];
    smem_run[0][tid] = 0.0; smem_run[1][tid] = 0.0; smem_run[2][tid] = 0.0;
    float f_sumsq = 0.f, f_css = 0.f, f_chan = 0.f;

    for (int it = 0; it < a.iters; ++it) {
        const int64_t g = ((int64_t)it * gridDim.x + blockIdx.x) * NT_THREADS + tid;
        const int64_t col = g << 2;
        int nvalid = 0;
        if (g < ngroups) nvalid = (a.P - col) >= 4 ? 4 : (int)(a.P - col);
        const elem_t* rowp = reinterpret_cast<const elem_t*>(a.G) + (nvalid > 0 ? col : 0);

        float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
        float4 sd = c, sdd = c;
        // switch mode: the sums so far are fetched now, so that their latency hides behind the rows
        float4 so = make_float4(0.f, 0.f, 0.f, 0.f);
        if (MICRO && nvalid > 0) so = load4<VEC>(a.S + col, nvalid);
        for (int64_t i0 = 0; i0 < B; i0 += RB) {
            if (nvalid == 4 && i0 + RB <= B)
                nt_row_tile<RB, CH, VEC, false>(rowp, a.stride, RB, 4, i0 == 0, c, sd, sdd, acc);
            else
                nt_row_tile<RB, CH, VEC, true>(rowp, a.stride, B - i0, nvalid, i0 == 0, c, sd, sdd, acc);
            rowp += (int64_t)RB * a.stride;
            if (!single_tile) {
                warp_rows_flush<RB>(acc, my_rows + i0, lane);
#pragma unroll
                for (int r = 0; r < RB; ++r) acc[r] = 0.f;
            }
        }

        // per-column results of this group
        float4 s;  // column sums over the B rows
        s.x = fmaf(Bf, c.x, sd.x); s.y = fmaf(Bf, c.y, sd.y); s.z = fmaf(Bf, c.z, sd.z); s.w = fmaf(Bf, c.w, sd.w);
        f_css += (sdd.x - sd.x * sd.x * invB) + (sdd.y - sd.y * sd.y * invB) +
                 (sdd.z - sd.z * sd.z * invB) + (sdd.w - sd.w * sd.w * invB);
        if (MICRO) {
            // pairwise (Chan) update of the centred sum of squares needs ||mean_mb - mean_prev||^2
            const float ex = s.x * invB - so.x * inv_cprev, ey = s.y * invB - so.y * inv_cprev;
            const float ez = s.z * invB - so.z * inv_cprev, ew = s.w * invB - so.w * inv_cprev;
            f_chan += ex * ex + ey * ey + ez * ez + ew * ew;
            s.x += so.x; s.y += so.y; s.z += so.z; s.w += so.w;
            if (nvalid > 0) store4<VEC>(a.S + col, s, nvalid);
        } else if (a.S != nullptr && nvalid > 0) {
            store4<VEC>(a.S + col, s, nvalid);
        }
        f_sumsq += s.x * s.x + s.y * s.y + s.z * s.z + s.w * s.w;
        if ((it & 15) == 15) {  // bound the length of the fp32 running sums
            smem_run[0][tid] += (double)f_sumsq; smem_run[1][tid] += (double)f_css;
            if (MICRO) smem_run[2][tid] += (double)f_chan;
            f_sumsq = f_css = f_chan = 0.f;
        }
    }
    const double t_sumsq = smem_run[0][tid] + (double)f_sumsq, t_css = smem_run[1][tid] + (double)f_css;
    const double t_chan = smem_run[2][tid] + (double)f_chan;
    if (single_tile) warp_rows_flush<RB>(acc, my_rows, lane);

    // block partials
    const double b_sumsq = block_sum(t_sumsq, smem_red);
    const double b_css = block_sum(t_css, smem_red);
    const double b_chan = block_sum(t_chan, smem_red);
    __syncthreads();
    for (int64_t i = tid; i < B; i += NT_THREADS) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < NT_WARPS; ++w) t += smem_rows[w * Bpad + i];
        a.n_partials[(int64_t)blockIdx.x * B + i] = t;
    }
    if (tid == 0) {
        double* bs = a.blk_scalars + (int64_t)blockIdx.x * 4;
        bs[0] = b_sumsq; bs[1] = b_css; bs[2] = b_chan;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(a.ticket, 1u);
        smem_is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!smem_is_last) return;
    __threadfence();

    // last block: combine all partials in a fixed order, in fp64
    __shared__ double smem_comb[NT_WARPS][32];
    double q_local = 0.0;
    for (int64_t i0 = 0; i0 < B; i0 += 32) {
        const double t = combine_rows32(a.n_partials, B, gridDim.x, i0, smem_comb);
        const int64_t i = i0 + lane;
        if (warp == 0 && i < B) {
            if (a.n_out != nullptr) a.n_out[i] = a.n_accum ? a.n_out[i] + (float)t : (float)t;
            q_local += t;
        }
    }
    double p0 = 0.0, p1 = 0.0, p2 = 0.0;
    for (unsigned blk = tid; blk < gridDim.x; blk += NT_THREADS) {
        p0 += __ldcg(a.blk_scalars + (int64_t)blk * 4 + 0);
        p1 += __ldcg(a.blk_scalars + (int64_t)blk * 4 + 1);
        p2 += __ldcg(a.blk_scalars + (int64_t)blk * 4 + 2);
    }
    const double Q = block_sum(q_local, smem_red);
    const double sumsq = block_sum(p0, smem_red);
    const double css = block_sum(p1, smem_red);
    const double chan = block_sum(p2, smem_red);
    if (tid == 0) {
        adloco_test_sums s = *a.sums;
        if (a.mode == NT_ONESHOT || (a.mode == NT_PANEL && a.first_panel)) {
            s.sum_sqnorm = Q; s.sum_sq_gsum = sumsq; s.centred_ss = css;
            s.batch_count = B; s.has_centred = 1; s.device_status = 0;
        } else if (a.mode == NT_PANEL) {
            s.sum_sqnorm += Q; s.sum_sq_gsum += sumsq; s.centred_ss += css;
        } else {  // NT_MICRO: rows are appended
            const double cp = (double)s.batch_count, bb = (double)B;
            s.centred_ss += css + (cp > 0.0 ? (cp * bb / (cp + bb)) * chan : 0.0);
            // the centred sum stays valid while every micro-batch so far came materialised
            if (cp == 0.0) s.has_centred = 1;
            s.sum_sqnorm += Q;
            s.sum_sq_gsum = sumsq;  // ||S||^2 of the updated sum buffer
            s.batch_count += B;
        }
        *a.sums = s;
        if (a.result != nullptr) decide_device(s, a.params, a.result, a.result_mirror);
        *a.ticket = 0u;
    }
}

// The workspace is sized at creation for the largest launch, so this never allocates in
// practice; it stays as the guard for a device with more resident blocks per SM than assumed.
static int grow_workspace(adloco_ctx* ctx, size_t need_elems) {
    if (need_elems <= ctx->n_partials_elems) return ADLOCO_OK;
    if (ctx->n_partials) {
        ADLOCO_CUDA_TRY(ctx, cudaDeviceSynchronize());
        ADLOCO_CUDA_TRY(ctx, cudaFree(ctx->n_partials));
        ctx->n_partials = nullptr;
        ctx->n_partials_elems = 0;
    }
    ADLOCO_CUDA_TRY(ctx, cudaMalloc(&ctx->n_partials, need_elems * sizeof(float)));
    ctx->n_partials_elems = need_elems;
    return ADLOCO_OK;
}

template <int RB, bool VEC, bool BF16, bool MICRO>
static int launch_nt(adloco_ctx* ctx, const NtLaunch& l, cudaStream_t st) {
    const int64_t ngroups = (l.P + 3) / 4;
    const int64_t tiles = (ngroups + NT_THREADS - 1) / NT_THREADS;
    const int Bpad = (int)(((l.B + RB - 1) / RB) * RB);
    const size_t smem = (size_t)NT_WARPS * Bpad * sizeof(float);
    auto kern = norm_test_kernel<RB, VEC, BF16, MICRO>;
    if (smem > 48 * 1024) ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // resident blocks per SM for this instantiation and shared-memory size (asked once)
    static std::mutex cache_mutex;            // contexts on different host threads share these statics
    static size_t cached_smem = ~(size_t)0;
    static int cached_per_sm = 0;
    int per_sm;
    {
        std::lock_guard<std::mutex> lock(cache_mutex);
        if (cached_smem != smem) {
            int q = 0;
            ADLOCO_CUDA_TRY(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&q, kern, NT_THREADS, smem));
            cached_per_sm = q;
            cached_smem = smem;
        }
        per_sm = cached_per_sm;
    }
    if (per_sm < 1) return ADLOCO_ERR_WORKSPACE;
    int64_t max_grid = (int64_t)ctx->sm_count * per_sm;
    if (max_grid > ctx->max_grid) max_grid = ctx->max_grid;
    // equal work per block: iters passes over a grid that just covers the tiles
    const int64_t iters = (tiles + max_grid - 1) / max_grid;
    const int64_t grid = (tiles + iters - 1) / iters;
    int rc = grow_workspace(ctx, (size_t)grid * (size_t)l.B);
    if (rc != ADLOCO_OK) return rc;

    NtArgs a;
    a.G = l.G; a.B = l.B; a.P = l.P; a.stride = l.stride;
    a.n_out = l.n_out; a.S = l.S; a.sums = l.sums; a.result = l.result; a.result_mirror = l.result_mirror; a.params = l.params;
    a.n_partials = ctx->n_partials; a.blk_scalars = ctx->blk_scalars; a.ticket = ctx->ticket;
    a.mode = l.mode; a.n_accum = l.n_accum; a.first_panel = l.first_panel; a.iters = (int)iters;
    kern<<<(unsigned)grid, NT_THREADS, smem, st>>>(a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_norm_test(adloco_ctx* ctx, const NtLaunch& l, cudaStream_t st) {
    // vector loads need every row to start on a 16-byte (fp32) or 8-byte (bf16) boundary, S on 16
    const uintptr_t row_align = l.bf16 ? 7u : 15u;
    const bool vec = (reinterpret_cast<uintptr_t>(l.G) & row_align) == 0 && (l.B == 1 || (l.stride % 4) == 0) &&
                     (l.S == nullptr || aligned16(l.S));
#define ADLOCO_NT_DISPATCH(V, H, M)                                      \
    do {                                                                 \
        if (l.B <= 4) return launch_nt<4, V, H, M>(ctx, l, st);          \
        if (l.B <= 8) return launch_nt<8, V, H, M>(ctx, l, st);          \
        if (l.B <= 16) return launch_nt<16, V, H, M>(ctx, l, st);        \
        if (l.B <= 32) return launch_nt<32, V, H, M>(ctx, l, st);        \
        return launch_nt<64, V, H, M>(ctx, l, st);                       \
    } while (0)
    if (l.mode == NT_MICRO) {
        if (l.bf16) { if (vec) ADLOCO_NT_DISPATCH(true, true, true); else ADLOCO_NT_DISPATCH(false, true, true); }
        if (vec) ADLOCO_NT_DISPATCH(true, false, true); else ADLOCO_NT_DISPATCH(false, false, true);
    }
    if (l.bf16) { if (vec) ADLOCO_NT_DISPATCH(true, true, false); else ADLOCO_NT_DISPATCH(false, true, false); }
    if (vec) ADLOCO_NT_DISPATCH(true, false, false); else ADLOCO_NT_DISPATCH(false, false, false);
#undef ADLOCO_NT_DISPATCH
}

int launch_decide(adloco_ctx* ctx, const adloco_test_sums* sums, const adloco_test_params& p,
                  adloco_test_result* result, adloco_test_result* mirror, cudaStream_t st) {
    decide_kernel<<<1, 32, 0, st>>>(sums, p, result, mirror);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// inner-product tests: second pass over G with the gradient sum S of the first
// ---------------------------------------------------------------------------------
struct IpArgs {
    const float* G;
    const float* S;            // [P] sum of the rows of G (adloco_norm_test's grad_sum)
    int64_t B, P, stride;
    const adloco_test_sums* sums;   // of the norm test on the same G
    adloco_ip_params params;
    float* dots_out;           // [B] <g_i, gbar>, may be null
    adloco_ip_result* result;
    adloco_ip_result* result_mirror;   // page-locked host copy, or null
    float* n_partials;
    unsigned* ticket;
    int iters;
};

// Batch rules of the inner-product test and its augmented form from
//   d_i = <g_i, gbar> - ||gbar||^2 (i = 0..b-1, their sum of squares and mean given),
//   css = sum_i ||g_i - gbar||^2,  N = ||gbar||^2:
//   Var_i <g_i, gbar> = sum (d_i - dbar)^2 / (b - ddof)
//   the parts of the g_i orthogonal to gbar have mean zero and
//   sum_i ||o_i||^2 = css - sum_i d_i^2 / N.
__device__ void ip_decide_device(double sum_d2, double sum_d, const adloco_test_sums& s, const adloco_ip_params& p,
                                 adloco_ip_result* out) {
    adloco_ip_result r;
    const int64_t b = s.batch_count;
    const double bd = (double)b;
    const double N = b > 0 ? s.sum_sq_gsum / (bd * bd) : 0.0;
    const int64_t i64max = 0x7fffffffffffffffLL;
    r.mean_sqnorm = N;
    r.batch_count = b;
    r.flags = 0;
    r.device_status = s.device_status;
    r.var_ip = r.stat_ip = r.var_orth = r.stat_orth = 0.0;
    const bool finite = isfinite(sum_d2) && isfinite(sum_d) && isfinite(s.sum_sqnorm) && isfinite(s.sum_sq_gsum) &&
                        (!s.has_centred || isfinite(s.centred_ss));
    if (!finite) {
        r.flags |= ADLOCO_FLAG_NONFINITE;
        r.b_ip = r.b_aug = p.b_cur > 1 ? p.b_cur : 1;
    } else if (b - p.ddof <= 0) {
        r.flags |= ADLOCO_FLAG_UNDEFINED;
        r.b_ip = r.b_aug = p.b_cur > 1 ? p.b_cur : 1;
    } else if (N == 0.0) {
        r.flags |= ADLOCO_FLAG_ZERO_MEAN;
        r.stat_ip = r.stat_orth = __longlong_as_double(0x7ff0000000000000LL);
        r.b_ip = r.b_aug = p.b_cap > 0 ? p.b_cap : i64max;
    } else {
        const double denom = (double)(b - p.ddof);
        double centred = sum_d2 - sum_d * sum_d / bd;
        if (centred < 0.0) centred = 0.0;
        r.var_ip = centred / denom;
        r.stat_ip = r.var_ip / (p.theta * p.theta * N * N);
        const double css = s.has_centred ? s.centred_ss : s.sum_sqnorm - bd * N;
        double orth = css - sum_d2 / N;
        if (orth < 0.0) orth = 0.0;
        r.var_orth = orth / denom;
        r.stat_orth = r.var_orth / (p.nu * p.nu * N);
        const int64_t c_ip = r.stat_ip < 9.0e18 ? (int64_t)ceil(r.stat_ip) : i64max;
        const int64_t c_or = r.stat_orth < 9.0e18 ? (int64_t)ceil(r.stat_orth) : i64max;
        r.b_ip = c_ip > 1 ? c_ip : 1;
        r.b_aug = c_or > r.b_ip ? c_or : r.b_ip;
    }
    if (p.b_cap > 0) {
        if (r.b_ip > p.b_cap) r.b_ip = p.b_cap;
        if (r.b_aug > p.b_cap) r.b_aug = p.b_cap;
    }
    if (r.b_aug > p.b_cur) r.flags |= ADLOCO_FLAG_GROW;
    *out = r;
}

// Thread layout as in norm_test_kernel: a thread owns four adjacent columns, loads
// their entries of S once and walks down the rows accumulating, per row,
// sum_j (G_ij - S_j / b) S_j = b (<g_i, gbar> - ||gbar||^2): centring before the
// product keeps the small deviation d_i free of cancellation.
// One tile of RB rows for the inner-product pass, as nt_row_tile does for the norm test: CHECKED = false
// (a full tile of a full column group) has no guards, so a chunk's loads stay in flight together.
template <int RB, int CH, bool VEC, bool CHECKED, typename elem_t>
__device__ __forceinline__ void ip_row_tile(const elem_t* rowp, int64_t stride, int64_t rows_left, int nvalid,
                                            float invB, const float4& s4, float (&acc)[RB]) {
    float4 m4;
#pragma unroll
    for (int r0 = 0; r0 < RB; r0 += CH) {
        float4 x[CH];
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            if (CHECKED) x[u] = load4<VEC>(rowp + (int64_t)(r0 + u) * stride, (r0 + u) < rows_left ? nvalid : 0);
            else x[u] = load4<VEC>(rowp + (int64_t)(r0 + u) * stride, 4);
        }
        // the column means are formed from the sums only now: a use of s4 ahead of the first chunk's loads
        // would hold those loads back by one memory round trip
        if (r0 == 0) m4 = make_float4(s4.x * invB, s4.y * invB, s4.z * invB, s4.w * invB);
#pragma unroll
        for (int u = 0; u < CH; ++u) {
            if (!CHECKED || (r0 + u) < rows_left) {
                // columns beyond P carry s4 = 0 and add nothing
                float q = (x[u].x - m4.x) * s4.x;
                q = fmaf(x[u].y - m4.y, s4.y, q);
                q = fmaf(x[u].z - m4.z, s4.z, q);
                q = fmaf(x[u].w - m4.w, s4.w, q);
                acc[r0 + u] += q;
            }
        }
    }
}

template <int RB, bool VEC, bool BF16 = false>
__global__ void __launch_bounds__(NT_THREADS, RB <= 8 ? 4 : 2) centred_dot_kernel(const __grid_constant__ IpArgs a) {
    using elem_t = typename std::conditional<BF16, __nv_bfloat16, float>::type;
    constexpr int CH = RB < NT_CHUNK ? RB : NT_CHUNK;   // rows loaded back to back
    extern __shared__ float smem_rows[];  // [NT_WARPS][Bpad]
    __shared__ double smem_red[32];
    __shared__ int smem_is_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t B = a.B;
    const int Bpad = (int)(((B + RB - 1) / RB) * RB);
    for (int i = tid; i < NT_WARPS * Bpad; i += NT_THREADS) smem_rows[i] = 0.f;
    __syncthreads();
    float* my_rows = smem_rows + warp * Bpad;
    const int64_t ngroups = (a.P + 3) >> 2;
    const bool single_tile = (B <= RB);
    const float invB = 1.0f / (float)B;

    float acc[RB];
#pragma unroll
    for (int r = 0; r < RB; ++r) acc[r] = 0.f;

    for (int it = 0; it < a.iters; ++it) {
        const int64_t g = ((int64_t)it * gridDim.x + blockIdx.x) * NT_THREADS + tid;
        const int64_t col = g << 2;
        int nvalid = 0;
        if (g < ngroups) nvalid = (a.P - col) >= 4 ? 4 : (int)(a.P - col);
        const elem_t* rowp = reinterpret_cast<const elem_t*>(a.G) + (nvalid > 0 ? col : 0);
        const float4 s4 = load4<VEC>(a.S + (nvalid > 0 ? col : 0), nvalid);
        for (int64_t i0 = 0; i0 < B; i0 += RB) {
            if (nvalid == 4 && i0 + RB <= B)
                ip_row_tile<RB, CH, VEC, false>(rowp, a.stride, RB, 4, invB, s4, acc);
            else
                ip_row_tile<RB, CH, VEC, true>(rowp, a.stride, B - i0, nvalid, invB, s4, acc);
            rowp += (int64_t)RB * a.stride;
            if (!single_tile) {
                warp_rows_flush<RB>(acc, my_rows + i0, lane);
#pragma unroll
                for (int r = 0; r < RB; ++r) acc[r] = 0.f;
            }
        }
    }
    if (single_tile) warp_rows_flush<RB>(acc, my_rows, lane);
    __syncthreads();
    for (int64_t i = tid; i < B; i += NT_THREADS) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < NT_WARPS; ++w) t += smem_rows[w * Bpad + i];
        a.n_partials[(int64_t)blockIdx.x * B + i] = t;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) smem_is_last = (atomicAdd(a.ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!smem_is_last) return;
    __threadfence();

    // last block: d_i in fp64, fixed order
    const adloco_test_sums s = *a.sums;
    const double bd = (double)B;
    const double N = s.sum_sq_gsum / (bd * bd);
    __shared__ double smem_comb[NT_WARPS][32];
    double l_d2 = 0.0, l_d = 0.0;
    for (int64_t i0 = 0; i0 < B; i0 += 32) {
        const double t = combine_rows32(a.n_partials, B, gridDim.x, i0, smem_comb);
        const int64_t i = i0 + (tid & 31);
        if ((tid >> 5) == 0 && i < B) {
            const double d = t / bd;
            if (a.dots_out != nullptr) a.dots_out[i] = (float)(N + d);
            l_d2 += d * d;
            l_d += d;
        }
    }
    const double sum_d2 = block_sum(l_d2, smem_red);
    const double sum_d = block_sum(l_d, smem_red);
    if (tid == 0) {
        ip_decide_device(sum_d2, sum_d, s, a.params, a.result);
        if (a.result_mirror != nullptr) {
            *a.result_mirror = *a.result;
            __threadfence_system();
        }
        *a.ticket = 0u;
    }
}

template <int RB, bool VEC, bool BF16>
static int launch_ip_t(adloco_ctx* ctx, const IpLaunch& l, cudaStream_t st) {
    const int64_t ngroups = (l.P + 3) / 4;
    const int64_t tiles = (ngroups + NT_THREADS - 1) / NT_THREADS;
    const int Bpad = (int)(((l.B + RB - 1) / RB) * RB);
    const size_t smem = (size_t)NT_WARPS * Bpad * sizeof(float);
    auto kern = centred_dot_kernel<RB, VEC, BF16>;
    if (smem > 48 * 1024) ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    // resident blocks per SM for this instantiation and shared-memory size (asked once)
    static std::mutex cache_mutex;            // contexts on different host threads share these statics
    static size_t cached_smem = ~(size_t)0;
    static int cached_per_sm = 0;
    int per_sm;
    {
        std::lock_guard<std::mutex> lock(cache_mutex);
        if (cached_smem != smem) {
            int q = 0;
            ADLOCO_CUDA_TRY(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&q, kern, NT_THREADS, smem));
            cached_per_sm = q;
            cached_smem = smem;
        }
        per_sm = cached_per_sm;
    }
    if (per_sm < 1) return ADLOCO_ERR_WORKSPACE;
    int64_t max_grid = (int64_t)ctx->sm_count * per_sm;
    if (max_grid > ctx->max_grid) max_grid = ctx->max_grid;
    const int64_t iters = (tiles + max_grid - 1) / max_grid;
    const int64_t grid = (tiles + iters - 1) / iters;
    int rc = grow_workspace(ctx, (size_t)grid * (size_t)l.B);
    if (rc != ADLOCO_OK) return rc;
    IpArgs a;
    a.G = l.G; a.S = l.S; a.B = l.B; a.P = l.P; a.stride = l.stride; a.sums = l.sums; a.params = l.params;
    a.dots_out = l.dots_out; a.result = l.result; a.result_mirror = l.result_mirror;
    a.n_partials = ctx->n_partials; a.ticket = ctx->ticket; a.iters = (int)iters;
    kern<<<(unsigned)grid, NT_THREADS, smem, st>>>(a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_inner_product(adloco_ctx* ctx, const IpLaunch& l, cudaStream_t st) {
    const uintptr_t row_align = l.bf16 ? 7u : 15u;
    const bool vec = (reinterpret_cast<uintptr_t>(l.G) & row_align) == 0 && aligned16(l.S) &&
                     (l.B == 1 || (l.stride % 4) == 0);
#define ADLOCO_IP_DISPATCH(V, H)                                         \
    do {                                                                 \
        if (l.B <= 4) return launch_ip_t<4, V, H>(ctx, l, st);           \
        if (l.B <= 8) return launch_ip_t<8, V, H>(ctx, l, st);           \
        if (l.B <= 16) return launch_ip_t<16, V, H>(ctx, l, st);         \
        if (l.B <= 32) return launch_ip_t<32, V, H>(ctx, l, st);         \
        return launch_ip_t<64, V, H>(ctx, l, st);                        \
    } while (0)
    if (l.bf16) { if (vec) ADLOCO_IP_DISPATCH(true, true); else ADLOCO_IP_DISPATCH(false, true); }
    if (vec) ADLOCO_IP_DISPATCH(true, false); else ADLOCO_IP_DISPATCH(false, false);
#undef ADLOCO_IP_DISPATCH
}

// ---------------------------------------------------------------------------------
// vector parameters (bias, elementwise gain): g_i = sum_t delta_t (* x_t)
// ---------------------------------------------------------------------------------
struct VecParamArgs {
    const __nv_bfloat16* D;
    const __nv_bfloat16* X;   // null for a bias
    int64_t T, d;
    float* n;                 // [B], +=
    float* S;                 // [d], += ; may be null
};

// Block (f, i) owns 256 adjacent features of sample i: a lane holds 8 of them (one
// 128-bit load per token row), the 8 warps share the tokens; the per-warp sums meet in
// shared memory, are squared into n_i and added into S.
constexpr int VP_WARPS = 16;
constexpr int VP_THREADS = 32 * VP_WARPS;

template <bool HAS_X>
__global__ void __launch_bounds__(VP_THREADS) vec_param_kernel(const VecParamArgs a) {
    __shared__ float part[VP_WARPS][257];
    __shared__ double red[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t i = blockIdx.y;
    const int64_t f0 = (int64_t)blockIdx.x * 256 + lane * 8;
    const bool live = f0 < a.d;                      // d is a multiple of 8
    const __nv_bfloat16* dp = a.D + (i * a.T) * a.d + f0;
    const __nv_bfloat16* xp = HAS_X ? a.X + (i * a.T) * a.d + f0 : nullptr;
    float acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    if (live) {
        // token rows in flight per warp: 8 (x 2 operands) for a gain, 4 for a bias (measured on [32,1024,3072]:
        // bias 5.30 / 5.41 / 4.86 / 5.00 TB/s with 2 / 4 / 8 / 16 rows)
        constexpr int U = HAS_X ? 8 : 4;
        for (int64_t t = warp; t < a.T; t += VP_WARPS * U) {
            uint4 dv[U], xv[U];
            if (t + (int64_t)(U - 1) * VP_WARPS < a.T) {
                // all U rows exist: plain loads, nothing guarded, so that they are in flight together
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int64_t tt = t + (int64_t)u * VP_WARPS;
                    dv[u] = __ldcs(reinterpret_cast<const uint4*>(dp + tt * a.d));
                    if (HAS_X) xv[u] = __ldcs(reinterpret_cast<const uint4*>(xp + tt * a.d));
                    else xv[u] = make_uint4(0, 0, 0, 0);
                }
            } else {
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int64_t tt = t + (int64_t)u * VP_WARPS;
                    dv[u] = make_uint4(0, 0, 0, 0);
                    xv[u] = make_uint4(0, 0, 0, 0);
                    if (tt < a.T) {
                        dv[u] = __ldcs(reinterpret_cast<const uint4*>(dp + tt * a.d));
                        if (HAS_X) xv[u] = __ldcs(reinterpret_cast<const uint4*>(xp + tt * a.d));
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const uint32_t dw[4] = {dv[u].x, dv[u].y, dv[u].z, dv[u].w};
                const uint32_t xw[4] = {xv[u].x, xv[u].y, xv[u].z, xv[u].w};
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    if (HAS_X) {
                        acc[2 * h] = fmaf(bf16_lo(dw[h]), bf16_lo(xw[h]), acc[2 * h]);
                        acc[2 * h + 1] = fmaf(bf16_hi(dw[h]), bf16_hi(xw[h]), acc[2 * h + 1]);
                    } else {
                        acc[2 * h] += bf16_lo(dw[h]);
                        acc[2 * h + 1] += bf16_hi(dw[h]);
                    }
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) part[warp][lane * 8 + e] = acc[e];
    __syncthreads();
    float g = 0.f;
    if (threadIdx.x < 256) {
#pragma unroll
        for (int w = 0; w < VP_WARPS; ++w) g += part[w][threadIdx.x];
    }
    const int64_t f = (int64_t)blockIdx.x * 256 + threadIdx.x;
    double sq = 0.0;
    if (threadIdx.x < 256 && f < a.d) {
        sq = (double)g * (double)g;
        if (a.S != nullptr) atomicAdd(a.S + f, g);
    }
    const double tot = block_sum(sq, red);
    if (threadIdx.x == 0) atomicAdd(a.n + i, (float)tot);
}

int launch_vec_param(adloco_ctx* ctx, const void* D, const void* X, int64_t B, int64_t T, int64_t d, float* n,
                     int accumulate_norms, float* S, int accumulate_sum, cudaStream_t st) {
    if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
    if (S && !accumulate_sum) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(S, 0, (size_t)d * sizeof(float), st));
    VecParamArgs a;
    a.D = static_cast<const __nv_bfloat16*>(D);
    a.X = static_cast<const __nv_bfloat16*>(X);
    a.T = T; a.d = d; a.n = n; a.S = S;
    const dim3 grid((unsigned)((d + 255) / 256), (unsigned)B);
    if (X) vec_param_kernel<true><<<grid, VP_THREADS, 0, st>>>(a);
    else vec_param_kernel<false><<<grid, VP_THREADS, 0, st>>>(a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// norm test without any allocation
// ---------------------------------------------------------------------------------
// Some callers cannot allocate device memory at the point where they need the
// test: a training step whose caching-allocator pool is frozen for the step, or
// a process that was handed a fixed device-memory budget and has spent it.  For them the reduction
// scratch of the norm test (per-block partial row sums, per-block scalars, the
// ticket counter and the sums record) lives in this file-scope device array
// instead of a context's workspace.  Every GPU that loads the library holds
// these bytes until the process exits.
constexpr int NA_MAX_ROWS = 64;      // largest B the entry point accepts
constexpr int NA_MAX_GRID = 1024;    // most blocks it ever launches
constexpr size_t NA_PARTIALS_BYTES = (size_t)NA_MAX_GRID * NA_MAX_ROWS * sizeof(float);   // 256 KB
constexpr size_t NA_SCALARS_BYTES = (size_t)NA_MAX_GRID * 4 * sizeof(double);             // 32 KB
constexpr size_t NA_TAIL_BYTES = 512;                                                      // ticket + sums
constexpr size_t NA_SCRATCH_BYTES = NA_PARTIALS_BYTES + NA_SCALARS_BYTES + NA_TAIL_BYTES;

static __device__ __align__(256) unsigned char g_noalloc_scratch[NA_SCRATCH_BYTES];

constexpr int NA_MAX_DEVICES = 64;
static void* g_noalloc_ptr[NA_MAX_DEVICES];   // device address of the array, per device; nullptr until set up
static int g_noalloc_sms[NA_MAX_DEVICES];

static std::mutex g_noalloc_mutex;

template <int RB, bool VEC>
static cudaError_t launch_nt_noalloc(const NtArgs& proto, int sm_count, cudaStream_t st) {
    NtArgs a = proto;
    const int64_t ngroups = (a.P + 3) / 4;
    const int64_t tiles = (ngroups + NT_THREADS - 1) / NT_THREADS;
    const int Bpad = (int)(((a.B + RB - 1) / RB) * RB);
    const size_t smem = (size_t)NT_WARPS * Bpad * sizeof(float);   // at most 2 KB here
    int64_t max_grid = (int64_t)sm_count * 2;
    if (max_grid > NA_MAX_GRID) max_grid = NA_MAX_GRID;
    const int64_t iters = (tiles + max_grid - 1) / max_grid;
    const int64_t grid = (tiles + iters - 1) / iters;
    a.iters = (int)iters;
    norm_test_kernel<RB, VEC><<<(unsigned)grid, NT_THREADS, smem, st>>>(a);
    return cudaGetLastError();
}

}  // namespace adloco

extern "C" __attribute__((visibility("default")))
int adloco_norm_test_noalloc(const float* grads, int64_t B, int64_t P, int64_t row_stride,
                             const adloco_test_params* params, float* per_sample_sqnorm,
                             adloco_test_result* result_dev, adloco_test_result* result_host, void* stream) {
    using namespace adloco;
    if (!grads || !result_dev || B < 1 || P < 1 || row_stride < P) return ADLOCO_ERR_INVALID_ARG;
    int rc = check_params(params);
    if (rc != ADLOCO_OK) return rc;
    if (B > NA_MAX_ROWS) return ADLOCO_ERR_UNSUPPORTED;   // the static scratch holds 64 rows per block
    if ((reinterpret_cast<uintptr_t>(grads) & 3u) != 0) return ADLOCO_ERR_ALIGNMENT;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return ADLOCO_ERR_CUDA;
    {
        // once per device, with that device current: the array's name is only a
        // host-side handle, the kernel needs the address the runtime maps it to
        std::lock_guard<std::mutex> lock(g_noalloc_mutex);
        if (g_noalloc_ptr[dev] == nullptr) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) return ADLOCO_ERR_CUDA;
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
                return ADLOCO_ERR_CUDA;
            g_noalloc_sms[dev] = sms;
            g_noalloc_ptr[dev] = ptr;
        }
    }
    unsigned char* base = static_cast<unsigned char*>(g_noalloc_ptr[dev]);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    NtArgs a;
    a.G = grads; a.B = B; a.P = P; a.stride = row_stride;
    a.n_out = per_sample_sqnorm; a.S = nullptr;
    a.n_partials = reinterpret_cast<float*>(base);
    a.blk_scalars = reinterpret_cast<double*>(base + NA_PARTIALS_BYTES);
    a.ticket = reinterpret_cast<unsigned*>(base + NA_PARTIALS_BYTES + NA_SCALARS_BYTES);
    a.sums = reinterpret_cast<adloco_test_sums*>(base + NA_PARTIALS_BYTES + NA_SCALARS_BYTES + 256);
    a.result = result_dev; a.result_mirror = nullptr; a.params = *params;
    a.mode = NT_ONESHOT; a.n_accum = 0; a.first_panel = 1; a.iters = 0;
    // the array keeps whatever the last call left: the ticket must start at zero
    if (cudaMemsetAsync(a.ticket, 0, NA_TAIL_BYTES, st) != cudaSuccess) return ADLOCO_ERR_CUDA;
    const bool vec = aligned16(grads) && (B == 1 || (row_stride % 4) == 0);
    cudaError_t e;
    const int sms = g_noalloc_sms[dev];
    if (vec) {
        e = B <= 16 ? launch_nt_noalloc<16, true>(a, sms, st)
          : B <= 32 ? launch_nt_noalloc<32, true>(a, sms, st) : launch_nt_noalloc<64, true>(a, sms, st);
    } else {
        e = B <= 16 ? launch_nt_noalloc<16, false>(a, sms, st)
          : B <= 32 ? launch_nt_noalloc<32, false>(a, sms, st) : launch_nt_noalloc<64, false>(a, sms, st);
    }
    if (e != cudaSuccess) return ADLOCO_ERR_CUDA;
    if (result_host &&
        cudaMemcpyAsync(result_host, result_dev, sizeof(adloco_test_result), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return ADLOCO_ERR_CUDA;
    return ADLOCO_OK;
}

namespace adloco {

// ---------------------------------------------------------------------------------
// outer step: K-way pseudo-gradient average + momentum update, one pass
// ---------------------------------------------------------------------------------
struct OuterArgs {
    const void* inst[kMaxInstances];
    void* wb[kMaxInstances];
    const float* th_in;
    float* th_out;
    const float* v_in;
    float* v_out;
    int64_t P;
    double invK;
    float lr, mu;
    int K, nesterov;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}

// The K differences theta - theta_k are summed in fp64: each difference is then
// exact and so is (to 2^-53) their sum, which cancels heavily when the instances
// scatter around theta.  The update itself is carried in fp64 as well and each
// output is rounded to fp32 once, so results sit within one rounding of the
// exact update for the fp32 lr and momentum given.
__device__ __forceinline__ void outer_update(float th, float v, double acc, const OuterArgs& a, float& th_new, float& v_new) {
    const double d = acc * a.invK;
    const double vn = fma((double)a.mu, (double)v, d);
    const double u = a.nesterov ? fma((double)a.mu, vn, d) : vn;
    v_new = (float)vn;
    th_new = (float)fma(-(double)a.lr, u, (double)th);
}

// Every thread owns four consecutive elements per iteration: theta and v arrive as
// one 128-bit load each, an instance as 128 bits (fp32) or 64 bits (bf16), so all
// accesses of a warp are contiguous and every fetched sector is used in full.
// four consecutive elements of an instance as they sit in memory (64 bits of bf16 or 128
// bits of fp32): kept packed in registers until used, so that KB loads in flight cost
// 2 KB registers for bf16 instances instead of 4 KB
template <bool BF16>
struct InstRaw {
    typename std::conditional<BF16, uint2, float4>::type w;
};
template <bool BF16>
__device__ __forceinline__ InstRaw<BF16> load_inst4(const void* base, int64_t i) {
    InstRaw<BF16> r;
    if constexpr (BF16) r.w = __ldcs(reinterpret_cast<const uint2*>(base) + i);
    else r.w = __ldcs(reinterpret_cast<const float4*>(base) + i);
    return r;
}
template <bool BF16>
__device__ __forceinline__ void unpack_inst4(const InstRaw<BF16>& r, float (&x)[4]) {
    if constexpr (BF16) {
        x[0] = bf16_lo(r.w.x); x[1] = bf16_hi(r.w.x); x[2] = bf16_lo(r.w.y); x[3] = bf16_hi(r.w.y);
    } else {
        x[0] = r.w.x; x[1] = r.w.y; x[2] = r.w.z; x[3] = r.w.w;
    }
}

// KB = instance loads issued back to back: 8 (with registers for them, 4 blocks per SM)
// when there are at least 8 instances, else 4 (6 blocks per SM) -- measured: K=8 runs 3 %
// faster with the former, K=4 5 % faster with the latter.
template <bool BF16, bool WB, int KB>
__global__ void __launch_bounds__(256, (KB == 8 && !BF16) ? 3 : 4) outer_step_kernel(const __grid_constant__ OuterArgs a) {
    constexpr int VEC = 4;
    const int64_t nvec = a.P / VEC;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step) {
        // all loads of the element group are issued before anything is used: the first KB instances,
        // then theta and v (a use of theta ahead of the instance loads costs a second memory round trip)
        InstRaw<BF16> x[KB];
#pragma unroll
        for (int u = 0; u < KB; ++u)
            if (u < a.K) x[u] = load_inst4<BF16>(a.inst[u], i);
        const float4 t4 = __ldcs(reinterpret_cast<const float4*>(a.th_in) + i);
        const float4 v4 = __ldcs(reinterpret_cast<const float4*>(a.v_in) + i);
        const float th[VEC] = {t4.x, t4.y, t4.z, t4.w};
        const float v[VEC] = {v4.x, v4.y, v4.z, v4.w};
        double acc[VEC], thd[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) { acc[e] = 0.0; thd[e] = (double)th[e]; }
#pragma unroll
        for (int u = 0; u < KB; ++u)
            if (u < a.K) {
                float xe[VEC];
                unpack_inst4<BF16>(x[u], xe);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] += thd[e] - (double)xe[e];
            }
        for (int k = KB; k < a.K; k += KB) {
#pragma unroll
            for (int u = 0; u < KB; ++u)
                if (k + u < a.K) x[u] = load_inst4<BF16>(a.inst[k + u], i);
#pragma unroll
            for (int u = 0; u < KB; ++u)
                if (k + u < a.K) {
                    float xe[VEC];
                    unpack_inst4<BF16>(x[u], xe);
#pragma unroll
                    for (int e = 0; e < VEC; ++e) acc[e] += thd[e] - (double)xe[e];
                }
        }
        float tn[VEC], vn[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) outer_update(th[e], v[e], acc[e], a, tn[e], vn[e]);
        __stcs(reinterpret_cast<float4*>(a.th_out) + i, make_float4(tn[0], tn[1], tn[2], tn[3]));
        __stcs(reinterpret_cast<float4*>(a.v_out) + i, make_float4(vn[0], vn[1], vn[2], vn[3]));
        if (WB) {
            for (int kk = 0; kk < a.K; ++kk) {
                if (a.wb[kk] == nullptr) continue;
                if (BF16) {
                    reinterpret_cast<uint2*>(a.wb[kk])[i] = make_uint2(pack_bf16(tn[0], tn[1]), pack_bf16(tn[2], tn[3]));
                } else {
                    reinterpret_cast<float4*>(a.wb[kk])[i] = make_float4(tn[0], tn[1], tn[2], tn[3]);
                }
            }
        }
    }
    // ragged tail (P not a multiple of the vector width): scalar, first block only
    if (blockIdx.x == 0) {
        for (int64_t j = nvec * VEC + threadIdx.x; j < a.P; j += blockDim.x) {
            const float th = a.th_in[j], v = a.v_in[j];
            double acc = 0.0;
            for (int k = 0; k < a.K; ++k) {
                float x;
                if (BF16) x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.inst[k])[j]);
                else x = reinterpret_cast<const float*>(a.inst[k])[j];
                acc += (double)th - (double)x;
            }
            float tn, vn;
            outer_update(th, v, acc, a, tn, vn);
            a.th_out[j] = tn;
            a.v_out[j] = vn;
            if (WB) {
                for (int k = 0; k < a.K; ++k) {
                    if (a.wb[k] == nullptr) continue;
                    if (BF16) reinterpret_cast<__nv_bfloat16*>(a.wb[k])[j] = __float2bfloat16_rn(tn);
                    else reinterpret_cast<float*>(a.wb[k])[j] = tn;
                }
            }
        }
    }
}

// Persistent grid for the elementwise kernels: as many blocks as are resident at
// once (so no partial last wave), fewer when the problem is smaller than that.
template <typename Kern>
static unsigned elementwise_grid(const adloco_ctx* ctx, Kern kern, int64_t nvec, int threads) {
    // resident blocks per SM, asked once per kernel
    static std::mutex cache_mutex;
    static const void* seen[16];
    static int seen_per_sm[16];
    static int n_seen = 0;
    std::lock_guard<std::mutex> lock(cache_mutex);
    int per_sm = 0;
    for (int k = 0; k < n_seen; ++k)
        if (seen[k] == reinterpret_cast<const void*>(kern)) per_sm = seen_per_sm[k];
    if (per_sm < 1) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
        if (n_seen < 16) { seen[n_seen] = reinterpret_cast<const void*>(kern); seen_per_sm[n_seen] = per_sm; ++n_seen; }
    }
    int64_t want = (nvec + threads - 1) / threads;
    const int64_t cap = (int64_t)ctx->sm_count * per_sm;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    return (unsigned)want;
}

int launch_outer_step(adloco_ctx* ctx, const OuterLaunch& l, cudaStream_t st) {
    OuterArgs a;
    for (int k = 0; k < kMaxInstances; ++k) {
        a.inst[k] = k < l.K ? l.inst[k] : nullptr;
        a.wb[k] = (k < l.K && l.has_wb) ? l.wb[k] : nullptr;
    }
    a.th_in = l.th_in; a.th_out = l.th_out; a.v_in = l.v_in; a.v_out = l.v_out;
    a.P = l.P; a.lr = l.lr; a.mu = l.mu; a.invK = 1.0 / (double)l.K; a.K = l.K; a.nesterov = l.nesterov;
    const int64_t nvec = l.P / 4;
#define ADLOCO_OUTER_LAUNCH(BF, WBK, KBV) \
    outer_step_kernel<BF, WBK, KBV><<<elementwise_grid(ctx, outer_step_kernel<BF, WBK, KBV>, nvec, 256), 256, 0, st>>>(a)
    if (l.K >= 8) {
        if (l.bf16) { if (l.has_wb) ADLOCO_OUTER_LAUNCH(true, true, 8); else ADLOCO_OUTER_LAUNCH(true, false, 8); }
        else { if (l.has_wb) ADLOCO_OUTER_LAUNCH(false, true, 8); else ADLOCO_OUTER_LAUNCH(false, false, 8); }
    } else {
        if (l.bf16) { if (l.has_wb) ADLOCO_OUTER_LAUNCH(true, true, 4); else ADLOCO_OUTER_LAUNCH(true, false, 4); }
        else { if (l.has_wb) ADLOCO_OUTER_LAUNCH(false, true, 4); else ADLOCO_OUTER_LAUNCH(false, false, 4); }
    }
#undef ADLOCO_OUTER_LAUNCH
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// outer step with an exchange: each GPU holds one whole instance and a slice of v
// ---------------------------------------------------------------------------------
// Three elementwise passes around the one exchange of the pseudo-gradients:
//   pseudo_grad_kernel   g = theta - x_k                  (this rank's term of the sum)
//   [the K terms are summed slice-wise across the ranks by a reduce-scatter]
//   outer_apply_kernel   d = g_sum / K, then the same update as outer_step_kernel
//   refresh_kernel       x_k = theta' (cast to the instance type) once theta' is gathered
template <bool BF16>
__global__ void __launch_bounds__(256) pseudo_grad_kernel(const float* __restrict__ theta, const void* __restrict__ inst,
                                                           float* __restrict__ g, int64_t P) {
    const int64_t nvec = P / 4;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step) {
        const InstRaw<BF16> raw = load_inst4<BF16>(inst, i);
        const float4 t = __ldcs(reinterpret_cast<const float4*>(theta) + i);
        float x[4];
        unpack_inst4<BF16>(raw, x);
        __stcs(reinterpret_cast<float4*>(g) + i, make_float4(t.x - x[0], t.y - x[1], t.z - x[2], t.w - x[3]));
    }
    if (blockIdx.x == 0) {
        for (int64_t j = nvec * 4 + threadIdx.x; j < P; j += blockDim.x) {
            float x;
            if (BF16) x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(inst)[j]);
            else x = reinterpret_cast<const float*>(inst)[j];
            g[j] = theta[j] - x;
        }
    }
}

struct ApplyArgs {
    const float* g_sum;
    const float* th_in;
    float* th_out;
    const float* v_in;
    float* v_out;
    int64_t P;
    OuterArgs u;      // invK, lr, mu, nesterov (the instance pointers are unused)
};

__global__ void __launch_bounds__(256) outer_apply_kernel(const __grid_constant__ ApplyArgs a) {
    const int64_t nvec = a.P / 4;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step) {
        const float4 g4 = __ldcs(reinterpret_cast<const float4*>(a.g_sum) + i);
        const float4 t4 = __ldcs(reinterpret_cast<const float4*>(a.th_in) + i);
        const float4 v4 = __ldcs(reinterpret_cast<const float4*>(a.v_in) + i);
        const float g[4] = {g4.x, g4.y, g4.z, g4.w}, th[4] = {t4.x, t4.y, t4.z, t4.w}, v[4] = {v4.x, v4.y, v4.z, v4.w};
        float tn[4], vn[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) outer_update(th[e], v[e], (double)g[e], a.u, tn[e], vn[e]);
        __stcs(reinterpret_cast<float4*>(a.th_out) + i, make_float4(tn[0], tn[1], tn[2], tn[3]));
        __stcs(reinterpret_cast<float4*>(a.v_out) + i, make_float4(vn[0], vn[1], vn[2], vn[3]));
    }
    if (blockIdx.x == 0) {
        for (int64_t j = nvec * 4 + threadIdx.x; j < a.P; j += blockDim.x) {
            float tn, vn;
            outer_update(a.th_in[j], a.v_in[j], (double)a.g_sum[j], a.u, tn, vn);
            a.th_out[j] = tn;
            a.v_out[j] = vn;
        }
    }
}

template <bool BF16>
__global__ void __launch_bounds__(256) refresh_kernel(const float* __restrict__ theta, void* __restrict__ inst, int64_t P) {
    const int64_t nvec = P / 4;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step) {
        const float4 t = __ldcs(reinterpret_cast<const float4*>(theta) + i);
        if (BF16) reinterpret_cast<uint2*>(inst)[i] = make_uint2(pack_bf16(t.x, t.y), pack_bf16(t.z, t.w));
        else reinterpret_cast<float4*>(inst)[i] = t;
    }
    if (blockIdx.x == 0) {
        for (int64_t j = nvec * 4 + threadIdx.x; j < P; j += blockDim.x) {
            if (BF16) reinterpret_cast<__nv_bfloat16*>(inst)[j] = __float2bfloat16_rn(theta[j]);
            else reinterpret_cast<float*>(inst)[j] = theta[j];
        }
    }
}

int launch_pseudo_grad(adloco_ctx* ctx, const float* theta, const void* inst, int bf16, float* g, int64_t P, cudaStream_t st) {
    if (bf16) pseudo_grad_kernel<true><<<elementwise_grid(ctx, pseudo_grad_kernel<true>, P / 4, 256), 256, 0, st>>>(theta, inst, g, P);
    else pseudo_grad_kernel<false><<<elementwise_grid(ctx, pseudo_grad_kernel<false>, P / 4, 256), 256, 0, st>>>(theta, inst, g, P);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_outer_apply(adloco_ctx* ctx, const float* g_sum, int K, int64_t P, const float* th_in, float* th_out,
                       const float* v_in, float* v_out, float lr, float mu, int nesterov, cudaStream_t st) {
    ApplyArgs a;
    memset(&a, 0, sizeof(a));
    a.g_sum = g_sum; a.th_in = th_in; a.th_out = th_out; a.v_in = v_in; a.v_out = v_out; a.P = P;
    a.u.invK = 1.0 / (double)K; a.u.lr = lr; a.u.mu = mu; a.u.K = K; a.u.nesterov = nesterov;
    outer_apply_kernel<<<elementwise_grid(ctx, outer_apply_kernel, P / 4, 256), 256, 0, st>>>(a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_refresh(adloco_ctx* ctx, const float* theta, void* inst, int bf16, int64_t P, cudaStream_t st) {
    if (bf16) refresh_kernel<true><<<elementwise_grid(ctx, refresh_kernel<true>, P / 4, 256), 256, 0, st>>>(theta, inst, P);
    else refresh_kernel<false><<<elementwise_grid(ctx, refresh_kernel<false>, P / 4, 256), 256, 0, st>>>(theta, inst, P);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// weighted merge of trainers (Algorithm 2): out = sum_k coef_k x_k
// ---------------------------------------------------------------------------------
struct MergeArgs {
    const void* x[kMaxInstances];
    float coef[kMaxInstances];
    void* out;
    int64_t P;
    int K;
};

template <bool BF16>
__global__ void __launch_bounds__(256) merge_kernel(const __grid_constant__ MergeArgs a) {
    constexpr int VEC = BF16 ? 8 : 4;
    const int64_t nvec = a.P / VEC;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec; i += step) {
        float acc[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
#pragma unroll 4
        for (int k = 0; k < a.K; ++k) {
            const float w = a.coef[k];
            if (BF16) {
                const uint4 x = __ldcs(reinterpret_cast<const uint4*>(a.x[k]) + i);
                acc[0] = fmaf(w, bf16_lo(x.x), acc[0]); acc[1] = fmaf(w, bf16_hi(x.x), acc[1]);
                acc[2] = fmaf(w, bf16_lo(x.y), acc[2]); acc[3] = fmaf(w, bf16_hi(x.y), acc[3]);
                acc[4 % VEC] = fmaf(w, bf16_lo(x.z), acc[4 % VEC]); acc[5 % VEC] = fmaf(w, bf16_hi(x.z), acc[5 % VEC]);
                acc[6 % VEC] = fmaf(w, bf16_lo(x.w), acc[6 % VEC]); acc[7 % VEC] = fmaf(w, bf16_hi(x.w), acc[7 % VEC]);
            } else {
                const float4 x = __ldcs(reinterpret_cast<const float4*>(a.x[k]) + i);
                acc[0] = fmaf(w, x.x, acc[0]); acc[1] = fmaf(w, x.y, acc[1]);
                acc[2] = fmaf(w, x.z, acc[2]); acc[3] = fmaf(w, x.w, acc[3]);
            }
        }
        if (BF16) {
            uint4 o;
            o.x = pack_bf16(acc[0], acc[1]); o.y = pack_bf16(acc[2], acc[3]);
            o.z = pack_bf16(acc[4 % VEC], acc[5 % VEC]); o.w = pack_bf16(acc[6 % VEC], acc[7 % VEC]);
            reinterpret_cast<uint4*>(a.out)[i] = o;
        } else {
            reinterpret_cast<float4*>(a.out)[i] = make_float4(acc[0], acc[1], acc[2], acc[3]);
        }
    }
    if (blockIdx.x == 0) {
        for (int64_t j = nvec * VEC + threadIdx.x; j < a.P; j += blockDim.x) {
            float acc = 0.f;
            for (int k = 0; k < a.K; ++k) {
                float x;
                if (BF16) x = __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(a.x[k])[j]);
                else x = reinterpret_cast<const float*>(a.x[k])[j];
                acc = fmaf(a.coef[k], x, acc);
            }
            if (BF16) reinterpret_cast<__nv_bfloat16*>(a.out)[j] = __float2bfloat16_rn(acc);
            else reinterpret_cast<float*>(a.out)[j] = acc;
        }
    }
}

int launch_merge(adloco_ctx* ctx, const MergeLaunch& l, cudaStream_t st) {
    MergeArgs a;
    for (int k = 0; k < kMaxInstances; ++k) {
        a.x[k] = k < l.K ? l.x[k] : nullptr;
        a.coef[k] = k < l.K ? l.coef[k] : 0.f;
    }
    a.out = l.out; a.P = l.P; a.K = l.K;
    const int vec = l.bf16 ? 8 : 4;
    if (l.bf16) merge_kernel<true><<<elementwise_grid(ctx, merge_kernel<true>, l.P / vec, 256), 256, 0, st>>>(a);
    else merge_kernel<false><<<elementwise_grid(ctx, merge_kernel<false>, l.P / vec, 256), 256, 0, st>>>(a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// ---------------------------------------------------------------------------------
// accumulator helpers for the tensor-core path
// ---------------------------------------------------------------------------------
// Q += sum(n[0..b)), count += b; the centred sum is no longer available.
__global__ void accum_add_norms_kernel(adloco_test_sums* state, const float* n, int64_t b) {
    __shared__ double red[32];
    double t = 0.0;
    for (int64_t i = threadIdx.x; i < b; i += blockDim.x) t += (double)n[i];
    const double tot = block_sum(t, red);
    if (threadIdx.x == 0) {
        state->sum_sqnorm += tot;
        state->batch_count += b;
        state->has_centred = 0;
    }
}

int launch_accum_add_norms(adloco_ctx* ctx, adloco_accum* acc, const float* n, int64_t b, cudaStream_t st) {
    accum_add_norms_kernel<<<1, 256, 0, st>>>(acc->state, n, b);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

constexpr int SQ_CHUNK = 4096;  // elements per block-iteration: 256 threads x 4 float4

// ||S||^2 summed over all buffers of the accumulator -> state->sum_sq_gsum.
__global__ void __launch_bounds__(256) accum_sqnorm_kernel(float* const* bufs, const int64_t* sizes,
                                                           const int64_t* chunk_prefix, int n_bufs,
                                                           int64_t total_chunks, double* blk_scalars,
                                                           unsigned* ticket, adloco_test_sums* state) {
    __shared__ double red[32];
    __shared__ int is_last;
    float f = 0.f;
    double t = 0.0;
    int since = 0;
    for (int64_t ch = blockIdx.x; ch < total_chunks; ch += gridDim.x) {
        // which buffer holds chunk ch: largest b with chunk_prefix[b] <= ch
        int lo = 0, hi = n_bufs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (chunk_prefix[mid] <= ch) lo = mid; else hi = mid - 1;
        }
        const float* base = bufs[lo];
        const int64_t size = sizes[lo];
        const int64_t off = (ch - chunk_prefix[lo]) * SQ_CHUNK;
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t j = off + ((int64_t)h * 256 + threadIdx.x) * 4;
            if (j < size) {
                const int nv = (size - j) >= 4 ? 4 : (int)(size - j);
                const float4 x = load4(base + j, nv);
                f += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
            }
        }
        if (++since == 16) { t += (double)f; f = 0.f; since = 0; }
    }
    t += (double)f;
    const double b = block_sum(t, red);
    if (threadIdx.x == 0) blk_scalars[(int64_t)blockIdx.x * 4] = b;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double p = 0.0;
    for (unsigned blk = threadIdx.x; blk < gridDim.x; blk += blockDim.x) p += __ldcg(blk_scalars + (int64_t)blk * 4);
    const double tot = block_sum(p, red);
    if (threadIdx.x == 0) {
        state->sum_sq_gsum = tot;
        *ticket = 0u;
    }
}

// All gradient-sum buffers of the accumulator and its state set to zero in one launch (a model's
// accumulator has one buffer per parameter: a memset each would put dozens of tiny operations on the stream).
__global__ void __launch_bounds__(256) accum_zero_kernel(float* const* bufs, const int64_t* sizes, const int64_t* chunk_prefix,
                                                         int n_bufs, int64_t total_chunks, adloco_test_sums* state) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        adloco_test_sums z;
        memset(&z, 0, sizeof(z));
        *state = z;
    }
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t ch = blockIdx.x; ch < total_chunks; ch += gridDim.x) {
        int lo = 0, hi = n_bufs - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (chunk_prefix[mid] <= ch) lo = mid; else hi = mid - 1;
        }
        float* base = bufs[lo];
        const int64_t size = sizes[lo];
        const int64_t off = (ch - chunk_prefix[lo]) * SQ_CHUNK;
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t j = off + ((int64_t)h * 256 + threadIdx.x) * 4;
            if (j < size) store4(base + j, zero, (size - j) >= 4 ? 4 : (int)(size - j));
        }
    }
}

int launch_accum_zero(adloco_ctx* ctx, adloco_accum* acc, cudaStream_t st) {
    int64_t grid = acc->total_chunks;
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    accum_zero_kernel<<<(unsigned)grid, 256, 0, st>>>(acc->bufs_dev, acc->sizes_dev, acc->chunk_prefix_dev, acc->n_bufs,
                                                     acc->total_chunks, acc->state);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_accum_sqnorm(adloco_ctx* ctx, adloco_accum* acc, cudaStream_t st) {
    int64_t grid = acc->total_chunks;
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (grid > cap) grid = cap;
    if (grid > ctx->max_grid) grid = ctx->max_grid;
    if (grid < 1) grid = 1;
    accum_sqnorm_kernel<<<(unsigned)grid, 256, 0, st>>>(acc->bufs_dev, acc->sizes_dev, acc->chunk_prefix_dev,
                                                       acc->n_bufs, acc->total_chunks, ctx->blk_scalars,
                                                       ctx->ticket, acc->state);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

}  // namespace adloco
