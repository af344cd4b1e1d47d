// Tensor-core path (tcgen05 + TMEM + TMA) for linear layers:
//
//   gram_sqnorm_kernel  n_i = <X_i X_i^T, D_i D_i^T>_F, the squared Frobenius norm of
//                       sample i's weight gradient D_i^T X_i, without forming it:
//                       for every tile on or above the diagonal of the token-by-token
//                       Gram matrices both products are accumulated in TMEM and the
//                       epilogue reduces their elementwise product.
//   gram_pair_kernel    the same over pairs of CTAs (cta_group::2, 256-token tiles).
//   mean_grad_kernel    S (+)= sum_i D_i^T X_i, the batch gradient sum, a GEMM whose
//                       contraction runs over all tokens of all samples.
//   direct_group_kernel every sample's weight-gradient tile formed in TMEM (norms and the
//                       gradient sum from one GEMM), over groups of layers, one CTA or a
//                       pair of CTAs per tile.
//   embed_gram_kernel / embed_segment_kernel / embed_scatter_kernel: embedding tables
//                       (the segment and scatter kernels are plain streaming kernels; they
//                       sit here beside the masked Gram form of the same norms).
//
// The tensor-core kernels are persistent and warp-specialised: warp 0 issues TMA tile loads
// into a ring of shared-memory stages, warp 1 issues tcgen05.mma from shared
// memory into TMEM accumulators, the remaining warps drain the accumulators.
// Every wait is bounded; a wait that runs out raises a status word and all
// roles leave through the common teardown.
#include <atomic>
#include <mutex>
#include <new>
#include <unordered_map>

#include "common.cuh"
#include "ptx.cuh"

namespace adloco {

using namespace ptx;

constexpr int kDirectGroupCap = 48;                 // layers per launch of the grouped direct kernel
constexpr uint64_t kDrainLimitNs = 50000000ull;    // 50 ms per barrier while leaving after a time-out
constexpr uint64_t kPairGraceNs = 1000000ull;      // 1 ms: a CTA pair leaving after a time-out; copies in flight land long before

struct PipeState {
    uint32_t stage = 0, phase = 0;
    __device__ __forceinline__ void advance(uint32_t nstages) {
        if (++stage == nstages) { stage = 0; phase ^= 1u; }
    }
};

__device__ __forceinline__ float warp_sum_f(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// =====================================================================================
// Gram kernel
// =====================================================================================
// Work item = (sample i, 128-token row tile ti, one or two adjacent 128-token column
// blocks c0, c0+1) on or above the diagonal of the T x T Gram matrices.  Row ti's
// blocks ti..nt-1 are grouped in pairs from the diagonal outwards, a left-over
// single block last; a pair is one 128x256 MMA tile (each operand byte fetched
// into shared memory then feeds twice the math of a 128x128 tile, which is what
// the L2 -> shared-memory path needs to keep the tensor pipe busy).
constexpr int GR_TILE = 128;                       // tokens per block side
constexpr int GR_BK = 64;                          // features per stage: 64 bf16 = one 128-byte swizzle row
constexpr int GR_STAGES = 4;
constexpr int GR_BLOCK_BYTES = GR_TILE * GR_BK * 2;          // 16 KB: 128 rows of one stage
constexpr int GR_STAGE_BYTES = 3 * GR_BLOCK_BYTES;           // row tile + up to two column blocks
constexpr int GR_SMEM = GR_STAGES * GR_STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
constexpr int GR_EPI_WARPS = 8;                              // epilogue warps: GR_PARTS per TMEM lane quarter
constexpr int GR_PARTS = GR_EPI_WARPS / 4;                   // each takes 1/GR_PARTS of the tile's columns
constexpr int GR_THREADS = 64 + 32 * GR_EPI_WARPS;           // warp 0 TMA, warp 1 MMA, the rest epilogue

struct GramArgs {
    int B, T, d_in, d_out;
    int nt;               // 128-token blocks per sample side
    int full_per_sample;  // items with two column blocks
    int half_per_sample;  // items with one
    int n_full;           // B * full_per_sample; items [0, n_full) are the two-block ones
    int total_items;
    float* n;             // [B], += (zeroed by the launcher unless accumulating)
    int* status;
    uint64_t wait_ns;   // bound of every in-kernel wait
};

__device__ __forceinline__ void gram_decode(int item, const GramArgs& a, int& i, int& ti, int& c0, int& ncb) {
    const bool full = item < a.n_full;
    int local;
    if (full) {
        i = item / a.full_per_sample;
        local = item - i * a.full_per_sample;
    } else {
        const int h = item - a.n_full;
        i = h / a.half_per_sample;
        local = h - i * a.half_per_sample;
    }
    for (ti = 0; ti < a.nt - 1; ++ti) {
        const int blocks = a.nt - ti;
        const int cnt = full ? (blocks >> 1) : (blocks & 1);
        if (local < cnt) break;
        local -= cnt;
    }
    if (full) { c0 = ti + 2 * local; ncb = 2; }
    else { c0 = a.nt - 1; ncb = 1; }
}

// The k-th work item of CTA b out of G, or -1 when it has no more.  Two-block items (indices below
// n_full) are dealt round-robin: CTAs [0, r) get one more of them than the rest.  The one-block items even
// that out first -- two to each of the CTAs that got one two-block item fewer -- and only what is left of
// them goes round all CTAs again.  (One plain round-robin over the whole list gave the CTAs with the extra
// two-block item a one-block item on top: 9 blocks against an average of 7.8 at B = 32, T = 1024 on 148 SMs.)
__device__ __forceinline__ int gram_cta_item(int k, int b, int G, const GramArgs& a) {
    const int n_full = a.n_full, n_half = a.total_items - a.n_full;
    const int q = n_full / G, r = n_full - q * G;
    const int mine_full = q + (b < r ? 1 : 0);
    if (k < mine_full) return b + k * G;
    k -= mine_full;
    const int low = G - r;                                      // CTAs with q two-block items (all of them when r == 0)
    const int first = n_half < 2 * low ? n_half : 2 * low;      // one-block items dealt to those, up to two each
    if (b >= r) {
        const int h0 = b - r;
        const int cnt = h0 < first ? 1 + (h0 + low < first ? 1 : 0) : 0;
        if (k < cnt) return n_full + h0 + k * low;
        k -= cnt;
    }
    const int h = first + b + k * G;
    return h < n_half ? n_full + h : -1;
}

__global__ void __launch_bounds__(GR_THREADS, 1)
gram_sqnorm_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD,
                   const GramArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + GR_STAGES * GR_STAGE_BYTES;
    // barrier slots (8 bytes each): full[S], empty[S], tmem_full, tmem_empty, drain
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (GR_STAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * GR_STAGES);
    const uint32_t tempty_bar = bar_base + 8u * (2 * GR_STAGES + 1);
    const uint32_t drain_bar = bar_base + 8u * (2 * GR_STAGES + 2);
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (uint32_t s = 0; s < GR_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, GR_EPI_WARPS);
        mbar_init(drain_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmD);
    }
    if (warp == 1) {  // TMEM: X X^T accumulator in columns 0-255, D D^T in 256-511
        tmem_alloc(smem_u32(&tmem_base_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;

    const int kx = (a.d_in + GR_BK - 1) / GR_BK, kd = (a.d_out + GR_BK - 1) / GR_BK;
    const int chunks = kx + kd;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            PipeState ps;
            uint32_t issued = 0;
            bool ok = true;
            for (int k_item = 0, item; ok && (item = gram_cta_item(k_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++k_item) {
                int i, ti, c0, ncb;
                gram_decode(item, a, i, ti, c0, ncb);
                // on the diagonal the row tile is the first column block: fetch it once
                const bool diag = (c0 == ti);
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait(empty_bar(ps.stage), ps.phase ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    const bool is_x = c < kx;
                    const CUtensorMap* map = is_x ? &tmX : &tmD;
                    const int k0 = (is_x ? c : c - kx) * GR_BK;
                    const uint32_t sA = smem_base + ps.stage * GR_STAGE_BYTES;
                    mbar_arrive_expect_tx(full_bar(ps.stage), ((diag ? 0 : 1) + ncb) * GR_BLOCK_BYTES);
                    if (!diag) tma_load_3d(sA, map, full_bar(ps.stage), k0, ti * GR_TILE, i);
                    tma_load_3d(sA + GR_BLOCK_BYTES, map, full_bar(ps.stage), k0, c0 * GR_TILE, i);
                    if (ncb == 2)
                        tma_load_3d(sA + 2 * GR_BLOCK_BYTES, map, full_bar(ps.stage), k0, (c0 + 1) * GR_TILE, i);
                    ++issued;
                    ps.advance(GR_STAGES);
                }
            }
            if (!ok) {
                // leaving after a time-out: let the copies still in flight land first
                PipeState q = ps;
                const uint32_t back = issued < GR_STAGES ? issued : GR_STAGES;
                for (uint32_t r = 0; r < back; ++r) {
                    if (q.stage == 0) { q.stage = GR_STAGES - 1; q.phase ^= 1u; } else { --q.stage; }
                    int never = 0;
                    mbar_wait(full_bar(q.stage), q.phase, &never, kDrainLimitNs);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            PipeState ps;
            bool ok = true;
            int n_item = 0;
            for (int item; ok && (item = gram_cta_item(n_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++n_item) {
                int i, ti, c0, ncb;
                gram_decode(item, a, i, ti, c0, ncb);
                const uint32_t idesc = idesc_bf16_f32(GR_TILE, GR_TILE * ncb, 0, 0);
                // the single accumulator pair must have been drained by the epilogue
                if (!mbar_wait(tempty_bar, (n_item & 1u) ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait(full_bar(ps.stage), ps.phase, abortp, a.wait_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (c < kx ? 0u : 256u);
                    const bool first = (c == 0 || c == kx);
                    const uint32_t sB = smem_base + ps.stage * GR_STAGE_BYTES + GR_BLOCK_BYTES;
                    const uint32_t sA = (c0 == ti) ? sB : sB - GR_BLOCK_BYTES;
#pragma unroll
                    for (int kk = 0; kk < GR_BK / 16; ++kk) {
                        // K-major, 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart;
                        // 16 features further along K = 32 bytes further in the row
                        const uint64_t da = smem_desc_sw128(sA + kk * 32, 16, 1024);
                        const uint64_t db = smem_desc_sw128(sB + kk * 32, 16, 1024);
                        mma_bf16(acc, da, db, idesc, (first && kk == 0) ? 0u : 1u);
                    }
                    mma_commit(empty_bar(ps.stage));   // stage reusable once these MMAs have read it
                    ps.advance(GR_STAGES);
                }
                if (ok) mma_commit(tfull_bar);         // both accumulators of this item complete
            }
            if (!ok) {
                mma_commit(drain_bar);
                int never = 0;
                mbar_wait(drain_bar, 0, &never, kDrainLimitNs);
            }
        }
    } else {
        // ---------------- epilogue: sum over the tile of (X X^T) .* (D D^T) ----------------
        const uint32_t q = warp & 3;            // TMEM lanes 32q .. 32q+31 belong to this warp
        const uint32_t half = (warp - 2) >> 2;  // which part of the tile's columns
        int n_item = 0;
        for (int item; (item = gram_cta_item(n_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++n_item) {
            int i, ti, c0, ncb;
            gram_decode(item, a, i, ti, c0, ncb);
            // the whole warp takes the same decision: the TMEM loads below are warp-collective
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar, n_item & 1u, abortp, a.wait_ns))) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16);
            const int cols_per_half = (GR_TILE * ncb) / GR_PARTS;
            const int col_begin = (int)half * cols_per_half;
            float sum = 0.f;
#pragma unroll 1
            for (int col = col_begin; col < col_begin + cols_per_half; col += 32) {
                uint32_t x[32], d[32];
                tmem_ld32(taddr + col, x);
                tmem_ld32(taddr + 256 + col, d);
                tmem_ld_wait();
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < 32; ++e) part = fmaf(__uint_as_float(x[e]), __uint_as_float(d[e]), part);
                // blocks below the diagonal are never computed: an off-diagonal block counts twice
                sum += (c0 + (col >> 7) == ti) ? part : 2.0f * part;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
            const float w = warp_sum_f(sum);
            if (lane == 0) atomicAdd(a.n + i, w);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(a.status, (int)ADLOCO_ERR_TIMEOUT);
}

// =====================================================================================
// Gram kernel over CTA pairs
// =====================================================================================
// The T x T Gram matrices are cut into 256-token blocks; a work item is (sample i, block
// row p, block column q >= p).  The two CTAs of a cluster share one 256 x 256 MMA per K
// step (cta_group::2): CTA r holds token rows 256 p + 128 r .. + 127 in its tensor memory
// and loads those rows (16 KB per stage) plus ONE half of the column operand, tokens
// 256 q + 128 r .. + 127 (16 KB) -- 32 KB per stage per CTA for a 128 x 256 tile of
// output, 131 flops per byte brought into shared memory against 87 for the one-CTA item
// (whose feed of operands, not the tensor pipe, sets its time).  On the diagonal (p == q)
// a CTA's row tile IS its column half and is fetched once.  Of a diagonal item's four
// 128 x 128 sub-blocks the one below the diagonal is computed and not used (weight 0);
// blocks beyond T read as zeros.
//
// The X X^T product (TMEM columns 0-255) is complete before the D D^T product (columns
// 256-511) starts: the 16 epilogue warps copy their 64 columns of X X^T into registers
// while the D D^T MMAs run and hand the columns back, so the next item's X X^T MMAs start
// the moment this item's D D^T MMAs have been issued and the tensor pipe never waits for
// the epilogue; the elementwise product is then formed against D D^T straight from TMEM.
//
// Items are drawn in list order (sample-major) from a global counter, so all workers sit
// on the same few samples at a time and those samples' operands stay in L2.
constexpr int GP_STAGES = 7;                                   // 224 KB of operands in flight: 7 stages measured 5 % faster than 6, 6 % than 4
constexpr int GP_STAGE_BYTES = 2 * GR_BLOCK_BYTES;             // row tile + this CTA's half of the columns: 32 KB
constexpr int GP_EPI_WARPS = 16;                               // four column slices of 64 per TMEM lane quarter
constexpr int GP_THREADS = 64 + 32 * GP_EPI_WARPS;             // warp 0 TMA, warp 1 MMA, the rest epilogue
constexpr int GP_SCHED_Q = 8;
constexpr int GP_SMEM = GP_STAGES * GP_STAGE_BYTES + 1024 /*align*/ + 512 /*barriers*/;

struct GramPairArgs {
    int B, T, d_in, d_out;
    int nt;               // 128-token blocks per side
    int m;                // 256-token blocks per side
    int rects;            // items per sample: m (m + 1) / 2
    int total_items;
    int* counter;         // zero at launch
    float* n;             // [B], +=
    int* status;
    uint64_t wait_ns;
};

__device__ __forceinline__ void gram_pair_decode(int item, const GramPairArgs& a, int& i, int& p, int& q) {
    i = item / a.rects;
    int r = item - i * a.rects;
    for (p = 0; p < a.m - 1; ++p) {         // block row p has the m - p block columns p .. m - 1
        const int cnt = a.m - p;
        if (r < cnt) break;
        r -= cnt;
    }
    q = p + r;
}

__global__ void __launch_bounds__(GP_THREADS, 1)
gram_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD,
                 const GramPairArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + GP_STAGES * GP_STAGE_BYTES;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (GP_STAGES + s); };
    const uint32_t xx_full = bar_base + 8u * (2 * GP_STAGES);
    const uint32_t dd_full = bar_base + 8u * (2 * GP_STAGES + 1);
    const uint32_t xx_empty = bar_base + 8u * (2 * GP_STAGES + 2);
    const uint32_t dd_empty = bar_base + 8u * (2 * GP_STAGES + 3);
    const uint32_t drain_bar = bar_base + 8u * (2 * GP_STAGES + 4);
    auto sched_full = [&](uint32_t s) { return bar_base + 8u * (2 * GP_STAGES + 5 + s); };
    auto sched_empty = [&](uint32_t s) { return bar_base + 8u * (2 * GP_STAGES + 5 + GP_SCHED_Q + s); };
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int sched_item[GP_SCHED_Q];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_cta_rank();          // 0 = the CTA that issues the MMAs and draws the items
    const int worker = (int)(blockIdx.x >> 1);
    const int n_workers = (int)(gridDim.x >> 1);
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (uint32_t s = 0; s < (uint32_t)GP_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(xx_full, 1);
        mbar_init(dd_full, 1);
        mbar_init(xx_empty, 2 * GP_EPI_WARPS);          // the epilogue warps of both CTAs
        mbar_init(dd_empty, 2 * GP_EPI_WARPS);
        mbar_init(drain_bar, 1);
        for (uint32_t s = 0; s < (uint32_t)GP_SCHED_Q; ++s) {
            mbar_init(sched_full(s), 1);
            // readers of a slot: the even CTA's MMA thread, the odd CTA's TMA thread, both CTAs' epilogue warps
            mbar_init(sched_empty(s), 2 * (1 + GP_EPI_WARPS));
        }
        fence_barrier_init();
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmD);
    }
    if (warp == 1) { tmem_alloc_pair(smem_u32(&tmem_base_slot), 512); tmem_relinquish_pair(); }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();        // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int kx = (a.d_in + GR_BK - 1) / GR_BK, kd = (a.d_out + GR_BK - 1) / GR_BK;
    const int chunks = kx + kd;
    const uint32_t sched_empty_remote0 = map_to_cta(sched_empty(0), 0);

    // item number k of this worker, as published by the drawing thread; -1 when the wait ran out
    auto take_item = [&](int k, bool whole_warp) -> int {
        const uint32_t slot = (uint32_t)k % GP_SCHED_Q, ph = ((uint32_t)k / GP_SCHED_Q) & 1u;
        bool got = mbar_wait<true>(sched_full(slot), ph, abortp, a.wait_ns);
        if (whole_warp) got = __all_sync(0xffffffffu, got);
        if (!got) return -1;
        const int item = *reinterpret_cast<volatile int*>(&sched_item[slot]);
        if (whole_warp) __syncwarp();
        if (!whole_warp || lane == 0) {
            if (rank != 0) mbar_arrive_cluster(sched_empty_remote0 + 8u * slot);
            else mbar_arrive(sched_empty(slot));
        }
        return item;
    };

    if (warp == 0) {
        // ---------------- TMA producer (one per CTA; the even CTA's also draws the items) ----------------
        if (lane == 0) {
            PipeState ps;
            bool ok = true;
            int item = worker;                      // the first item needs no draw
            for (int k = 0; ok; ++k) {
                if (rank == 0) {
                    const uint32_t slot = (uint32_t)k % GP_SCHED_Q, ph = ((uint32_t)k / GP_SCHED_Q) & 1u;
                    if (!mbar_wait<true>(sched_empty(slot), ph ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    *reinterpret_cast<volatile int*>(&sched_item[slot]) = item;
                    st_cluster_u32(map_to_cta(smem_u32(&sched_item[slot]), 1u), (uint32_t)item);
                    mbar_arrive(sched_full(slot));
                    mbar_arrive_cluster(map_to_cta(sched_full(slot), 1u));
                } else {
                    item = take_item(k, false);
                    if (item < 0) { ok = false; break; }
                }
                if (item >= a.total_items) break;   // the list is exhausted: every role has been told
                int next_item = 0;
                if (rank == 0) next_item = n_workers + atomicAdd(a.counter, 1);
                int i, p, q;
                gram_pair_decode(item, a, i, p, q);
                const int row0 = (2 * p + (int)rank) * GR_TILE;      // this CTA's token rows
                const int col0 = (2 * q + (int)rank) * GR_TILE;      // this CTA's half of the token columns
                const bool diag = (p == q);
                const uint32_t bytes = diag ? GR_BLOCK_BYTES : GP_STAGE_BYTES;
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait(empty_bar(ps.stage), ps.phase ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    const bool is_x = c < kx;
                    const CUtensorMap* map = is_x ? &tmX : &tmD;
                    const int k0 = (is_x ? c : c - kx) * GR_BK;
                    const uint32_t sA = smem_base + ps.stage * GP_STAGE_BYTES;
                    const uint32_t bar = map_to_cta(full_bar(ps.stage), 0);
                    if (rank == 0) mbar_arrive_expect_tx(full_bar(ps.stage), 2 * bytes);
                    tma_load_3d_pair(sA, map, bar, k0, row0, i);
                    if (!diag) tma_load_3d_pair(sA + GR_BLOCK_BYTES, map, bar, k0, col0, i);
                    ps.advance(GP_STAGES);
                }
                item = next_item;
            }
            if (!ok) {
                // leaving after a time-out: the byte counts of copies in flight complete on the even CTA's
                // barriers, which the odd CTA cannot wait on: both sit out a grace period far beyond the
                // flight time of a copy
                st_cluster_u32(map_to_cta(smem_u32(&abort_flag), rank ^ 1u), 1u);
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < kPairGraceNs) { }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (even CTA only) ----------------
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(256, 256, 0, 0);     // both operands K-major
            PipeState ps;
            bool ok = true;
            for (int k = 0; ok; ++k) {
                const int item = take_item(k, false);
                if (item < 0) { ok = false; break; }
                if (item >= a.total_items) break;
                int i, p, q;
                gram_pair_decode(item, a, i, p, q);
                const uint32_t b_off = (p == q) ? 0u : (uint32_t)GR_BLOCK_BYTES;   // on the diagonal the row tile is the column half
                for (int c = 0; c < chunks; ++c) {
                    if (c == 0 || c == kx) {
                        // the accumulator about to be overwritten has been read by every epilogue warp
                        if (!mbar_wait<true>(c == 0 ? xx_empty : dd_empty, ((uint32_t)k & 1u) ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                        tc_fence_after();
                    }
                    if (!mbar_wait(full_bar(ps.stage), ps.phase, abortp, a.wait_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + (c < kx ? 0u : 256u);
                    const bool first = (c == 0 || c == kx);
                    const uint32_t sA = smem_base + ps.stage * GP_STAGE_BYTES;
                    const uint32_t sB = sA + b_off;
#pragma unroll
                    for (int kk = 0; kk < GR_BK / 16; ++kk) {
                        // K-major, 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart; 16 features
                        // further along K = 32 bytes further in the row
                        const uint64_t da = smem_desc_sw128(sA + kk * 32, 16, 1024);
                        const uint64_t db = smem_desc_sw128(sB + kk * 32, 16, 1024);
                        mma_bf16_pair(acc, da, db, idesc, (first && kk == 0) ? 0u : 1u);
                    }
                    mma_commit_pair(empty_bar(ps.stage), 3);       // the stage is free in both CTAs
                    ps.advance(GP_STAGES);
                    if (c == kx - 1) mma_commit_pair(xx_full, 3);  // X X^T of this item complete in both CTAs
                }
                if (ok) mma_commit_pair(dd_full, 3);
            }
            if (!ok) {
                st_cluster_u32(map_to_cta(smem_u32(&abort_flag), 1u), 1u);
                mma_commit_pair(drain_bar, 1);
                int never = 0;
                mbar_wait(drain_bar, 0, &never, kDrainLimitNs);
            }
        }
    } else {
        // ---------------- epilogue: sum over the tile of (X X^T) .* (D D^T) ----------------
        const uint32_t lq = warp & 3;                    // TMEM lane quarter: rows 32 lq .. 32 lq + 31 of this CTA's row tile
        const uint32_t slice = (uint32_t)(warp - 2) >> 2;   // columns 64 slice .. 64 slice + 63 of the 256
        const uint32_t xx_empty_remote = map_to_cta(xx_empty, 0), dd_empty_remote = map_to_cta(dd_empty, 0);
        const uint32_t taddr = tmem_base + ((lq * 32u) << 16) + slice * 64u;
        for (int k = 0;; ++k) {
            const int item = take_item(k, true);
            if (item < 0 || item >= a.total_items) break;
            int i, p, q;
            gram_pair_decode(item, a, i, p, q);
            // weight of this warp's 128 x 128 sub-block: 0 below the diagonal or beyond T (never read),
            // 1 on the diagonal, 2 above it (its mirror image is never computed)
            const int rb = 2 * p + (int)rank, cb = 2 * q + (int)(slice >> 1);
            const float w = (rb >= a.nt || cb >= a.nt || rb > cb) ? 0.f : (rb == cb ? 1.f : 2.f);
            const uint32_t par = (uint32_t)k & 1u;
            if (!__all_sync(0xffffffffu, mbar_wait(xx_full, par, abortp, a.wait_ns))) break;
            tc_fence_after();
            uint32_t xx[4][16];
            if (w != 0.f) {                              // uniform across the warp
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) tmem_ld16(taddr + cc * 16, xx[cc]);
                tmem_ld_wait();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(xx_empty_remote);
            if (!__all_sync(0xffffffffu, mbar_wait(dd_full, par, abortp, a.wait_ns))) break;
            tc_fence_after();
            float sum = 0.f;
            if (w != 0.f) {
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    uint32_t r[16];
                    tmem_ld16(taddr + 256u + cc * 16, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 16; ++e) sum = fmaf(__uint_as_float(xx[cc][e]), __uint_as_float(r[e]), sum);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(dd_empty_remote);
            if (w != 0.f) {
                const float tot = warp_sum_f(sum) * w;
                if (lane == 0) atomicAdd(a.n + i, tot);
            }
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();   // neither CTA frees tensor memory or leaves while its peer still works
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(a.status, (int)ADLOCO_ERR_TIMEOUT);
}

// =====================================================================================
// embedding kernel: Gram identity with the activations' Gram matrix replaced by a mask
// =====================================================================================
// Sample i's gradient of an embedding table has row v = sum of delta_t over the tokens
// with id_t = v, so ||G_i||^2 = sum_{t,s} [id_t == id_s] (delta_t . delta_s): the Gram
// kernel without the X X^T product -- the epilogue keeps the entries of D D^T whose two
// tokens carry the same id.  Same work items (sample, row tile, one or two column
// blocks on or above the diagonal); the accumulator is double-buffered.
struct EmbedArgs {
    GramArgs g;          // B, T, d_out = embedding width, item bookkeeping, n, status, wait bound
    const int* ids;      // [B, T]
    int V;               // rows of the table: ids outside [0, V) belong to no row and match nothing
};

__global__ void __launch_bounds__(GR_THREADS, 1)
embed_gram_kernel(const __grid_constant__ CUtensorMap tmD, const EmbedArgs ea) {
    const GramArgs& a = ea.g;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bar_base = smem_base + GR_STAGES * GR_STAGE_BYTES;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (GR_STAGES + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * GR_STAGES + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * GR_STAGES + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * GR_STAGES + 4);
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (uint32_t s = 0; s < GR_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (uint32_t b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), GR_EPI_WARPS); }
        mbar_init(drain_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&tmD);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);   // two 128x256 accumulators of D D^T
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int chunks = (a.d_out + GR_BK - 1) / GR_BK;

    if (warp == 0) {
        if (lane == 0) {
            PipeState ps;
            uint32_t issued = 0;
            bool ok = true;
            for (int k_item = 0, item; ok && (item = gram_cta_item(k_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++k_item) {
                int i, ti, c0, ncb;
                gram_decode(item, a, i, ti, c0, ncb);
                const bool diag = (c0 == ti);
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait(empty_bar(ps.stage), ps.phase ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    const uint32_t sA = smem_base + ps.stage * GR_STAGE_BYTES;
                    mbar_arrive_expect_tx(full_bar(ps.stage), ((diag ? 0 : 1) + ncb) * GR_BLOCK_BYTES);
                    if (!diag) tma_load_3d(sA, &tmD, full_bar(ps.stage), c * GR_BK, ti * GR_TILE, i);
                    tma_load_3d(sA + GR_BLOCK_BYTES, &tmD, full_bar(ps.stage), c * GR_BK, c0 * GR_TILE, i);
                    if (ncb == 2)
                        tma_load_3d(sA + 2 * GR_BLOCK_BYTES, &tmD, full_bar(ps.stage), c * GR_BK, (c0 + 1) * GR_TILE, i);
                    ++issued;
                    ps.advance(GR_STAGES);
                }
            }
            if (!ok) {
                PipeState q = ps;
                const uint32_t back = issued < GR_STAGES ? issued : GR_STAGES;
                for (uint32_t r = 0; r < back; ++r) {
                    if (q.stage == 0) { q.stage = GR_STAGES - 1; q.phase ^= 1u; } else { --q.stage; }
                    int never = 0;
                    mbar_wait(full_bar(q.stage), q.phase, &never, kDrainLimitNs);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            PipeState ps;
            bool ok = true;
            int n_item = 0;
            for (int item; ok && (item = gram_cta_item(n_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++n_item) {
                int i, ti, c0, ncb;
                gram_decode(item, a, i, ti, c0, ncb);
                const uint32_t idesc = idesc_bf16_f32(GR_TILE, GR_TILE * ncb, 0, 0);
                const uint32_t buf = n_item & 1, use = n_item >> 1;
                if (!mbar_wait(tempty_bar(buf), (use & 1u) ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t acc = tmem_base + buf * 256u;
                for (int c = 0; c < chunks; ++c) {
                    if (!mbar_wait(full_bar(ps.stage), ps.phase, abortp, a.wait_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sB = smem_base + ps.stage * GR_STAGE_BYTES + GR_BLOCK_BYTES;
                    const uint32_t sA = (c0 == ti) ? sB : sB - GR_BLOCK_BYTES;
#pragma unroll
                    for (int kk = 0; kk < GR_BK / 16; ++kk) {
                        const uint64_t da = smem_desc_sw128(sA + kk * 32, 16, 1024);
                        const uint64_t db = smem_desc_sw128(sB + kk * 32, 16, 1024);
                        mma_bf16(acc, da, db, idesc, (c == 0 && kk == 0) ? 0u : 1u);
                    }
                    mma_commit(empty_bar(ps.stage));
                    ps.advance(GR_STAGES);
                }
                if (ok) mma_commit(tfull_bar(buf));
            }
            if (!ok) {
                mma_commit(drain_bar);
                int never = 0;
                mbar_wait(drain_bar, 0, &never, kDrainLimitNs);
            }
        }
    } else {
        const uint32_t q = warp & 3;
        const uint32_t half = (warp - 2) >> 2;
        int n_item = 0;
        for (int item; (item = gram_cta_item(n_item, (int)blockIdx.x, (int)gridDim.x, a)) >= 0; ++n_item) {
            int i, ti, c0, ncb;
            gram_decode(item, a, i, ti, c0, ncb);
            // ids of this thread's row and of the columns it will visit; tokens beyond T and ids
            // outside the table (padding, ignore markers) get two different sentinels: they match nothing
            const int* ids_i = ea.ids + (int64_t)i * a.T;
            const int t_row = ti * GR_TILE + (int)q * 32 + lane;
            int id_row = t_row < a.T ? __ldg(ids_i + t_row) : -1;
            if (id_row < 0 || id_row >= ea.V) id_row = -1;
            const uint32_t buf = n_item & 1, use = n_item >> 1;
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abortp, a.wait_ns))) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + buf * 256u;
            const int cols_per_half = (GR_TILE * ncb) / GR_PARTS;
            const int col_begin = (int)half * cols_per_half;
            float sum = 0.f;
#pragma unroll 1
            for (int col = col_begin; col < col_begin + cols_per_half; col += 32) {
                uint32_t d[32];
                tmem_ld32(taddr + col, d);
                const int t_col = c0 * GR_TILE + col + lane;                 // lane l holds the id of column col + l
                int id_col = t_col < a.T ? __ldg(ids_i + t_col) : -2;
                if (id_col < 0 || id_col >= ea.V) id_col = -2;
                tmem_ld_wait();
                float part = 0.f;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    part += (__shfl_sync(0xffffffffu, id_col, e) == id_row) ? __uint_as_float(d[e]) : 0.f;
                sum += (c0 + (col >> 7) == ti) ? part : 2.0f * part;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(buf));
            const float w = warp_sum_f(sum);
            if (lane == 0) atomicAdd(a.n + i, w);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(a.status, (int)ADLOCO_ERR_TIMEOUT);
}

// =====================================================================================
// embedding norms by grouping: the streaming form
// =====================================================================================
// ||G_i||^2 = sum over the table rows v of || sum_{t: id_t = v} delta_t ||^2 needs every delta row once:
// B T d reads against the B T^2 d flops of the masked Gram sum above, which stays as the route for
// sequences longer than ES_MAX_T.  Written as  sum_t ||delta_t||^2  +  sum over the ids that occur more
// than once of ( ||sum of their rows||^2 - sum of their ||.||^2 ):  the first term is a plain stream over
// all rows, the second touches only the rows of repeated ids (again; they are in L2).  Each block of
// sample i groups the sample's T tokens by id in shared memory -- an open-addressing table of H >= 2T
// slots, a count per slot, a prefix sum, a scatter: the tokens of one id end up next to each other in
// `order` -- streams its share of the rows, and sums the groups that start at its share of the
// positions: a warp per group, lane = 8 features per 256; groups of more than ES_BIG rows are summed by
// all warps of the block together.  All blocks of a sample build the same table (T atomics in shared
// memory: cheap next to the rows), so nothing passes through global memory between them.
constexpr int ES_WARPS = 16;
constexpr int ES_THREADS = 32 * ES_WARPS;
constexpr int ES_MAX_T = 4096;          // (3 H + 4 T) ints of shared memory: 160 KB at T = 4096
constexpr int ES_BIG = 64;              // rows from which a group is summed by the whole block
constexpr int ES_NF = 2;                // feature chunks of 256 a warp carries per pass over a small group
constexpr int ES_MAX_BIG = ES_MAX_T / ES_BIG;

struct EmbedSegArgs {
    const int* ids;                 // [B, T]
    const __nv_bfloat16* D;         // [B, T, d]
    int T, d, V, H, chunks;         // H: power of two >= 2 T; chunks: blocks per sample
    float* n;                       // [B], +=
};

__device__ __forceinline__ void es_add_row(float (&acc)[8], const uint4& w) {
    acc[0] += __uint_as_float(w.x << 16); acc[1] += __uint_as_float(w.x & 0xffff0000u);
    acc[2] += __uint_as_float(w.y << 16); acc[3] += __uint_as_float(w.y & 0xffff0000u);
    acc[4] += __uint_as_float(w.z << 16); acc[5] += __uint_as_float(w.z & 0xffff0000u);
    acc[6] += __uint_as_float(w.w << 16); acc[7] += __uint_as_float(w.w & 0xffff0000u);
}

__global__ void __launch_bounds__(ES_THREADS, 2) embed_segment_kernel(const EmbedSegArgs a) {
    extern __shared__ int es_smem[];
    int* keys = es_smem;             // [H] id held by the slot, -1 = free
    int* cnt = keys + a.H;           // [H] tokens of that id
    int* start = cnt + a.H;          // [H] first position of the id's group in `order`
    int* slot_of = start + a.H;      // [T] slot of token t, -1 = id outside the table
    int* rank = slot_of + a.T;       // [T] arrival number of token t within its group
    int* order = rank + a.T;         // [T] token indices, grouped by id
    int* glen = order + a.T;         // [T] length of the group that starts at this position, else 0
    __shared__ float part[ES_WARPS][256];
    __shared__ int big_list[ES_MAX_BIG];
    __shared__ int n_big;
    __shared__ int scan_warp[ES_WARPS];
    __shared__ double red[ES_WARPS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int i = blockIdx.y, c = blockIdx.x;
    const int T = a.T, H = a.H, d = a.d;
    const int* ids_i = a.ids + (int64_t)i * T;
    const __nv_bfloat16* D_i = a.D + (int64_t)i * T * d;

    for (int s = tid; s < H; s += ES_THREADS) { keys[s] = -1; cnt[s] = 0; }
    for (int t = tid; t < T; t += ES_THREADS) glen[t] = 0;
    if (tid == 0) n_big = 0;
    __syncthreads();
    // every token finds the slot of its id (the first to arrive claims it) and takes a number
    for (int t = tid; t < T; t += ES_THREADS) {
        const int id = __ldg(ids_i + t);
        int slot = -1;
        if (id >= 0 && id < a.V) {
            slot = (int)(((uint32_t)id * 2654435761u) & (uint32_t)(H - 1));
            for (;;) {
                const int prev = atomicCAS(&keys[slot], -1, id);
                if (prev == -1 || prev == id) break;
                slot = (slot + 1) & (H - 1);       // H >= 2 T slots: a free one always turns up
            }
            rank[t] = atomicAdd(&cnt[slot], 1);
        }
        slot_of[t] = slot;
    }
    __syncthreads();
    // exclusive prefix sum of the counts: each thread owns H / ES_THREADS consecutive slots (H is a power of two)
    {
        const int per = H >= ES_THREADS ? H / ES_THREADS : 1;
        const int s0 = tid * per;
        int local = 0;
        if (s0 < H)
            for (int k = 0; k < per; ++k) local += cnt[s0 + k];
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) scan_warp[warp] = incl;
        __syncthreads();
        int base = 0;
        for (int w = 0; w < warp; ++w) base += scan_warp[w];
        int run = base + incl - local;
        if (s0 < H)
            for (int k = 0; k < per; ++k) { start[s0 + k] = run; run += cnt[s0 + k]; }
    }
    __syncthreads();
    for (int t = tid; t < T; t += ES_THREADS) {
        const int slot = slot_of[t];
        if (slot >= 0) {
            const int p0 = start[slot];
            order[p0 + rank[t]] = t;
            if (rank[t] == 0) glen[p0] = cnt[slot];
        }
    }
    __syncthreads();

    // (A) every token inside the table adds ||delta_t||^2: the block streams its share of the rows, eight
    // rows in flight per warp.  For an id that occurs once this is the whole contribution.
    float sa = 0.f;
    {
        const int rows_per = (T + a.chunks - 1) / a.chunks;
        const int t_lo = c * rows_per;
        const int t_hi = t_lo + rows_per < T ? t_lo + rows_per : T;
        for (int fc = 0; fc < d; fc += 256) {
            const int f = fc + lane * 8;
            if (f >= d) break;                                   // the same for every later fc too
            for (int t = t_lo + warp; t < t_hi; t += 8 * ES_WARPS) {
                uint4 w[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int tt = t + u * ES_WARPS;
                    w[u] = make_uint4(0, 0, 0, 0);
                    if (tt < t_hi && slot_of[tt] >= 0) w[u] = __ldcs(reinterpret_cast<const uint4*>(D_i + (int64_t)tt * d + f));
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    float r[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    es_add_row(r, w[u]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) sa = fmaf(r[e], r[e], sa);
                }
            }
        }
    }
    // (B) an id that occurs L >= 2 times adds ||sum of its rows||^2 - sum of their ||.||^2 on top (twice the
    // inner products between its rows).  Groups of up to ES_BIG rows: one warp each; the group that starts
    // at position p belongs to warp p % ES_WARPS of block (p / ES_WARPS) % chunks.
    double sq = 0.0;
    for (int p = c * ES_WARPS + warp; p < T; p += a.chunks * ES_WARPS) {
        const int L = glen[p];
        if (L < 2) continue;
        if (L > ES_BIG) {
            if (lane == 0) big_list[atomicAdd(&n_big, 1)] = p;     // at most T / ES_BIG of them
            continue;
        }
        for (int fc = 0; fc < d; fc += 256 * ES_NF) {
            float acc[ES_NF][8];
#pragma unroll
            for (int j = 0; j < ES_NF; ++j)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[j][e] = 0.f;
            float own = 0.f;                                     // sum of the rows' own squared norms
            for (int r = 0; r < L; r += 2) {
                const int t0 = order[p + r];
                const int t1 = (r + 1 < L) ? order[p + r + 1] : -1;
                uint4 w0[ES_NF], w1[ES_NF];
#pragma unroll
                for (int j = 0; j < ES_NF; ++j) {
                    const int f = fc + j * 256 + lane * 8;
                    w0[j] = make_uint4(0, 0, 0, 0);
                    w1[j] = make_uint4(0, 0, 0, 0);
                    if (f < d) {
                        w0[j] = __ldg(reinterpret_cast<const uint4*>(D_i + (int64_t)t0 * d + f));
                        if (t1 >= 0) w1[j] = __ldg(reinterpret_cast<const uint4*>(D_i + (int64_t)t1 * d + f));
                    }
                }
#pragma unroll
                for (int j = 0; j < ES_NF; ++j) {
                    float r0[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, r1[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                    es_add_row(r0, w0[j]);
                    es_add_row(r1, w1[j]);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        own = fmaf(r0[e], r0[e], own);
                        own = fmaf(r1[e], r1[e], own);
                        acc[j][e] += r0[e] + r1[e];
                    }
                }
            }
            float s2 = 0.f;
#pragma unroll
            for (int j = 0; j < ES_NF; ++j)
#pragma unroll
                for (int e = 0; e < 8; ++e) s2 = fmaf(acc[j][e], acc[j][e], s2);
            sq += (double)s2 - (double)own;
        }
    }
    __syncthreads();
    // long groups (a frequent token, padding that maps inside the table): all warps of the block share
    // the rows of one group; their partial sums meet in shared memory before they are squared
    const int nb = n_big;
    for (int k = 0; k < nb; ++k) {
        const int p = big_list[k];
        const int L = glen[p];
        for (int fc = 0; fc < d; fc += 256) {
            const int f = fc + lane * 8;
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            float own = 0.f;
            if (f < d) {
                for (int r = warp; r < L; r += 4 * ES_WARPS) {
                    uint4 w[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int rr = r + u * ES_WARPS;
                        w[u] = make_uint4(0, 0, 0, 0);
                        if (rr < L) w[u] = __ldg(reinterpret_cast<const uint4*>(D_i + (int64_t)order[p + rr] * d + f));
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float r8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                        es_add_row(r8, w[u]);
#pragma unroll
                        for (int e = 0; e < 8; ++e) { own = fmaf(r8[e], r8[e], own); acc[e] += r8[e]; }
                    }
                }
            }
            sq -= (double)own;
#pragma unroll
            for (int e = 0; e < 8; ++e) part[warp][lane * 8 + e] = acc[e];
            __syncthreads();
            if (tid < 256) {
                float g = 0.f;
#pragma unroll
                for (int w = 0; w < ES_WARPS; ++w) g += part[w][tid];
                sq += (double)g * (double)g;
            }
            __syncthreads();
        }
    }
    sq += (double)sa;
    // block total -> n_i
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
    if (lane == 0) red[warp] = sq;
    __syncthreads();
    if (tid == 0) {
        double tot = 0.0;
        for (int w = 0; w < ES_WARPS; ++w) tot += red[w];
        if (tot != 0.0) atomicAdd(a.n + i, (float)tot);
    }
}

// S[id_t, :] += delta_t for every token: one warp per token row, 128-bit loads, vector reductions
__global__ void __launch_bounds__(256) embed_scatter_kernel(const int* ids, const __nv_bfloat16* D, int64_t tokens,
                                                            int d, int V, float* S) {
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = warp_global; t < tokens; t += n_warps) {
        const int id = __ldg(ids + t);
        if (id < 0 || id >= V) continue;             // ids outside the table are ignored
        const __nv_bfloat16* row = D + t * d;
        float* dst = S + (int64_t)id * d;
        for (int f = lane * 8; f < d; f += 256) {    // d is a multiple of 8
            const uint4 w = __ldcs(reinterpret_cast<const uint4*>(row + f));
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + f),
                         "f"(__uint_as_float(w.x << 16)), "f"(__uint_as_float(w.x & 0xffff0000u)),
                         "f"(__uint_as_float(w.y << 16)), "f"(__uint_as_float(w.y & 0xffff0000u)) : "memory");
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + f + 4),
                         "f"(__uint_as_float(w.z << 16)), "f"(__uint_as_float(w.z & 0xffff0000u)),
                         "f"(__uint_as_float(w.w << 16)), "f"(__uint_as_float(w.w & 0xffff0000u)) : "memory");
        }
    }
}

// Work split shared by the two token-contraction kernels.  The (tile, sample) units of
// one output tile are cut into `splits` chunks of `chunk` consecutive samples, every
// chunk starting at a multiple of `chunk`; work item j = (tile j / splits, chunk
// j % splits).  CTAs that start together therefore walk through the same few samples
// at the same time, which keeps the operands of those samples resident in L2 (a plain
// even split lets the CTAs drift over all samples and doubles the DRAM reads).
struct SplitPlan {
    int splits, chunk, items;
};
static SplitPlan make_split(int64_t tiles, int64_t B, int sm_count) {
    SplitPlan p;
    int64_t s = tiles >= sm_count ? 1 : sm_count / tiles;
    if (s > B) s = B;
    p.chunk = (int)((B + s - 1) / s);
    p.splits = (int)((B + p.chunk - 1) / p.chunk);
    p.items = (int)(tiles * p.splits);
    return p;
}
__device__ __forceinline__ void item_range(int item, int splits, int chunk, int B, int64_t& u0, int64_t& u1) {
    const int tile = item / splits, k = item - tile * splits;
    const int b0 = k * chunk;
    const int b1 = b0 + chunk < B ? b0 + chunk : B;
    u0 = (int64_t)tile * B + b0;
    u1 = (int64_t)tile * B + b1;
}

// =====================================================================================
// mean-gradient kernel: S[d_out, d_in] += sum over samples and tokens of delta x^T
// =====================================================================================
// Output tile 256 (d_out) x 256 (d_in): two M=128 MMAs per K step share the X
// operand, their accumulators fill all 512 TMEM columns.  Per byte fetched into
// shared memory this does 128 flops, which is what lets the tensor pipe run
// ahead of the L2 -> shared-memory path (a 128x256 tile does 85).
constexpr int MG_BM = 256;                          // d_out rows per tile (two MMA halves of 128)
constexpr int MG_BN = 256;                          // d_in columns per tile
constexpr int MG_BK = 64;                           // tokens per stage
constexpr int MG_STAGES = 3;
constexpr int MG_BOX_BYTES = 64 * MG_BK * 2;        // one TMA box: 64 features x 64 tokens = 8 KB
constexpr int MG_A_BYTES = (MG_BM / 64) * MG_BOX_BYTES;
constexpr int MG_B_BYTES = (MG_BN / 64) * MG_BOX_BYTES;
constexpr int MG_STAGE_BYTES = MG_A_BYTES + MG_B_BYTES;   // 64 KB
constexpr int MG_BOX_OUT = 32 * 32 * 4;             // per-epilogue-warp staging box: 32 rows x 32 fp32 columns
constexpr int MG_STAGING = 8 * MG_BOX_OUT;
constexpr int MG_SMEM = MG_STAGES * MG_STAGE_BYTES + MG_STAGING + 1024 + 256;
constexpr int MG_THREADS = 320;                     // warp 0 TMA, warp 1 MMA, warps 2-9 epilogue

struct MeanGradArgs {
    int B, T, d_in, d_out;
    int ntm, ntn;       // tiles along d_out, d_in
    int splits, chunk, items;   // see SplitPlan
    float* S;           // [d_out, d_in], += (zeroed by the launcher unless accumulating)
    int* status;
    uint64_t wait_ns;   // bound of every in-kernel wait
};

__global__ void __launch_bounds__(MG_THREADS, 1)
mean_grad_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmD,
                 const __grid_constant__ CUtensorMap tmS, const MeanGradArgs a) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base + MG_STAGES * MG_STAGE_BYTES;   // 1024-aligned
    const uint32_t bar_base = staging_base + MG_STAGING;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (MG_STAGES + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * MG_STAGES);
    const uint32_t tempty_bar = bar_base + 8u * (2 * MG_STAGES + 1);
    const uint32_t drain_bar = bar_base + 8u * (2 * MG_STAGES + 2);
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (uint32_t s = 0; s < MG_STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tfull_bar, 1);
        mbar_init(tempty_bar, 8);
        mbar_init(drain_bar, 1);
        fence_barrier_init();
        prefetch_tmap(&tmX);
        prefetch_tmap(&tmD);
        prefetch_tmap(&tmS);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_slot), 512);   // rows 0-127 in columns 0-255, rows 128-255 in 256-511
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;

    const int kt = (a.T + MG_BK - 1) / MG_BK;

    if (warp == 0) {
        if (lane == 0) {
            PipeState ps;
            uint32_t issued = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < a.items; item += gridDim.x) {
            int64_t u0, u1;
            item_range(item, a.splits, a.chunk, a.B, u0, u1);
            for (int64_t u = u0; ok && u < u1; ++u) {
                const int tile = (int)(u / a.B), i = (int)(u % a.B);
                const int tm = tile / a.ntn, tn = tile % a.ntn;
                for (int c = 0; c < kt; ++c) {
                    if (!mbar_wait(empty_bar(ps.stage), ps.phase ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    const uint32_t sA = smem_base + ps.stage * MG_STAGE_BYTES;
                    const uint32_t sB = sA + MG_A_BYTES;
                    mbar_arrive_expect_tx(full_bar(ps.stage), MG_STAGE_BYTES);
#pragma unroll
                    for (int mb = 0; mb < MG_BM / 64; ++mb)
                        tma_load_3d(sA + mb * MG_BOX_BYTES, &tmD, full_bar(ps.stage), tm * MG_BM + mb * 64, c * MG_BK, i);
#pragma unroll
                    for (int nb = 0; nb < MG_BN / 64; ++nb)
                        tma_load_3d(sB + nb * MG_BOX_BYTES, &tmX, full_bar(ps.stage), tn * MG_BN + nb * 64, c * MG_BK, i);
                    ++issued;
                    ps.advance(MG_STAGES);
                }
            }
            }
            if (!ok) {
                PipeState q = ps;
                const uint32_t back = issued < MG_STAGES ? issued : MG_STAGES;
                for (uint32_t r = 0; r < back; ++r) {
                    if (q.stage == 0) { q.stage = MG_STAGES - 1; q.phase ^= 1u; } else { --q.stage; }
                    int never = 0;
                    mbar_wait(full_bar(q.stage), q.phase, &never, kDrainLimitNs);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // both operands are stored with the contraction index (tokens) strided: MN-major
            constexpr uint32_t idesc = idesc_bf16_f32(128, MG_BN, 1, 1);
            PipeState ps;
            bool ok = true;
            int seg = 0;
            for (int item = blockIdx.x; ok && item < a.items; item += gridDim.x) {
            int64_t u0, u1;
            item_range(item, a.splits, a.chunk, a.B, u0, u1);
            int64_t u = u0;
            while (ok && u < u1) {
                const int64_t u_end = u1;                      // an item never crosses a tile
                if (!mbar_wait(tempty_bar, (seg & 1u) ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                tc_fence_after();
                bool first = true;
                for (; ok && u < u_end; ++u) {
                    for (int c = 0; c < kt; ++c) {
                        if (!mbar_wait(full_bar(ps.stage), ps.phase, abortp, a.wait_ns)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sA = smem_base + ps.stage * MG_STAGE_BYTES;
                        const uint32_t sB = sA + MG_A_BYTES;
#pragma unroll
                        for (int kk = 0; kk < MG_BK / 16; ++kk) {
                            // MN-major, 128-byte swizzle: a token is a 128-byte row of 64 features,
                            // 8-token groups 1024 B apart (stride offset), the next 64 features one
                            // box further (leading offset); 16 tokens = 2 KB per MMA
                            const uint64_t db = smem_desc_sw128(sB + kk * 2048, MG_BOX_BYTES, 1024);
#pragma unroll
                            for (int h = 0; h < 2; ++h) {
                                const uint64_t da = smem_desc_sw128(sA + h * 2 * MG_BOX_BYTES + kk * 2048, MG_BOX_BYTES, 1024);
                                mma_bf16(tmem_base + h * 256u, da, db, idesc, (first && kk == 0) ? 0u : 1u);
                            }
                        }
                        first = false;
                        mma_commit(empty_bar(ps.stage));
                        ps.advance(MG_STAGES);
                    }
                }
                if (ok) mma_commit(tfull_bar);
                ++seg;
            }
            }
            if (!ok) {
                mma_commit(drain_bar);
                int never = 0;
                mbar_wait(drain_bar, 0, &never, kDrainLimitNs);
            }
        }
    } else {
        const uint32_t q = warp & 3;            // TMEM lane quarter
        const uint32_t half = (warp - 2) >> 2;  // rows 0-127 or 128-255 of the tile
        int seg = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < a.items; item += gridDim.x) {
        int64_t u0, u1;
        item_range(item, a.splits, a.chunk, a.B, u0, u1);
        int64_t u = u0;
        while (u < u1) {
            const int tile = (int)(u / a.B);
            const int64_t u_end = u1;
            const int tm = tile / a.ntn, tn = tile % a.ntn;
            if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar, seg & 1u, abortp, a.wait_ns))) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + half * 256u;
            const int m0 = tm * MG_BM + (int)half * 128 + (int)q * 32;   // first of this warp's 32 rows
            // The tile goes to S in 32x32 boxes: the warp writes a box to shared memory (lane =
            // row, 128-byte swizzle) and one TMA reduction adds it into S as full 128-byte lines;
            // rows and columns outside S are dropped by the hardware.
            const uint32_t box = staging_base + (uint32_t)(warp - 2) * MG_BOX_OUT;
            const uint32_t row_addr = box + (uint32_t)lane * 128u;
#pragma unroll 1
            for (int cc = 0; cc < MG_BN / 32; ++cc) {
                uint32_t r[32];
                tmem_ld32(taddr + cc * 32, r);
                tmem_ld_wait();
                const int n0 = tn * MG_BN + cc * 32;
                if (m0 < a.d_out && n0 < a.d_in) {            // uniform across the warp
                    if (lane == 0) bulk_wait_read_all();      // the previous box has been read
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        st_shared_v4(row_addr + (uint32_t)((j ^ (lane & 7)) << 4), r[4 * j], r[4 * j + 1], r[4 * j + 2],
                                     r[4 * j + 3]);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_reduce_add_2d(&tmS, box, n0, m0);
                        bulk_commit_group();
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar);
            u = u_end;
            ++seg;
        }
        }
        if (lane == 0) bulk_wait_all();   // this warp's reductions into S are complete
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(a.status, (int)ADLOCO_ERR_TIMEOUT);
}

// =====================================================================================
// direct kernel: per-sample weight-gradient tiles formed in TMEM, never written out
// =====================================================================================
// For one (output tile, sample i) unit the contraction over the sample's T tokens
// leaves the tile of G_i = D_i^T X_i in TMEM.  The epilogue squares and sums it into
// n_i and adds it to a register copy of the tile of S = sum_i G_i, which is flushed to
// global memory when the work item ends.  One GEMM (2 B T d_in d_out flops) thus
// yields both the per-sample norms and the gradient sum; it beats the Gram route
// whenever T exceeds d_in d_out / (d_in + d_out).
//
// The kernel takes a GROUP of layers (all with the same B and T): its work list runs
// over every layer's (chunk of samples, tile) items, so a whole micro-batch of a model is
// one persistent launch with one ramp and one tail, and the (tile, sample) units of
// layers whose tile count does not divide the SM count still spread evenly.  Items are
// handed out in list order through a global counter: a worker that finishes takes the
// next item, so all workers stay within a window of consecutive items -- the same few
// samples of the same layer, whose operands then stay in L2 (a fixed deal lets the workers
// drift apart over a long list and the DRAM traffic multiply).  The TMA thread draws the
// item and passes it to the other roles through a small queue in shared memory.
//
// PAIR = false: one CTA per SM, tile 128 (d_out) x 256 (d_in), stage = 48 KB.
// PAIR = true:  the two CTAs of a cluster share one MMA of 256 x 256: CTA r holds rows
//   128 r .. 128 r + 127 of the tile in its tensor memory, loads its own 128 rows of the
//   Delta operand and one half (128 columns) of the X operand -- 32 KB per stage for the
//   same math, i.e. 131 flops per byte brought into shared memory instead of 87.  The even
//   CTA issues the MMAs; byte counts of both CTAs' loads complete on its barriers; its
//   commits release the stages and publish the accumulators in both CTAs.
constexpr int DR_BM = 128;                          // d_out rows per CTA
constexpr int DR_BN = 256;                          // d_in columns per tile
constexpr int DR_BK = 64;                           // tokens per stage
constexpr int DR_BOX_BYTES = 64 * DR_BK * 2;        // 8 KB: 64 features x 64 tokens
constexpr int DR_A_BYTES = (DR_BM / 64) * DR_BOX_BYTES;
constexpr int DR_BOX_OUT = 32 * 16 * 4;             // per-epilogue-warp staging box: 32 rows x 16 fp32 columns
// Epilogue: four warps per TMEM lane quarter, each with four of the 16 column chunks (of
// 16) of a tile row, so a thread keeps 64 columns of the S tile in registers.
constexpr int DR_EPI_WARPS = 16;
constexpr int DR_STAGING = DR_EPI_WARPS * DR_BOX_OUT;
constexpr int DR_CHUNKS_MAX = 4;
constexpr int DR_COLS = DR_CHUNKS_MAX * 16;
constexpr int DR_THREADS = 64 + 32 * DR_EPI_WARPS;  // warp 0 TMA, warp 1 MMA, the rest epilogue
constexpr int DR_SCHED_Q = 8;                       // slots of the item queue between the TMA thread and the other roles

template <bool PAIR>
struct DirectCfg {
    static constexpr int B_BYTES = (PAIR ? 128 : DR_BN) / 64 * DR_BOX_BYTES;   // this CTA's share of the X operand
    static constexpr int STAGE_BYTES = DR_A_BYTES + B_BYTES;                   // 32 KB / 48 KB
    static constexpr int STAGES = PAIR ? 6 : 4;
    static constexpr int SMEM = STAGES * STAGE_BYTES + DR_STAGING + 1024 /*align*/ + 512 /*barriers*/;
    static constexpr int TILE_M = PAIR ? 256 : 128;                            // d_out rows per tile
};

struct alignas(64) DirectLayerMaps {
    CUtensorMap tmX, tmD, tmS;
};
struct DirectLayerMeta {
    float* S;            // [d_out, d_in], += ; may be null
    int d_in, d_out;
    int ntn, tiles;      // tiles along d_in, tiles of the layer
    int item_begin;      // first work item of the layer
    int pad;
};

// Work item j of a layer = (chunk of samples j / tiles, tile j % tiles): all tiles of one
// chunk of samples come first, so CTAs that run side by side read the same few samples
// and those samples' operands stay in L2.
template <int CAP>
struct DirectGroupArgs {
    DirectLayerMaps maps[CAP];
    DirectLayerMeta meta[CAP];
    int n_layers, B, T, kt;
    int chunk;           // samples per work item
    int total_items;
    int* counter;        // zero at launch: items beyond each worker's first are drawn from it
    float* n;            // [B], +=
    int* status;
    uint64_t wait_ns;    // bound of every in-kernel wait
};

struct DirectItem {
    int layer, tm, tn, b0, b1;
};

template <int CAP>
__device__ __forceinline__ DirectItem direct_decode(const DirectGroupArgs<CAP>& a, int item, int& layer_hint) {
    int l = layer_hint;
    while (l + 1 < a.n_layers && item >= a.meta[l + 1].item_begin) ++l;
    layer_hint = l;
    const DirectLayerMeta& m = a.meta[l];
    const int local = item - m.item_begin;
    const int k = local / m.tiles, tile = local - k * m.tiles;
    DirectItem it;
    it.layer = l;
    it.tm = tile / m.ntn;
    it.tn = tile - it.tm * m.ntn;
    it.b0 = k * a.chunk;
    it.b1 = it.b0 + a.chunk < a.B ? it.b0 + a.chunk : a.B;
    return it;
}

template <int CAP, bool PAIR>
__global__ void __launch_bounds__(DR_THREADS, 1)
direct_group_kernel(const __grid_constant__ DirectGroupArgs<CAP> a) {
    using Cfg = DirectCfg<PAIR>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int STAGE_BYTES = Cfg::STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t staging_base = smem_base + STAGES * STAGE_BYTES;
    const uint32_t bar_base = staging_base + DR_STAGING;
    auto full_bar = [&](uint32_t s) { return bar_base + 8u * s; };
    auto empty_bar = [&](uint32_t s) { return bar_base + 8u * (STAGES + s); };
    auto tfull_bar = [&](uint32_t b) { return bar_base + 8u * (2 * STAGES + b); };
    auto tempty_bar = [&](uint32_t b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
    const uint32_t drain_bar = bar_base + 8u * (2 * STAGES + 4);
    auto sched_full = [&](uint32_t s) { return bar_base + 8u * (2 * STAGES + 5 + s); };
    auto sched_empty = [&](uint32_t s) { return bar_base + 8u * (2 * STAGES + 5 + DR_SCHED_Q + s); };
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;
    __shared__ int sched_item[DR_SCHED_Q];

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = PAIR ? cluster_cta_rank() : 0u;          // 0 = the CTA that issues the MMAs and draws the items
    const int worker = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_workers = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (uint32_t s = 0; s < (uint32_t)STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (uint32_t b = 0; b < 2; ++b) {
            mbar_init(tfull_bar(b), 1);
            mbar_init(tempty_bar(b), DR_EPI_WARPS * (PAIR ? 2 : 1));    // the epilogue warps of both CTAs
        }
        mbar_init(drain_bar, 1);
        for (uint32_t s = 0; s < (uint32_t)DR_SCHED_Q; ++s) {
            mbar_init(sched_full(s), 1);
            // readers of a slot: the MMA thread and the epilogue warps; over a pair also the odd
            // CTA's TMA thread and epilogue warps
            mbar_init(sched_empty(s), (1 + DR_EPI_WARPS) * (PAIR ? 2 : 1));
        }
        fence_barrier_init();
    }
    if (warp == 1) {   // two 128 x 256 fp32 accumulators
        if constexpr (PAIR) { tmem_alloc_pair(smem_u32(&tmem_base_slot), 512); tmem_relinquish_pair(); }
        else { tmem_alloc(smem_u32(&tmem_base_slot), 512); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();    // the peer's barriers exist before anything is signalled on them
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;
    volatile int* abortp = &abort_flag;
    const int kt = a.kt;
    const uint32_t sched_empty_remote0 = PAIR ? map_to_cta(sched_empty(0), 0) : 0u;

    // item number k of this worker, as published by the drawing thread; -1 when the wait ran out.
    // Called by one thread (TMA / MMA role) or by all lanes of an epilogue warp.
    auto take_item = [&](int k, bool whole_warp) -> int {
        const uint32_t slot = (uint32_t)k % DR_SCHED_Q, ph = ((uint32_t)k / DR_SCHED_Q) & 1u;
        bool got = mbar_wait<PAIR>(sched_full(slot), ph, abortp, a.wait_ns);
        if (whole_warp) got = __all_sync(0xffffffffu, got);
        if (!got) return -1;
        const int item = *reinterpret_cast<volatile int*>(&sched_item[slot]);
        if (whole_warp) __syncwarp();
        if (!whole_warp || lane == 0) {
            if (PAIR && rank != 0) mbar_arrive_cluster(sched_empty_remote0 + 8u * slot);
            else mbar_arrive(sched_empty(slot));
        }
        return item;
    };

    if (warp == 0) {
        if (lane == 0) {
            PipeState ps;
            uint32_t issued = 0;
            bool ok = true;
            int hint = 0;
            int item = worker;                      // the first item needs no draw
            for (int k = 0; ok; ++k) {
                if (rank == 0) {
                    // publish item k to the other roles (and to the peer CTA)
                    const uint32_t slot = (uint32_t)k % DR_SCHED_Q, ph = ((uint32_t)k / DR_SCHED_Q) & 1u;
                    if (!mbar_wait<PAIR>(sched_empty(slot), ph ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    *reinterpret_cast<volatile int*>(&sched_item[slot]) = item;
                    if constexpr (PAIR) st_cluster_u32(map_to_cta(smem_u32(&sched_item[slot]), 1u), (uint32_t)item);
                    mbar_arrive(sched_full(slot));
                    if constexpr (PAIR) mbar_arrive_cluster(map_to_cta(sched_full(slot), 1u));
                } else {
                    item = take_item(k, false);
                    if (item < 0) { ok = false; break; }
                }
                if (item >= a.total_items) break;   // the list is exhausted: every role has been told
                // draw the next item now, its latency hides behind this item's copies
                int next_item = 0;
                if (rank == 0) next_item = n_workers + atomicAdd(a.counter, 1);
                const DirectItem it = direct_decode(a, item, hint);
                const CUtensorMap* tmD = &a.maps[it.layer].tmD;
                const CUtensorMap* tmX = &a.maps[it.layer].tmX;
                const int row0 = it.tm * Cfg::TILE_M + (int)rank * DR_BM;              // this CTA's d_out rows
                const int col0 = it.tn * DR_BN + (PAIR ? (int)rank * 128 : 0);         // this CTA's d_in columns
                for (int i = it.b0; ok && i < it.b1; ++i) {
                    for (int c = 0; c < kt; ++c) {
                        if (!mbar_wait(empty_bar(ps.stage), ps.phase ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                        const uint32_t sA = smem_base + ps.stage * STAGE_BYTES;
                        const uint32_t sB = sA + DR_A_BYTES;
                        if constexpr (PAIR) {
                            const uint32_t bar = map_to_cta(full_bar(ps.stage), 0);
                            if (rank == 0) mbar_arrive_expect_tx(full_bar(ps.stage), 2 * STAGE_BYTES);
#pragma unroll
                            for (int mb = 0; mb < DR_BM / 64; ++mb)
                                tma_load_3d_pair(sA + mb * DR_BOX_BYTES, tmD, bar, row0 + mb * 64, c * DR_BK, i);
#pragma unroll
                            for (int nb = 0; nb < 2; ++nb)
                                tma_load_3d_pair(sB + nb * DR_BOX_BYTES, tmX, bar, col0 + nb * 64, c * DR_BK, i);
                        } else {
                            mbar_arrive_expect_tx(full_bar(ps.stage), STAGE_BYTES);
#pragma unroll
                            for (int mb = 0; mb < DR_BM / 64; ++mb)
                                tma_load_3d(sA + mb * DR_BOX_BYTES, tmD, full_bar(ps.stage), row0 + mb * 64, c * DR_BK, i);
#pragma unroll
                            for (int nb = 0; nb < DR_BN / 64; ++nb)
                                tma_load_3d(sB + nb * DR_BOX_BYTES, tmX, full_bar(ps.stage), col0 + nb * 64, c * DR_BK, i);
                        }
                        ++issued;
                        ps.advance(STAGES);
                    }
                }
                item = next_item;
            }
            if (!ok) {
                // leaving after a time-out: let the copies still in flight land first
                if constexpr (PAIR) {
                    // their byte counts complete on the even CTA's barriers, which the odd CTA cannot
                    // wait on: both sit out a grace period far beyond the flight time of a copy
                    st_cluster_u32(map_to_cta(smem_u32(&abort_flag), rank ^ 1u), 1u);
                    const uint64_t t0 = globaltimer_ns();
                    while (globaltimer_ns() - t0 < kPairGraceNs) { }
                } else {
                    PipeState q = ps;
                    const uint32_t back = issued < (uint32_t)STAGES ? issued : (uint32_t)STAGES;
                    for (uint32_t r = 0; r < back; ++r) {
                        if (q.stage == 0) { q.stage = STAGES - 1; q.phase ^= 1u; } else { --q.stage; }
                        int never = 0;
                        mbar_wait(full_bar(q.stage), q.phase, &never, kDrainLimitNs);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // both operands MN-major; over a pair the MMA spans 256 rows (128 per CTA)
            constexpr uint32_t idesc = idesc_bf16_f32(PAIR ? 256 : DR_BM, DR_BN, 1, 1);
            PipeState ps;
            bool ok = true;
            int n_unit = 0;
            int hint = 0;
            for (int k = 0; ok; ++k) {
                const int item = take_item(k, false);
                if (item < 0) { ok = false; break; }
                if (item >= a.total_items) break;
                const DirectItem it = direct_decode(a, item, hint);
                for (int i = it.b0; ok && i < it.b1; ++i, ++n_unit) {
                    const uint32_t buf = n_unit & 1, use = n_unit >> 1;
                    if (!mbar_wait<PAIR>(tempty_bar(buf), (use & 1u) ^ 1u, abortp, a.wait_ns)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t acc = tmem_base + buf * 256u;
                    for (int c = 0; c < kt; ++c) {
                        if (!mbar_wait(full_bar(ps.stage), ps.phase, abortp, a.wait_ns)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t sA = smem_base + ps.stage * STAGE_BYTES;
                        const uint32_t sB = sA + DR_A_BYTES;
#pragma unroll
                        for (int kk = 0; kk < DR_BK / 16; ++kk) {
                            // MN-major, 128-byte swizzle: a token is a 128-byte row of 64 features, 8-token
                            // groups 1024 B apart (stride offset), the next 64 features one box further
                            // (leading offset); 16 tokens = 2 KB per MMA
                            const uint64_t da = smem_desc_sw128(sA + kk * 2048, DR_BOX_BYTES, 1024);
                            const uint64_t db = smem_desc_sw128(sB + kk * 2048, DR_BOX_BYTES, 1024);
                            if constexpr (PAIR) mma_bf16_pair(acc, da, db, idesc, (c == 0 && kk == 0) ? 0u : 1u);
                            else mma_bf16(acc, da, db, idesc, (c == 0 && kk == 0) ? 0u : 1u);
                        }
                        if constexpr (PAIR) mma_commit_pair(empty_bar(ps.stage), 3);   // the stage is free in both CTAs
                        else mma_commit(empty_bar(ps.stage));
                        ps.advance(STAGES);
                    }
                    if (ok) {
                        if constexpr (PAIR) mma_commit_pair(tfull_bar(buf), 3);
                        else mma_commit(tfull_bar(buf));
                    }
                }
            }
            if (!ok) {
                if constexpr (PAIR) {
                    st_cluster_u32(map_to_cta(smem_u32(&abort_flag), 1u), 1u);
                    mma_commit_pair(drain_bar, 1);
                } else {
                    mma_commit(drain_bar);
                }
                int never = 0;
                mbar_wait(drain_bar, 0, &never, kDrainLimitNs);
            }
        }
    } else {
        const uint32_t q = warp & 3;            // TMEM lane quarter: rows 32q .. 32q+31 of this CTA's part of the tile
        const uint32_t part = (warp - 2) >> 2;  // which column slice of the tile: chunks [c_begin, c_begin + n_chunks)
        const int c_begin = (int)part * DR_CHUNKS_MAX;
        constexpr int n_chunks = DR_CHUNKS_MAX;
        const uint32_t tempty_remote0 = PAIR ? map_to_cta(tempty_bar(0), 0) : 0u;
        float sacc[DR_COLS];                    // this thread's row of the S tile (its column slice)
#pragma unroll
        for (int e = 0; e < DR_COLS; ++e) sacc[e] = 0.f;
        int n_unit = 0;
        bool ok = true;
        int hint = 0;
        for (int k = 0; ok; ++k) {
            const int item = take_item(k, true);
            if (item < 0) { ok = false; break; }
            if (item >= a.total_items) break;
            const DirectItem it = direct_decode(a, item, hint);
            for (int i = it.b0; i < it.b1; ++i, ++n_unit) {
                const uint32_t buf = n_unit & 1, use = n_unit >> 1;
                if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(buf), use & 1u, abortp, a.wait_ns))) { ok = false; break; }
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((q * 32u) << 16) + buf * 256u + (uint32_t)c_begin * 16u;
                float sq = 0.f;
#pragma unroll
                for (int cc = 0; cc < DR_CHUNKS_MAX; ++cc) {
                    if (cc < n_chunks) {             // uniform across the warp
                        uint32_t r[16];
                        tmem_ld16(taddr + cc * 16, r);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 16; ++e) {
                            const float v = __uint_as_float(r[e]);
                            sq = fmaf(v, v, sq);
                            sacc[cc * 16 + e] += v;
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (PAIR) mbar_arrive_cluster(tempty_remote0 + 8u * buf);   // the even CTA's barrier
                    else mbar_arrive(tempty_bar(buf));
                }
                const float w = warp_sum_f(sq);
                if (lane == 0) atomicAdd(a.n + i, w);
            }
            // end of the item: add this warp's 32 rows x its column slice into S, 16 columns at a
            // time: the warp lays a 32 x 16 box out in shared memory (lane = row) and one TMA
            // reduction adds it into S; rows and columns outside S are dropped by the hardware
            const DirectLayerMeta& lm = a.meta[it.layer];
            const int m0 = it.tm * Cfg::TILE_M + (int)rank * DR_BM + (int)q * 32;
            const int n_base = it.tn * DR_BN + c_begin * 16;
            const uint32_t box = staging_base + (uint32_t)(warp - 2) * DR_BOX_OUT;
            const uint32_t row_addr = box + (uint32_t)lane * 64u;
            const bool flush = ok && lm.S != nullptr && m0 < lm.d_out;     // uniform across the warp
#pragma unroll
            for (int cc = 0; cc < DR_CHUNKS_MAX; ++cc) {
                if (flush && cc < n_chunks && n_base + cc * 16 < lm.d_in) {
                    if (lane == 0) bulk_wait_read_all();                 // the previous box has been read
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        st_shared_v4(row_addr + (uint32_t)(j << 4), __float_as_uint(sacc[cc * 16 + 4 * j]),
                                     __float_as_uint(sacc[cc * 16 + 4 * j + 1]), __float_as_uint(sacc[cc * 16 + 4 * j + 2]),
                                     __float_as_uint(sacc[cc * 16 + 4 * j + 3]));
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_reduce_add_2d(&a.maps[it.layer].tmS, box, n_base + cc * 16, m0);
                        bulk_commit_group();
                    }
                }
#pragma unroll
                for (int e = 0; e < 16; ++e) sacc[cc * 16 + e] = 0.f;
            }
        }
        if (lane == 0) bulk_wait_all();   // this warp's reductions into S are complete
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();   // neither CTA frees tensor memory or leaves while its peer still works
    if (warp == 1) {
        tc_fence_after();
        if constexpr (PAIR) tmem_dealloc_pair(tmem_base, 512);
        else tmem_dealloc(tmem_base, 512);
    }
    if (threadIdx.x == 0 && abort_flag) atomicExch(a.status, (int)ADLOCO_ERR_TIMEOUT);
}

// =====================================================================================
// host side
// =====================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn(adloco_ctx* ctx) {
    // looked up once; the initialisation of a function-local static is thread-safe
    static const EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        const cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
        if (e != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    if (!fn) set_cuda_error(ctx, cudaErrorUnknown, "cuTensorMapEncodeTiled entry point");
    return fn;
}

// bf16 tensor [B, T, d] (d contiguous) as a 3-D map {d, T, B} with a {64, box_tokens, 1}
// box and 128-byte swizzle; out-of-range rows and columns read as zero.
static int make_map(adloco_ctx* ctx, CUtensorMap* m, const void* base, int64_t B, int64_t T, int64_t d,
                    uint32_t box_tokens) {
    EncodeTiledFn fn = encode_fn(ctx);
    if (!fn) return ADLOCO_ERR_CUDA;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)T, (cuuint64_t)B};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)T * (cuuint64_t)d * 2};
    const cuuint32_t box[3] = {64, box_tokens, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return ADLOCO_ERR_CUDA;
    }
    return ADLOCO_OK;
}

// fp32 matrix [rows, cols] (cols contiguous) as a 2-D map with a 32-row box of box_cols
// columns: 32 columns with the 128-byte swizzle, 16 columns unswizzled
static int make_map_f32(adloco_ctx* ctx, CUtensorMap* m, float* base, int64_t rows, int64_t cols, uint32_t box_cols) {
    EncodeTiledFn fn = encode_fn(ctx);
    if (!fn) return ADLOCO_ERR_CUDA;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    const cuuint32_t box[2] = {box_cols, 32};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "cuTensorMapEncodeTiled (fp32) failed with CUresult %d", (int)r);
        return ADLOCO_ERR_CUDA;
    }
    return ADLOCO_OK;
}

// Encoded tensor maps are kept per context, keyed by what determines them (base pointer,
// extents, box, element type), so a layer that comes back every micro-batch is encoded once.
struct MapKey {
    const void* base;
    int64_t e0, e1, e2;
    uint32_t box, f32;
    bool operator==(const MapKey& o) const {
        return base == o.base && e0 == o.e0 && e1 == o.e1 && e2 == o.e2 && box == o.box && f32 == o.f32;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        uint64_t h = reinterpret_cast<uintptr_t>(k.base) * 0x9E3779B97F4A7C15ull;
        for (uint64_t v : {(uint64_t)k.e0, (uint64_t)k.e1, (uint64_t)k.e2, (uint64_t)k.box, (uint64_t)k.f32})
            h = (h ^ v) * 0x100000001B3ull + (h >> 29);
        return (size_t)h;
    }
};
struct MapCache {
    std::mutex mutex;
    std::unordered_map<MapKey, CUtensorMap, MapKeyHash> maps;
};
constexpr size_t kMapCacheLimit = 8192;   // entries; beyond it the cache starts over

static MapCache* map_cache(adloco_ctx* ctx) {
    static std::mutex create_mutex;
    std::lock_guard<std::mutex> lock(create_mutex);
    if (!ctx->tensor_maps) ctx->tensor_maps = new (std::nothrow) MapCache();
    return static_cast<MapCache*>(ctx->tensor_maps);
}
void free_tensor_map_cache(adloco_ctx* ctx) {
    delete static_cast<MapCache*>(ctx->tensor_maps);
    ctx->tensor_maps = nullptr;
}

template <typename Encode>
static int cached_lookup(adloco_ctx* ctx, const MapKey& key, CUtensorMap* out, Encode encode) {
    MapCache* c = map_cache(ctx);
    if (!c) return encode(out);
    std::lock_guard<std::mutex> lock(c->mutex);
    auto it = c->maps.find(key);
    if (it != c->maps.end()) { *out = it->second; return ADLOCO_OK; }
    const int rc = encode(out);
    if (rc != ADLOCO_OK) return rc;
    if (c->maps.size() >= kMapCacheLimit) c->maps.clear();
    c->maps.emplace(key, *out);
    return ADLOCO_OK;
}
static int cached_map(adloco_ctx* ctx, CUtensorMap* m, const void* base, int64_t B, int64_t T, int64_t d,
                      uint32_t box_tokens) {
    const MapKey key{base, B, T, d, box_tokens, 0u};
    return cached_lookup(ctx, key, m, [&](CUtensorMap* out) { return make_map(ctx, out, base, B, T, d, box_tokens); });
}
static int cached_map_f32(adloco_ctx* ctx, CUtensorMap* m, float* base, int64_t rows, int64_t cols, uint32_t box_cols) {
    const MapKey key{base, rows, cols, 0, box_cols, 1u};
    return cached_lookup(ctx, key, m, [&](CUtensorMap* out) { return make_map_f32(ctx, out, base, rows, cols, box_cols); });
}

int launch_gram_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                       int64_t d_out, float* n, int accumulate_norms, cudaStream_t st) {
    CUtensorMap tmX, tmD;
    int rc = cached_map(ctx, &tmX, X, B, T, d_in, GR_TILE);
    if (rc != ADLOCO_OK) return rc;
    rc = cached_map(ctx, &tmD, D, B, T, d_out, GR_TILE);
    if (rc != ADLOCO_OK) return rc;
    GramArgs a;
    a.B = (int)B; a.T = (int)T; a.d_in = (int)d_in; a.d_out = (int)d_out;
    a.nt = (int)((T + GR_TILE - 1) / GR_TILE);
    int64_t fulls = 0;
    for (int ti = 0; ti < a.nt; ++ti) fulls += (a.nt - ti) / 2;
    const int64_t halves = (a.nt + 1) / 2;
    if ((fulls + halves) * B > 0x7fffffff) return ADLOCO_ERR_UNSUPPORTED;
    a.full_per_sample = (int)fulls;
    a.half_per_sample = (int)halves;
    a.n_full = (int)(fulls * B);
    a.total_items = (int)((fulls + halves) * B);
    a.n = n; a.status = ctx->gemm_status; a.wait_ns = ctx->wait_limit_ns;
    if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
    static std::atomic<bool> attr_set[64];   // the attribute is per device
    if (!attr_set[ctx->device & 63].load()) {
        ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(gram_sqnorm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GR_SMEM));
        attr_set[ctx->device & 63].store(true);
    }
    const int grid = a.total_items < ctx->sm_count ? a.total_items : ctx->sm_count;
    gram_sqnorm_kernel<<<grid, GR_THREADS, GR_SMEM, st>>>(tmX, tmD, a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// The CTA-pair form of the Gram kernel
int launch_gram_pair(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                     int64_t d_out, float* n, int accumulate_norms, cudaStream_t st) {
    CUtensorMap tmX, tmD;
    int rc = cached_map(ctx, &tmX, X, B, T, d_in, GR_TILE);
    if (rc != ADLOCO_OK) return rc;
    rc = cached_map(ctx, &tmD, D, B, T, d_out, GR_TILE);
    if (rc != ADLOCO_OK) return rc;
    GramPairArgs a;
    a.B = (int)B; a.T = (int)T; a.d_in = (int)d_in; a.d_out = (int)d_out;
    a.nt = (int)((T + GR_TILE - 1) / GR_TILE);
    a.m = (a.nt + 1) / 2;
    const int64_t rects = (int64_t)a.m * (a.m + 1) / 2;
    if (rects * B > 0x3fffffff) return ADLOCO_ERR_UNSUPPORTED;
    a.rects = (int)rects;
    a.total_items = (int)(rects * B);
    a.n = n; a.status = ctx->gemm_status; a.wait_ns = ctx->wait_limit_ns;
    if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
    a.counter = ctx->sched_counters + (ctx->sched_next.fetch_add(1) % kSchedCounters);
    ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(a.counter, 0, sizeof(int), st));
    static std::atomic<bool> attr_set[64];   // the attribute is per device
    if (!attr_set[ctx->device & 63].load()) {
        ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(gram_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GP_SMEM));
        attr_set[ctx->device & 63].store(true);
    }
    const int workers = ctx->sm_count / 2;
    const int grid_workers = a.total_items < workers ? a.total_items : workers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * grid_workers));
    cfg.blockDim = dim3(GP_THREADS);
    cfg.dynamicSmemBytes = GP_SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ADLOCO_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, gram_pair_kernel, tmX, tmD, a));
    ctx->launches++;
    return ADLOCO_OK;
}

// the scatter-add of the gradient sum, shared by both routes of the norms
static int launch_embed_scatter(adloco_ctx* ctx, const int* ids, const void* D, int64_t B, int64_t T, int64_t d, int64_t V,
                                float* S, int accumulate_sum, cudaStream_t st) {
    if (!accumulate_sum) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(S, 0, (size_t)V * (size_t)d * sizeof(float), st));
    const int64_t tokens = B * T;
    int64_t blocks = (tokens + 7) / 8;
    const int64_t cap = (int64_t)ctx->sm_count * 8;
    if (blocks > cap) blocks = cap;
    embed_scatter_kernel<<<(unsigned)blocks, 256, 0, st>>>(ids, static_cast<const __nv_bfloat16*>(D), tokens, (int)d, (int)V, S);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_embedding(adloco_ctx* ctx, const int* ids, const void* D, int64_t B, int64_t T, int64_t d, int64_t V,
                     float* n, int accumulate_norms, float* S, int accumulate_sum, cudaStream_t st) {
    if (T <= ES_MAX_T && B <= 65535) {
        // the streaming form: every delta row read once
        EmbedSegArgs ea;
        ea.ids = ids; ea.D = static_cast<const __nv_bfloat16*>(D);
        ea.T = (int)T; ea.d = (int)d; ea.V = (int)V; ea.n = n;
        int H = 64;
        while (H < 2 * T) H <<= 1;
        ea.H = H;
        int64_t chunks = (2 * (int64_t)ctx->sm_count) / B;             // all blocks resident at once, two per SM
        const int64_t most = (T + ES_WARPS - 1) / ES_WARPS;
        if (chunks > most) chunks = most;
        if (chunks > 32) chunks = 32;
        if (chunks < 1) chunks = 1;
        ea.chunks = (int)chunks;
        const size_t smem = ((size_t)3 * H + (size_t)4 * T) * sizeof(int);
        if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
        static std::atomic<bool> attr_set[64];   // the attribute is per device
        if (!attr_set[ctx->device & 63].load()) {
            ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(embed_segment_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                      (int)(((size_t)3 * 2 * ES_MAX_T + (size_t)4 * ES_MAX_T) * sizeof(int))));
            attr_set[ctx->device & 63].store(true);
        }
        embed_segment_kernel<<<dim3((unsigned)chunks, (unsigned)B), ES_THREADS, smem, st>>>(ea);
        ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
        ctx->launches++;
        if (S) return launch_embed_scatter(ctx, ids, D, B, T, d, V, S, accumulate_sum, st);
        return ADLOCO_OK;
    }
    CUtensorMap tmD;
    int rc = cached_map(ctx, &tmD, D, B, T, d, GR_TILE);
    if (rc != ADLOCO_OK) return rc;
    EmbedArgs ea;
    GramArgs& a = ea.g;
    a.B = (int)B; a.T = (int)T; a.d_in = 0; a.d_out = (int)d;
    a.nt = (int)((T + GR_TILE - 1) / GR_TILE);
    int64_t fulls = 0;
    for (int ti = 0; ti < a.nt; ++ti) fulls += (a.nt - ti) / 2;
    const int64_t halves = (a.nt + 1) / 2;
    if ((fulls + halves) * B > 0x7fffffff) return ADLOCO_ERR_UNSUPPORTED;
    a.full_per_sample = (int)fulls;
    a.half_per_sample = (int)halves;
    a.n_full = (int)(fulls * B);
    a.total_items = (int)((fulls + halves) * B);
    a.n = n; a.status = ctx->gemm_status; a.wait_ns = ctx->wait_limit_ns;
    ea.ids = ids;
    ea.V = (int)V;
    if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
    static std::atomic<bool> attr_set[64];   // the attribute is per device
    if (!attr_set[ctx->device & 63].load()) {
        ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(embed_gram_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, GR_SMEM));
        attr_set[ctx->device & 63].store(true);
    }
    const int grid = a.total_items < ctx->sm_count ? a.total_items : ctx->sm_count;
    embed_gram_kernel<<<grid, GR_THREADS, GR_SMEM, st>>>(tmD, ea);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    if (S) return launch_embed_scatter(ctx, ids, D, B, T, d, V, S, accumulate_sum, st);
    return ADLOCO_OK;
}

int launch_mean_grad(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                     int64_t d_out, float* S, int accumulate_sum, cudaStream_t st) {
    CUtensorMap tmX, tmD;
    int rc = cached_map(ctx, &tmX, X, B, T, d_in, MG_BK);
    if (rc != ADLOCO_OK) return rc;
    rc = cached_map(ctx, &tmD, D, B, T, d_out, MG_BK);
    if (rc != ADLOCO_OK) return rc;
    CUtensorMap tmS;
    rc = cached_map_f32(ctx, &tmS, S, d_out, d_in, 32);
    if (rc != ADLOCO_OK) return rc;
    MeanGradArgs a;
    a.B = (int)B; a.T = (int)T; a.d_in = (int)d_in; a.d_out = (int)d_out;
    a.ntm = (int)((d_out + MG_BM - 1) / MG_BM);
    a.ntn = (int)((d_in + MG_BN - 1) / MG_BN);
    if ((int64_t)a.ntm * a.ntn * B > 0x3fffffff) return ADLOCO_ERR_UNSUPPORTED;
    const SplitPlan sp = make_split((int64_t)a.ntm * a.ntn, B, ctx->sm_count);
    a.splits = sp.splits; a.chunk = sp.chunk; a.items = sp.items;
    a.S = S; a.status = ctx->gemm_status; a.wait_ns = ctx->wait_limit_ns;
    if (!accumulate_sum) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(S, 0, (size_t)d_out * (size_t)d_in * sizeof(float), st));
    static std::atomic<bool> attr_set[64];   // the attribute is per device
    if (!attr_set[ctx->device & 63].load()) {
        ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(mean_grad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, MG_SMEM));
        attr_set[ctx->device & 63].store(true);
    }
    const int grid = a.items < ctx->sm_count ? a.items : ctx->sm_count;
    mean_grad_kernel<<<grid, MG_THREADS, MG_SMEM, st>>>(tmX, tmD, tmS, a);
    ADLOCO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches++;
    return ADLOCO_OK;
}

// Samples per work item: the count that minimises the time of the busiest worker.  Items
// are all alike, so the workers finish them in rounds: rounds x (samples per item + the
// flush of the S tile, measured at about 0.4 of a sample's time).  Capped at 16 so that
// the samples the workers walk through side by side stay resident in L2.
static int choose_chunk(int64_t total_tiles, int64_t B, int workers) {
    int best = 1;
    double best_cost = 1e300;
    const int64_t cap = B < 16 ? B : 16;
    for (int64_t c = 1; c <= cap; ++c) {
        const int64_t items = total_tiles * ((B + c - 1) / c);
        const int64_t rounds = (items + workers - 1) / workers;
        const double cost = (double)rounds * ((double)c + 0.4);
        if (cost <= best_cost) { best_cost = cost; best = (int)c; }
    }
    return best;
}

template <int CAP, bool PAIR>
static int launch_direct_group_t(adloco_ctx* ctx, const adloco_linear_layer* layers, int n_layers, int64_t B, int64_t T,
                                 float* n, cudaStream_t st) {
    using Cfg = DirectCfg<PAIR>;
    static DirectGroupArgs<CAP> a;             // 20 KB for CAP = 48: kept off the stack
    static std::mutex args_mutex;              // the staging copy above is shared by all callers
    std::lock_guard<std::mutex> lock(args_mutex);
    const int workers = PAIR ? ctx->sm_count / 2 : ctx->sm_count;
    int64_t total_tiles = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int64_t ntm = (layers[l].d_out + Cfg::TILE_M - 1) / Cfg::TILE_M;
        const int64_t ntn = (layers[l].d_in + DR_BN - 1) / DR_BN;
        total_tiles += ntm * ntn;
    }
    const int chunk = choose_chunk(total_tiles, B, workers);
    const int64_t n_chunks = (B + chunk - 1) / chunk;
    if (total_tiles * n_chunks > 0x3fffffff) return ADLOCO_ERR_UNSUPPORTED;
    int item = 0;
    for (int l = 0; l < n_layers; ++l) {
        const adloco_linear_layer& L = layers[l];
        int rc = cached_map(ctx, &a.maps[l].tmX, L.X, B, T, L.d_in, DR_BK);
        if (rc != ADLOCO_OK) return rc;
        rc = cached_map(ctx, &a.maps[l].tmD, L.D, B, T, L.d_out, DR_BK);
        if (rc != ADLOCO_OK) return rc;
        if (L.grad_sum) {
            rc = cached_map_f32(ctx, &a.maps[l].tmS, L.grad_sum, L.d_out, L.d_in, 16);
            if (rc != ADLOCO_OK) return rc;
        } else {
            a.maps[l].tmS = a.maps[l].tmX;   // never used by the kernel when S is null
        }
        DirectLayerMeta& m = a.meta[l];
        m.S = L.grad_sum;
        m.d_in = (int)L.d_in; m.d_out = (int)L.d_out;
        m.ntn = (int)((L.d_in + DR_BN - 1) / DR_BN);
        m.tiles = (int)((L.d_out + Cfg::TILE_M - 1) / Cfg::TILE_M) * m.ntn;
        m.item_begin = item;
        m.pad = 0;
        item += m.tiles * (int)n_chunks;
    }
    a.n_layers = n_layers; a.B = (int)B; a.T = (int)T; a.kt = (int)((T + DR_BK - 1) / DR_BK);
    a.chunk = chunk; a.total_items = item;
    a.n = n; a.status = ctx->gemm_status; a.wait_ns = ctx->wait_limit_ns;
    // every launch gets a work counter of its own from a small pool, so that launches on several
    // streams do not share one
    a.counter = ctx->sched_counters + (ctx->sched_next.fetch_add(1) % kSchedCounters);
    ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(a.counter, 0, sizeof(int), st));
    auto kern = direct_group_kernel<CAP, PAIR>;
    static std::atomic<bool> attr_set[64];   // the attribute is per device
    if (!attr_set[ctx->device & 63].load()) {
        ADLOCO_CUDA_TRY(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM));
        attr_set[ctx->device & 63].store(true);
    }
    const int grid_workers = item < workers ? item : workers;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * grid_workers : grid_workers));
    cfg.blockDim = dim3(DR_THREADS);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    if (PAIR) {
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    ADLOCO_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, kern, a));
    ctx->launches++;
    return ADLOCO_OK;
}

int launch_direct_group(adloco_ctx* ctx, const adloco_linear_layer* layers, int n_layers, int64_t B, int64_t T,
                        float* n, int accumulate_norms, int accumulate_sum, int pair, cudaStream_t st) {
    if (!accumulate_norms) ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(n, 0, (size_t)B * sizeof(float), st));
    if (!accumulate_sum)
        for (int l = 0; l < n_layers; ++l)
            if (layers[l].grad_sum)
                ADLOCO_CUDA_TRY(ctx, cudaMemsetAsync(layers[l].grad_sum, 0,
                                                     (size_t)layers[l].d_out * (size_t)layers[l].d_in * sizeof(float), st));
    // as many layers per launch as the kernel's argument block holds
    for (int l0 = 0; l0 < n_layers; l0 += kDirectGroupCap) {
        const int nl = n_layers - l0 < kDirectGroupCap ? n_layers - l0 : kDirectGroupCap;
        int rc;
        if (nl == 1) rc = pair ? launch_direct_group_t<1, true>(ctx, layers + l0, 1, B, T, n, st)
                               : launch_direct_group_t<1, false>(ctx, layers + l0, 1, B, T, n, st);
        else rc = pair ? launch_direct_group_t<kDirectGroupCap, true>(ctx, layers + l0, nl, B, T, n, st)
                       : launch_direct_group_t<kDirectGroupCap, false>(ctx, layers + l0, nl, B, T, n, st);
        if (rc != ADLOCO_OK) return rc;
    }
    return ADLOCO_OK;
}

int launch_direct_sqnorm(adloco_ctx* ctx, const void* X, const void* D, int64_t B, int64_t T, int64_t d_in,
                         int64_t d_out, float* n, int accumulate_norms, float* S, int accumulate_sum, int pair,
                         cudaStream_t st) {
    adloco_linear_layer L;
    L.X = X; L.D = D; L.d_in = d_in; L.d_out = d_out; L.grad_sum = S;
    return launch_direct_group(ctx, &L, 1, B, T, n, accumulate_norms, accumulate_sum, pair, st);
}

}  // namespace adloco
