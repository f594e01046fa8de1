// K7 -- datastore-side preprocessing: the keys of the datastore are the token embeddings
// of the corpus after the SAME three steps the query takes (Sections 3.2-3.4 of the paper:
// Eq. 1 z-scoring, v_l <- v W_l, Eq. 2 unit length), applied to N rows of LLM hidden
// states.  Unlike the per-step retrieval this is a real GEMM, [N x d_in] . [d_in x d], and
// it is tensor-bound: tcgen05.mma with TMEM accumulators, TMA-fed.
//
// Algebra.  With sigma_j = sqrt(Var_j + eps):
//     ((h - mu) / sigma - m) W  =  h W'  +  c,      W'[j][c] = W[j][c] / sigma_j,
//                                                   c[c]     = -sum_j (mu_j / sigma_j + m_j) W[j][c].
// The hidden states h enter the tensor cores exactly (they are stored in 16 bits); W' is
// split into two 16-bit terms (W' = hi + lo) and both products accumulate into the same
// fp32 accumulator, so the result carries fp32-level accuracy before the final rounding to
// the store dtype.  c is computed in float64 by a small kernel.
//
// One persistent CTA per SM, ten warps: warp 0 = TMA producer (per 64-column k-slab: two
// 128-row slabs of h, the hi and the lo slab of W'^T, all 128-byte swizzled); warp 1 =
// TMEM allocation + MMA issue (a 256-row tile = two 128-row accumulators of d columns);
// warps 2-9 = epilogue (a thread owns one row: adds c, takes the norm in a first pass over
// its accumulator row, scales, rounds and stores in a second).  Every wait is bounded.
#include <type_traits>

#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

// Arrives on the barrier at the same shared-memory offset in every CTA of `mask` once all
// MMAs issued so far by this thread have retired.
__device__ __forceinline__ void tc_commit2(uint64_t *bar, uint16_t mask)
{
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(
            smem_u32(bar)),
        "h"(mask)
        : "memory");
}

constexpr int kThreads = 10 * 32;
constexpr int kSubRows = 128;
constexpr int kTileRows = 2 * kSubRows;
constexpr int kSlabBytes = 128;
constexpr int kSlabElems = 64;
constexpr int kASlab = kSubRows * kSlabBytes;        // 16 KB
constexpr int kMaxStages = 6;


template <typename T> __device__ __forceinline__ float w_to_f32(T x);
template <> __device__ __forceinline__ float w_to_f32<__half>(__half x) { return __half2float(x); }
template <> __device__ __forceinline__ float w_to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T w_from_f32(float x);
template <> __device__ __forceinline__ __half w_from_f32<__half>(float x) { return __float2half_rn(x); }
template <> __device__ __forceinline__ __nv_bfloat16 w_from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }
template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b)
{
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b)
{
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&h);
}

// W'^T = (W / sigma)^T split into hi + lo, [d][kpad] K-major, zero padded; bias in float64.
template <typename T>
__global__ void build_prep_kernel(const T *__restrict__ W, const float *__restrict__ mean,
                                  const float *__restrict__ var, float eps_z, const float *__restrict__ pca_mean,
                                  int d_in, int d, int kpad, T *__restrict__ wt_hi, T *__restrict__ wt_lo,
                                  float *__restrict__ bias)
{
    const int c = blockIdx.x;                              // output column
    __shared__ double red[32];
    double acc = 0.0;
    for (int j = threadIdx.x; j < kpad; j += blockDim.x) {
        float hi = 0.f, lo = 0.f;
        if (j < d_in) {
            const float w = w_to_f32<T>(W[(size_t)j * d + c]);
            const float sigma = mean ? sqrtf(var[j] + eps_z) : 1.f;
            const float wp = w / sigma;
            const T h = w_from_f32<T>(wp);
            hi = w_to_f32<T>(h);
            lo = w_to_f32<T>(w_from_f32<T>(wp - hi));
            const double shift = (mean ? (double)mean[j] / (double)sigma : 0.0) + (pca_mean ? (double)pca_mean[j] : 0.0);
            acc -= shift * (double)w;
        }
        wt_hi[(size_t)c * kpad + j] = w_from_f32<T>(hi);
        wt_lo[(size_t)c * kpad + j] = w_from_f32<T>(lo);
    }
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
        bias[c] = (float)t;
    }
}

// Epilogue of one row: two passes over the thread's accumulator row in TMEM -- the squared
// length of v W' + c (Eq. 2), then scale, round to the store dtype and store 16 bytes at a time.
template <typename T>
__device__ __forceinline__ void finish_row(uint32_t row_addr, const float *bias_s, int d, float eps_n, T *out,
                                           long long row, long long N)
{
    float ss = 0.f;
    for (int c0 = 0; c0 < d; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(row_addr + (uint32_t)c0, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            const float x = __uint_as_float(r[i]) + bias_s[c0 + i];
            ss = fmaf(x, x, ss);
        }
    }
    const float inv = 1.0f / fmaxf(sqrtf(ss), eps_n);
    for (int c0 = 0; c0 < d; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(row_addr + (uint32_t)c0, r);
        tmem_ld_wait();
        if (row < N) {
            uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)row * d + c0);
#pragma unroll
            for (int v = 0; v < 4; ++v) {
                uint4 o;
                const int i = 8 * v;
                o.x = pack2<T>((__uint_as_float(r[i + 0]) + bias_s[c0 + i + 0]) * inv,
                               (__uint_as_float(r[i + 1]) + bias_s[c0 + i + 1]) * inv);
                o.y = pack2<T>((__uint_as_float(r[i + 2]) + bias_s[c0 + i + 2]) * inv,
                               (__uint_as_float(r[i + 3]) + bias_s[c0 + i + 3]) * inv);
                o.z = pack2<T>((__uint_as_float(r[i + 4]) + bias_s[c0 + i + 4]) * inv,
                               (__uint_as_float(r[i + 5]) + bias_s[c0 + i + 5]) * inv);
                o.w = pack2<T>((__uint_as_float(r[i + 6]) + bias_s[c0 + i + 6]) * inv,
                               (__uint_as_float(r[i + 7]) + bias_s[c0 + i + 7]) * inv);
                dst[v] = o;
            }
        }
    }
}

struct BuildArgs {
    long long N;
    int d_in, d, n_tiles, stages;
    int terms;               // 2: W' = hi + lo; 1: W' is exact in 16 bits (no z-score), lo is not read
    const float *bias;       // [d]
    void *out;               // [N][d] store dtype
    float eps_n;
    int *status;
    long long wait_cycles;   // bound of every device-side wait in cycles, 0 = default
    int lose_stage;          // test hook: the first CTA (pair) never receives stage (value-1); 0 = off
};

template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
build_keys_kernel(const __grid_constant__ CUtensorMap h_map, const __grid_constant__ CUtensorMap whi_map,
                  const __grid_constant__ CUtensorMap wlo_map, const BuildArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    const int kslabs = (a.d_in + kSlabElems - 1) / kSlabElems;
    const int b_slab = a.d * kSlabBytes;                    // one 64-column slab of W'^T (hi or lo)
    const int stage_bytes = 2 * kASlab + a.terms * b_slab;
    uint8_t *stages = base;
    float *bias_s = reinterpret_cast<float *>(stages + (size_t)n_stages * stage_bytes);
    uint64_t *full = reinterpret_cast<uint64_t *>(bias_s + 256);
    uint64_t *empty = full + kMaxStages;
    uint64_t *tfull = empty + kMaxStages;
    uint64_t *tempty = tfull + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int my_tiles = cta < a.n_tiles ? (a.n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * kslabs;
    const long long wl = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;   // bound of every wait below
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * a.d) tmem_cols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(tfull, 1);
        mbar_init(tempty, 8);
        mbar_fence_init();
    }
    for (int c = tid; c < a.d; c += kThreads) bias_s[c] = a.bias[c];
    if (warp == 1) {
        tmem_alloc(tmem_slot, tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&h_map);
            tma_prefetch_desc(&whi_map);
            tma_prefetch_desc(&wlo_map);
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
                const int tile = cta + (it / kslabs) * G;
                const int ks = it % kslabs;
                uint8_t *dst = stages + (size_t)s * stage_bytes;
                mbar_arrive_expect_tx(&full[s], (uint32_t)stage_bytes);
                // Test hook: CTA 0 "loses" the copies of one stage, so that the waits on it run out.
                if (a.lose_stage > 0 && cta == 0 && it == a.lose_stage - 1) {
                    issued = it + 1;
                    continue;
                }
                tma_load_2d(dst, &h_map, ks * kSlabElems, tile * kTileRows, &full[s]);
                tma_load_2d(dst + kASlab, &h_map, ks * kSlabElems, tile * kTileRows + kSubRows, &full[s]);
                tma_load_2d(dst + 2 * kASlab, &whi_map, ks * kSlabElems, 0, &full[s]);
                if (a.terms == 2) tma_load_2d(dst + 2 * kASlab + b_slab, &wlo_map, ks * kSlabElems, 0, &full[s]);
                issued = it + 1;
            }
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t kFmt = std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
            const uint32_t idesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((uint32_t)(a.d >> 3) << 17) |
                                   ((uint32_t)(kSubRows >> 4) << 24);
            bool ok = true;
            const bool two = a.terms == 2;
            for (int tl = 0; tl < my_tiles && ok; ++tl) {
                // one accumulator set: wait until the epilogue has drained the previous tile
                if (tl >= 1 && !mbar_wait(tempty, (tl - 1) & 1, wl)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < kslabs; ++ks) {
                    const int it = tl * kslabs + ks;
                    const int s = it % n_stages;
                    if (!mbar_wait(&full[s], (it / n_stages) & 1, wl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = smem_u32(stages + (size_t)s * stage_bytes);
                    const uint64_t bhi = make_desc(st + 2 * kASlab), blo = make_desc(st + 2 * kASlab + b_slab);
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        const uint64_t ad = make_desc(st + sub * kASlab);
                        const uint32_t dt = tmem_base + (uint32_t)(sub * a.d);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            umma_f16(dt, ad + 2 * k, bhi + 2 * k, idesc, (ks | k) != 0);
                            if (two) umma_f16(dt, ad + 2 * k, blo + 2 * k, idesc, 1);
                        }
                    }
                    tc_commit(&empty[s]);
                }
                if (!ok) break;
                tc_commit(tfull);
            }
            if (!ok) report_timeout(a.status);
        }
    } else {
        // epilogue: warps 2-5 own sub-tile 0, warps 6-9 sub-tile 1; lane group = warp & 3
        const int ew = warp - 2;
        const int sub = ew >> 2;
        const int lane_grp = warp & 3;
        const uint32_t row_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(sub * a.d);
        T *out = static_cast<T *>(a.out);
        bool dead = false;
        for (int tl = 0; tl < my_tiles; ++tl) {
            if (!dead && !mbar_wait(tfull, tl & 1, wl)) {
                report_timeout(a.status);
                dead = true;
            }
            dead = __any_sync(0xFFFFFFFFu, dead);
            tc_fence_after();
            const long long row = (long long)(cta + tl * G) * kTileRows + sub * kSubRows + lane_grp * 32 + lane;
            if (!dead) {
                finish_row<T>(row_addr, bias_s, a.d, a.eps_n, out, row, a.N);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ---- the same GEMM on CTA pairs ------------------------------------------------------------
// Two CTAs of a cluster (two SMs of one TPC) work as one: the leader (cluster rank 0) issues
// tcgen05.mma.cta_group::2 with M = 256 -- 128 rows of hidden states from each CTA's shared
// memory, and a W' slab of which each CTA holds HALF the rows (d/2 output columns).  Per
// 64-column k-slab a CTA therefore stages 2 x 16 KB of hidden states and d/2 x 128 B per W'
// term instead of d x 128 B: more stages fit and the L2 -> SM traffic for W' halves.  Each CTA
// owns 256 rows of a 512-row pair tile; its accumulators (two 128-row x d-column blocks) live
// in its own TMEM and are drained by its own epilogue warps.
//
// Barriers: full[s] lives in the leader and counts the TMA bytes of BOTH CTAs (the peer's
// loads complete on the leader's barrier); empty[s] and tfull exist in both CTAs and are
// signalled together by a multicast tcgen05.commit; tempty lives in the leader and collects
// the epilogue warps of both CTAs.  No TMA multicast anywhere.
template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
build_keys_pair_kernel(const __grid_constant__ CUtensorMap h_map, const __grid_constant__ CUtensorMap whi_map,
                       const __grid_constant__ CUtensorMap wlo_map, const BuildArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    const int kslabs = (a.d_in + kSlabElems - 1) / kSlabElems;
    const int b_half = (a.d / 2) * kSlabBytes;              // this CTA's half of a W' slab (hi or lo)
    const int stage_bytes = 2 * kASlab + a.terms * b_half;
    uint8_t *stages = base;
    float *bias_s = reinterpret_cast<float *>(stages + (size_t)n_stages * stage_bytes);
    uint64_t *full = reinterpret_cast<uint64_t *>(bias_s + 256);
    uint64_t *empty = full + kMaxStages;
    uint64_t *tfull = empty + kMaxStages;
    uint64_t *tempty = tfull + 1;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tempty + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int my_tiles = pair < a.n_tiles ? (a.n_tiles - pair + n_pairs - 1) / n_pairs : 0;   // 512-row pair tiles
    const int n_it = my_tiles * kslabs;
    const long long wl = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;   // bound of every wait below
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * a.d) tmem_cols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);          // used in the leader only
            mbar_init(&empty[s], 1);
        }
        mbar_init(tfull, 1);
        mbar_init(tempty, 16);               // 8 epilogue warps of each CTA (leader's copy is used)
        mbar_fence_init();
    }
    for (int c = tid; c < a.d; c += kThreads) bias_s[c] = a.bias[c];
    if (warp == 1) {
        tmem_alloc2(tmem_slot, tmem_cols);
        tmem_relinquish2();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&h_map);
            tma_prefetch_desc(&whi_map);
            if (a.terms == 2) tma_prefetch_desc(&wlo_map);
            bool ok = true;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wl)) {
                    report_timeout(a.status);
                    ok = false;
                    break;
                }
                const int tile = pair + (it / kslabs) * n_pairs;
                const int ks = it % kslabs;
                const int row0 = tile * (2 * kTileRows) + (int)rank * kTileRows;
                uint8_t *dst = stages + (size_t)s * stage_bytes;
                const uint32_t lead_full = mapa_rank(smem_u32(&full[s]), 0);
                if (rank == 0) mbar_arrive_expect_tx(&full[s], (uint32_t)(2 * stage_bytes));
                // Test hook: the leader of pair 0 "loses" its copies of one stage (the peer's still
                // arrive), so that the leader's barrier never completes and the waits on it run out.
                if (a.lose_stage > 0 && pair == 0 && rank == 0 && it == a.lose_stage - 1) continue;
                tma_load_2d_pair(dst, &h_map, ks * kSlabElems, row0, lead_full);
                tma_load_2d_pair(dst + kASlab, &h_map, ks * kSlabElems, row0 + kSubRows, lead_full);
                tma_load_2d_pair(dst + 2 * kASlab, &whi_map, ks * kSlabElems, (int)rank * (a.d / 2), lead_full);
                if (a.terms == 2)
                    tma_load_2d_pair(dst + 2 * kASlab + b_half, &wlo_map, ks * kSlabElems, (int)rank * (a.d / 2),
                                     lead_full);
            }
            if (!ok) {
                // copies of this CTA may still be in flight towards its shared memory: give them
                // time to land before the CTA can leave (bounded, about a millisecond)
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t kFmt = std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
            // M = 256 over the pair, N = d
            const uint32_t idesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((uint32_t)(a.d >> 3) << 17) |
                                   ((uint32_t)((2 * kSubRows) >> 4) << 24);
            bool ok = true;
            const bool two = a.terms == 2;
            for (int tl = 0; tl < my_tiles && ok; ++tl) {
                // one accumulator set: both epilogues have drained the previous tile
                if (tl >= 1 && !mbar_wait(tempty, (tl - 1) & 1, wl)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < kslabs; ++ks) {
                    const int it = tl * kslabs + ks;
                    const int s = it % n_stages;
                    if (!mbar_wait(&full[s], (it / n_stages) & 1, wl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = smem_u32(stages + (size_t)s * stage_bytes);
                    const uint64_t bhi = make_desc(st + 2 * kASlab), blo = make_desc(st + 2 * kASlab + b_half);
#pragma unroll
                    for (int sub = 0; sub < 2; ++sub) {
                        const uint64_t ad = make_desc(st + sub * kASlab);
                        const uint32_t dt = tmem_base + (uint32_t)(sub * a.d);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            umma2_f16(dt, ad + 2 * k, bhi + 2 * k, idesc, (ks | k) != 0);
                            if (two) umma2_f16(dt, ad + 2 * k, blo + 2 * k, idesc, 1);
                        }
                    }
                    tc_commit2(&empty[s], 3);            // frees the stage in both CTAs
                }
                if (!ok) break;
                tc_commit2(tfull, 3);                    // both epilogues may read their accumulators
            }
            if (!ok) report_timeout(a.status);
        }
    } else {
        // epilogue: warps 2-5 own sub-tile 0, warps 6-9 sub-tile 1; lane group = warp & 3
        const int ew = warp - 2;
        const int sub = ew >> 2;
        const int lane_grp = warp & 3;
        const uint32_t row_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(sub * a.d);
        const uint32_t lead_tempty = mapa_rank(smem_u32(tempty), 0);
        T *out = static_cast<T *>(a.out);
        bool dead = false;
        for (int tl = 0; tl < my_tiles; ++tl) {
            if (!dead && !mbar_wait(tfull, tl & 1, wl)) {
                report_timeout(a.status);
                dead = true;
            }
            dead = __any_sync(0xFFFFFFFFu, dead);
            tc_fence_after();
            const long long row = (long long)(pair + tl * n_pairs) * (2 * kTileRows) + (long long)rank * kTileRows +
                                  sub * kSubRows + lane_grp * 32 + lane;
            if (!dead) finish_row<T>(row_addr, bias_s, a.d, a.eps_n, out, row, a.N);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(lead_tempty);
        }
    }
    // Nobody leaves while the other CTA may still signal its barriers, read its shared memory
    // or write its TMEM.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, tmem_cols);
    }
}

}  // namespace

size_t build_keys_workspace_bytes(int d_in, int d)
{
    const size_t kpad = ((size_t)d_in + 63) / 64 * 64;
    return 2 * (size_t)d * kpad * 2 + 256 * sizeof(float) + 256;
}

cudaError_t launch_build_prep(const void *W, int dtype, const float *mean, const float *var, float eps_z,
                              const float *pca_mean, int d_in, int d, void *wt_hi, void *wt_lo, float *bias,
                              cudaStream_t stream)
{
    const int kpad = (d_in + 63) / 64 * 64;
    if (dtype == kF16)
        build_prep_kernel<__half><<<d, 256, 0, stream>>>(static_cast<const __half *>(W), mean, var, eps_z, pca_mean,
                                                          d_in, d, kpad, static_cast<__half *>(wt_hi),
                                                          static_cast<__half *>(wt_lo), bias);
    else
        build_prep_kernel<__nv_bfloat16><<<d, 256, 0, stream>>>(
            static_cast<const __nv_bfloat16 *>(W), mean, var, eps_z, pca_mean, d_in, d, kpad,
            static_cast<__nv_bfloat16 *>(wt_hi), static_cast<__nv_bfloat16 *>(wt_lo), bias);
    return cudaGetLastError();
}

cudaError_t launch_build_keys(const CUtensorMap &h_map, const CUtensorMap &whi_map, const CUtensorMap &wlo_map,
                              int dtype, long long N, int d_in, int d, int terms, int pair, const float *bias,
                              void *out, float eps_n, int *status, int grid, cudaStream_t stream, long long wait_cycles,
                              int lose_stage)
{
    BuildArgs a{};
    a.wait_cycles = wait_cycles;
    a.lose_stage = lose_stage;
    a.terms = terms == 1 ? 1 : 2;
    a.N = N;
    a.d_in = d_in;
    a.d = d;
    const int tile_rows = pair ? 2 * kTileRows : kTileRows;
    a.n_tiles = (int)((N + tile_rows - 1) / tile_rows);
    a.bias = bias;
    a.out = out;
    a.eps_n = eps_n;
    a.status = status;
    const size_t b_rows = pair ? (size_t)d / 2 : (size_t)d;          // W' rows staged per CTA
    const size_t stage = 2 * (size_t)kASlab + (size_t)a.terms * b_rows * kSlabBytes;
    const size_t fixed = 1024 + 256 * sizeof(float) + sizeof(uint64_t) * (2 * kMaxStages + 2) + 64;
    long long s = ((long long)227 * 1024 - (long long)fixed) / (long long)stage;
    if (s > kMaxStages) s = kMaxStages;
    if (s < 2) return cudaErrorInvalidValue;
    a.stages = (int)s;
    const size_t smem = fixed + (size_t)s * stage;
    cudaError_t e;
    if (!pair) {
        if (grid > a.n_tiles) grid = a.n_tiles;
        if (dtype == kF16) {
            auto k = build_keys_kernel<__half>;
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            k<<<grid, kThreads, smem, stream>>>(h_map, whi_map, wlo_map, a);
        } else {
            auto k = build_keys_kernel<__nv_bfloat16>;
            e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            k<<<grid, kThreads, smem, stream>>>(h_map, whi_map, wlo_map, a);
        }
        return cudaGetLastError();
    }
    // CTA pairs: clusters of two, one pair per two SMs
    int pairs = grid / 2;
    if (pairs > a.n_tiles) pairs = a.n_tiles;
    if (pairs < 1) pairs = 1;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (dtype == kF16) {
        auto k = build_keys_pair_kernel<__half>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        int max_clusters = 0;
        e = cudaOccupancyMaxActiveClusters(&max_clusters, k, &cfg);
        if (e != cudaSuccess) return e;
        if (max_clusters < 1) return cudaErrorLaunchOutOfResources;
        if (pairs > max_clusters) cfg.gridDim = dim3(2 * max_clusters);   // every pair must be resident
        return cudaLaunchKernelEx(&cfg, k, h_map, whi_map, wlo_map, a);
    }
    auto k = build_keys_pair_kernel<__nv_bfloat16>;
    e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int max_clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&max_clusters, k, &cfg);
    if (e != cudaSuccess) return e;
    if (max_clusters < 1) return cudaErrorLaunchOutOfResources;
    if (pairs > max_clusters) cfg.gridDim = dim3(2 * max_clusters);
    return cudaLaunchKernelEx(&cfg, k, h_map, whi_map, wlo_map, a);
}

}  // namespace dresd
