// K2+K3 (streaming path, 16-bit keys) -- Eq. 3 of the paper for every key:
// s_i = q . k_i, fused with the per-CTA top-n selection, for up to 8 queries
// per launch.  HBM-bound: every key byte is read exactly once.
//
// Structure (one persistent CTA per SM):
//   * warp 8 = producer: one thread streams key tiles global -> shared with
//     TMA (cp.async.bulk.tensor, 128-byte swizzle) through an mbarrier ring;
//   * warps 0..7 = consumers in two groups of four that take alternate tiles.
//     A warp scores 16 rows at a time with mma.sync.m16n8k16: the A operand is
//     the key block read from the swizzled tile with conflict-free LDS.128,
//     the B operand holds the queries split as q = hi + lo/scale (two columns
//     per query), accumulation is fp32.  The k index is permuted identically
//     on both operands so that each thread's 16 contiguous bytes feed the
//     fragments directly (a dot product does not care about term order
//     within the tensor-core accumulate).
//   * selection never leaves the SM: each warp filters its scores against the
//     running n-th best of its own list (WarpTopN) and only survivors are
//     queued; lists are merged across the CTA's warps at the end and written
//     to the workspace as one sorted list per (CTA, query).
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kConsumerWarps = 8;
constexpr int kGroupWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kStageBytes = 32 * 1024;
constexpr int kSlabBytes = 128;            // one swizzle row: 64 16-bit elements
constexpr int kSlabElems = 64;
constexpr int kMaxStages = 6;

template <typename T> struct Mma;
template <> struct Mma<__half> {
    __device__ static __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
    {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
            "{%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};
template <> struct Mma<__nv_bfloat16> {
    __device__ static __forceinline__ void run(float (&c)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
    {
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
            "{%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
};

// KS = 64-element slabs per key row when the whole row fits one stage (1, 2, 4:
// d <= 64, 128, 256; query fragments then live in registers), or 0 for the
// generic kernel that walks long rows in chunks of 4 slabs with the query
// operand in shared memory.  NG = groups of 4 queries per launch (1 or 2).
template <int KS> struct Shape {
    static constexpr int kSlabsPerStage = KS > 0 ? KS : 4;
    static constexpr int kRows = kStageBytes / (kSlabsPerStage * kSlabBytes);  // 256,128,64 / 64
    static constexpr int kBlocksPerWarp = kRows / 16 / kGroupWarps;
};

struct Smem {
    uint8_t *stages;     // [stages][kStageBytes], 1024-aligned
    WarpTopN *sel;       // [kConsumerWarps][NQ]
    uint64_t *full;      // [stages]
    uint64_t *empty;     // [stages]
    uint8_t *qs;         // generic kernel: [8*NG][dpad*2+16] bytes
};

template <int NG>
__host__ __device__ inline size_t sel_bytes()
{
    return sizeof(WarpTopN) * kConsumerWarps * 4 * NG;
}

template <typename T, int KS, int NG>
__global__ void __launch_bounds__(kThreads, 1)
scan_mma_kernel(const __grid_constant__ CUtensorMap keys_map, const ScanArgs a)
{
    using S = Shape<KS>;
    constexpr int NQ = 4 * NG;
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    uint8_t *stages = base;
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(stages + (size_t)n_stages * kStageBytes);
    uint64_t *full = reinterpret_cast<uint64_t *>(reinterpret_cast<uint8_t *>(sel) + sel_bytes<NG>());
    uint64_t *empty = full + kMaxStages;
    uint8_t *qs = reinterpret_cast<uint8_t *>(empty + kMaxStages);   // generic only
    const int qs_stride = a.dpad * 2 + 16;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kGroupWarps);
        }
        mbar_fence_init();
    }
    if (warp < kConsumerWarps)
        for (int q = 0; q < NQ; ++q) warp_topn_init(&sel[warp * NQ + q], lane);
    if (KS == 0) {
        // query operand rows -> shared memory (row stride padded by 16 bytes so
        // that the fragment reads of a quarter-warp fall in distinct banks)
        const uint4 *src = static_cast<const uint4 *>(a.qsplit);
        const int vec_per_row = a.dpad / 8;
        for (int i = tid; i < 8 * NG * vec_per_row; i += kThreads) {
            int r = i / vec_per_row, c = i % vec_per_row;
            *reinterpret_cast<uint4 *>(qs + (size_t)r * qs_stride + c * 16) = src[(size_t)r * vec_per_row + c];
        }
    }
    __syncthreads();

    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const int kch = KS > 0 ? 1 : (dslabs + 3) / 4;                 // k-chunks per tile
    const int my_tiles = cta < a.n_tiles ? (a.n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * kch;
    bool dead = false;
    const long long wait_limit = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;

    if (warp == kConsumerWarps) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&keys_map);
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wait_limit)) {
                    report_timeout(a.status);
                    break;
                }
                const int tile = cta + (it / kch) * G;
                const int kc = it % kch;
                const int nsl = KS > 0 ? KS : min(4, dslabs - kc * 4);
                mbar_arrive_expect_tx(&full[s], (uint32_t)(nsl * S::kRows * kSlabBytes));
                uint8_t *dst = stages + (size_t)s * kStageBytes;
                if (!debug_check(s >= 0 && s < n_stages && tile >= 0 && (long long)tile * S::kRows < a.N + S::kRows, a.status, 31)) break;
                // Test hook: one CTA "loses" the copies of one stage, so that the waits on it
                // run out and the timeout path (status word, orderly exit) can be exercised.
                const bool lose = a.debug_lose_stage > 0 && cta == 0 && it == a.debug_lose_stage - 1;
                for (int sl = 0; sl < nsl && !lose; ++sl)
                    tma_load_2d(dst + (size_t)sl * S::kRows * kSlabBytes, &keys_map,
                                (kc * 4 + sl) * kSlabElems, tile * S::kRows, &full[s]);
                issued = it + 1;
            }
            // Do not leave while copies into this CTA's shared memory are in flight.
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1, wait_limit)) {
                    report_timeout(a.status);
                    break;
                }
        }
    } else {
        // ------------------------------ consumers -----------------------------
        const int group = warp / kGroupWarps, wg = warp % kGroupWarps;
        const int g = lane >> 2, t = lane & 3;
        WarpTopN *my_sel = &sel[warp * NQ];

        uint32_t bq[NG][KS > 0 ? KS : 1][8];
        if (KS > 0) {
#pragma unroll
            for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                for (int s = 0; s < (KS > 0 ? KS : 1); ++s) {
                    const uint4 *p = reinterpret_cast<const uint4 *>(
                        static_cast<const T *>(a.qsplit) + (size_t)(grp * 8 + g) * a.dpad + s * 64 + 16 * t);
                    uint4 v0 = p[0], v1 = p[1];
                    bq[grp][s][0] = v0.x; bq[grp][s][1] = v0.y; bq[grp][s][2] = v0.z; bq[grp][s][3] = v0.w;
                    bq[grp][s][4] = v1.x; bq[grp][s][5] = v1.y; bq[grp][s][6] = v1.z; bq[grp][s][7] = v1.w;
                }
        }
        bool q_valid[NG];
        int want[NG];                                  // first-token filter of this thread's queries, -1 = off
#pragma unroll
        for (int grp = 0; grp < NG; ++grp) {
            q_valid[grp] = grp * 4 + t < a.B;
            want[grp] = (a.first_col && q_valid[grp]) ? a.want_first[grp * 4 + t] : -1;
        }

        const uint32_t swz = (uint32_t)g;          // (row & 7) of both of this thread's rows
        const uint32_t off0 = (uint32_t)(((2 * t) ^ swz) << 4);
        const uint32_t off1 = (uint32_t)(((2 * t + 1) ^ swz) << 4);

        for (int tl = group; tl < my_tiles && !dead; tl += 2) {
            const long long tile_row0 = (long long)(cta + tl * G) * S::kRows;
            // first stored tokens of this thread's rows, requested before the tile is waited for
            int tok_a[S::kBlocksPerWarp], tok_b[S::kBlocksPerWarp];
#pragma unroll
            for (int bi = 0; bi < S::kBlocksPerWarp; ++bi) {
                const long long ra = tile_row0 + (wg * S::kBlocksPerWarp + bi) * 16 + g;
                tok_a[bi] = (a.first_col && ra < a.N) ? a.first_col[ra] : 0;
                tok_b[bi] = (a.first_col && ra + 8 < a.N) ? a.first_col[ra + 8] : 0;
            }
            float acc[S::kBlocksPerWarp][NG][2][4];
#pragma unroll
            for (int bi = 0; bi < S::kBlocksPerWarp; ++bi)
#pragma unroll
                for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                    for (int ch = 0; ch < 2; ++ch)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[bi][grp][ch][i] = 0.f;

            for (int kc = 0; kc < kch; ++kc) {
                const int it = tl * kch + kc;
                const int s = it % n_stages;
                if (!mbar_wait(&full[s], (it / n_stages) & 1, wait_limit)) {
                    report_timeout(a.status);
                    dead = true;
                    break;
                }
                const uint8_t *st = stages + (size_t)s * kStageBytes;
                const int nsl = KS > 0 ? KS : min(4, dslabs - kc * 4);
#pragma unroll
                for (int bi = 0; bi < S::kBlocksPerWarp; ++bi) {
                    const int r0 = (wg * S::kBlocksPerWarp + bi) * 16;
                    const uint8_t *rowa = st + (size_t)(r0 + g) * kSlabBytes;
                    const uint8_t *rowb = rowa + 8 * kSlabBytes;
#pragma unroll
                    for (int sl = 0; sl < S::kSlabsPerStage; ++sl) {
                        if (KS == 0 && sl >= nsl) break;
                        const size_t so = (size_t)sl * S::kRows * kSlabBytes;
                        const uint4 x0 = *reinterpret_cast<const uint4 *>(rowa + so + off0);
                        const uint4 x1 = *reinterpret_cast<const uint4 *>(rowa + so + off1);
                        const uint4 y0 = *reinterpret_cast<const uint4 *>(rowb + so + off0);
                        const uint4 y1 = *reinterpret_cast<const uint4 *>(rowb + so + off1);
#pragma unroll
                        for (int grp = 0; grp < NG; ++grp) {
                            uint32_t b[8];
                            if (KS > 0) {
#pragma unroll
                                for (int i = 0; i < 8; ++i) b[i] = bq[grp][KS > 0 ? sl : 0][i];
                            } else {
                                const uint8_t *qp = qs + (size_t)(grp * 8 + g) * qs_stride +
                                                    ((size_t)(kc * 4 + sl) * 64 + 16 * t) * 2;
                                const uint4 v0 = *reinterpret_cast<const uint4 *>(qp);
                                const uint4 v1 = *reinterpret_cast<const uint4 *>(qp + 16);
                                b[0] = v0.x; b[1] = v0.y; b[2] = v0.z; b[3] = v0.w;
                                b[4] = v1.x; b[5] = v1.y; b[6] = v1.z; b[7] = v1.w;
                            }
                            Mma<T>::run(acc[bi][grp][0], x0.x, y0.x, x0.y, y0.y, b[0], b[1]);
                            Mma<T>::run(acc[bi][grp][1], x0.z, y0.z, x0.w, y0.w, b[2], b[3]);
                            Mma<T>::run(acc[bi][grp][0], x1.x, y1.x, x1.y, y1.y, b[4], b[5]);
                            Mma<T>::run(acc[bi][grp][1], x1.z, y1.z, x1.w, y1.w, b[6], b[7]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
            }
            if (dead) break;

            // -------- selection: filter against this warp's running n-th best
#pragma unroll
            for (int bi = 0; bi < S::kBlocksPerWarp; ++bi) {
                const long long row_a = tile_row0 + (wg * S::kBlocksPerWarp + bi) * 16 + g;
                const long long row_b = row_a + 8;
                float sa[NG], sb[NG];
                bool pa[NG], pb[NG];
                bool any = false;
#pragma unroll
                for (int grp = 0; grp < NG; ++grp) {
                    const float *c0 = acc[bi][grp][0], *c1 = acc[bi][grp][1];
                    sa[grp] = (c0[0] + c1[0]) + (c0[1] + c1[1]) * a.lo_inv_scale;
                    sb[grp] = (c0[2] + c1[2]) + (c0[3] + c1[3]) * a.lo_inv_scale;
                    const float tau = my_sel[grp * 4 + t].tau;
                    pa[grp] = q_valid[grp] && row_a < a.N && sa[grp] >= tau && (want[grp] < 0 || tok_a[bi] == want[grp]);
                    pb[grp] = q_valid[grp] && row_b < a.N && sb[grp] >= tau && (want[grp] < 0 || tok_b[bi] == want[grp]);
                    any |= pa[grp] | pb[grp];
                }
                if (__any_sync(0xFFFFFFFFu, any)) {
                    // Rare path.  First pull the grid-wide filter (other CTAs may know a
                    // better n-th best), re-test, queue what survives, publish our filter.
                    if (lane < NQ && lane < a.B) my_sel[lane].tau = peek_tau(&a.gtau[lane], my_sel[lane].tau);
                    __syncwarp();
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp) {
                        const float tau = my_sel[grp * 4 + t].tau;
                        pa[grp] = pa[grp] && sa[grp] >= tau;
                        pb[grp] = pb[grp] && sb[grp] >= tau;
                    }
#pragma unroll
                    for (int grp = 0; grp < NG; ++grp)
#pragma unroll
                        for (int tq = 0; tq < 4; ++tq) {
                            WarpTopN *sq = &my_sel[grp * 4 + tq];
                            warp_topn_push(sq, a.top_n, lane, pa[grp] && t == tq, sa[grp], (uint32_t)row_a);
                            warp_topn_push(sq, a.top_n, lane, pb[grp] && t == tq, sb[grp], (uint32_t)row_b);
                        }
                    if (lane < NQ && lane < a.B) my_sel[lane].tau = share_tau(&a.gtau[lane], my_sel[lane].tau);
                    __syncwarp();
                }
            }
        }
        // flush what is still queued
        for (int q = 0; q < NQ; ++q)
            if (my_sel[q].count > 0) warp_topn_merge(&my_sel[q], a.top_n, lane);
    }
    __syncthreads();

    // ---- merge the warps' lists: one warp per query, write the CTA's list ----
    if (warp < kConsumerWarps) {
        for (int q = warp; q < min(NQ, a.B); q += kConsumerWarps) {
            unsigned long long m = sel[q].list[lane];
            for (int w = 1; w < kConsumerWarps; ++w)
                m = warp_merge_top32(m, sel[w * NQ + q].list[lane], lane);
            if (lane >= a.top_n) m = 0ull;
            if (debug_check(q < a.cand_batch && (m == 0ull || (long long)candidate_id(m) < a.N), a.status, 34))
                a.cand[((size_t)cta * a.cand_batch + q) * kCandStride + lane] = m;
        }
    }
}

template <typename T, int KS, int NG>
cudaError_t launch_one(const CUtensorMap &map, const ScanArgs &a, int grid, size_t smem,
                       cudaStream_t stream)
{
    auto kernel = scan_mma_kernel<T, KS, NG>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, kThreads, smem, stream>>>(map, a);
    return cudaGetLastError();
}

int ks_of(int d) { return d <= 64 ? 1 : d <= 128 ? 2 : d <= 256 ? 4 : 0; }

}  // namespace

int scan_mma_tile_rows(int d)
{
    switch (ks_of(d)) {
    case 1: return Shape<1>::kRows;
    case 2: return Shape<2>::kRows;
    case 4: return Shape<4>::kRows;
    default: return Shape<0>::kRows;
    }
}

int scan_mma_queries_per_launch(int d, int B)
{
    if (ks_of(d) == 0) return 4;          // generic kernel: query operand in shared memory
    return B <= 4 ? 4 : 8;
}

size_t scan_mma_smem_bytes(int d, int B, int *stages_out)
{
    const int ng = scan_mma_queries_per_launch(d, B) / 4;
    size_t fixed = 1024 /*alignment slack*/ + sizeof(WarpTopN) * kConsumerWarps * 4 * ng +
                   2 * kMaxStages * sizeof(uint64_t);
    if (ks_of(d) == 0) fixed += (size_t)8 * ng * (((d + 63) / 64) * 64 * 2 + 16);
    int stages = (int)((227 * 1024 - fixed) / kStageBytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages_out) *stages_out = stages;
    return fixed + (size_t)stages * kStageBytes;
}

cudaError_t launch_scan_mma(const CUtensorMap &map, const ScanArgs &a_in, int grid, cudaStream_t stream)
{
    ScanArgs a = a_in;
    int stages = 0;
    const size_t smem = scan_mma_smem_bytes(a.d, a.B, &stages);
    if (stages < 2) return cudaErrorInvalidValue;
    a.stages = stages;
    const int ks = ks_of(a.d);
    const int ng = scan_mma_queries_per_launch(a.d, a.B) / 4;
    const bool h = a.dtype == kF16;
#define DRESD_GO(KS_, NG_)                                                                     \
    return h ? launch_one<__half, KS_, NG_>(map, a, grid, smem, stream)                        \
             : launch_one<__nv_bfloat16, KS_, NG_>(map, a, grid, smem, stream)
    if (ks == 1 && ng == 1) { DRESD_GO(1, 1); }
    if (ks == 1 && ng == 2) { DRESD_GO(1, 2); }
    if (ks == 2 && ng == 1) { DRESD_GO(2, 1); }
    if (ks == 2 && ng == 2) { DRESD_GO(2, 2); }
    if (ks == 4 && ng == 1) { DRESD_GO(4, 1); }
    if (ks == 4 && ng == 2) { DRESD_GO(4, 2); }
    DRESD_GO(0, 1);
#undef DRESD_GO
}

}  // namespace dresd
