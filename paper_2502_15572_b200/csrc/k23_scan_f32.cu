// K2+K3 for fp32 datastores -- Eq. 3 of the paper for every key, s_i = q . k_i,
// in plain fp32 FMA (tensor cores would round fp32 operands to 10-11 mantissa
// bits, far outside the 1e-5 score tolerance), fused with the per-CTA top-n.
//
// Same skeleton as the 16-bit streaming kernel: a producer thread streams
// 128-row key tiles into shared memory with TMA (128-byte swizzle, two
// 32-float slabs per stage) through an mbarrier ring; four consumer warps own
// one row per thread, read it with conflict-free LDS.128 against queries
// broadcast from shared memory, and keep four partial sums per query so that
// the accumulation error stays near d/4 ulps.  Up to QB queries per launch.
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kConsumerWarps = 4;
constexpr int kRows = kConsumerWarps * 32;       // 128 rows per stage, one per thread
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kSlabBytes = 128;                   // 32 floats
constexpr int kSlabElems = 32;
constexpr int kSlabsPerStage = 2;
constexpr int kStageBytes = kRows * kSlabsPerStage * kSlabBytes;   // 32 KB
constexpr int kMaxStages = 6;

template <int QB>
__global__ void __launch_bounds__(kThreads, 1)
scan_f32_kernel(const __grid_constant__ CUtensorMap keys_map, const ScanArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    uint8_t *stages = base;
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(stages + (size_t)n_stages * kStageBytes);
    uint64_t *full = reinterpret_cast<uint64_t *>(sel + kConsumerWarps * QB);
    uint64_t *empty = full + kMaxStages;
    float *qs = reinterpret_cast<float *>(empty + kMaxStages);     // [QB][dpad]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const int dpad = dslabs * kSlabElems;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        mbar_fence_init();
    }
    if (warp < kConsumerWarps)
        for (int q = 0; q < QB; ++q) warp_topn_init(&sel[warp * QB + q], lane);
    for (int i = tid; i < QB * dpad; i += kThreads) {
        int q = i / dpad, c = i % dpad;
        qs[i] = (q < a.B && c < a.d) ? a.qhat[(size_t)q * a.d + c] : 0.f;
    }
    __syncthreads();

    const int kch = (dslabs + kSlabsPerStage - 1) / kSlabsPerStage;
    const int my_tiles = cta < a.n_tiles ? (a.n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * kch;

    if (warp == kConsumerWarps) {
        if (lane == 0) {
            tma_prefetch_desc(&keys_map);
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1)) {
                    report_timeout(a.status);
                    break;
                }
                const int tile = cta + (it / kch) * G;
                const int kc = it % kch;
                const int nsl = min(kSlabsPerStage, dslabs - kc * kSlabsPerStage);
                mbar_arrive_expect_tx(&full[s], (uint32_t)(nsl * kRows * kSlabBytes));
                uint8_t *dst = stages + (size_t)s * kStageBytes;
                for (int sl = 0; sl < nsl; ++sl)
                    tma_load_2d(dst + (size_t)sl * kRows * kSlabBytes, &keys_map,
                                (kc * kSlabsPerStage + sl) * kSlabElems, tile * kRows, &full[s]);
                issued = it + 1;
            }
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1)) {
                    report_timeout(a.status);
                    break;
                }
        }
    } else {
        WarpTopN *my_sel = &sel[warp * QB];
        const int row_in_tile = tid;                  // 0..127
        const uint32_t swz = (uint32_t)(row_in_tile & 7);
        bool dead = false;
        int want[QB];                                  // first-token filter, -1 = off
#pragma unroll
        for (int q = 0; q < QB; ++q) want[q] = (a.first_col && q < a.B) ? a.want_first[q] : -1;
        for (int tl = 0; tl < my_tiles && !dead; ++tl) {
            // this row's first stored token, requested before the tile is waited for
            const long long row_pre = (long long)(cta + tl * G) * kRows + row_in_tile;
            const int tok = (a.first_col && row_pre < a.N) ? a.first_col[row_pre] : 0;
            float acc[QB][4];
#pragma unroll
            for (int q = 0; q < QB; ++q)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[q][i] = 0.f;
            for (int kc = 0; kc < kch; ++kc) {
                const int it = tl * kch + kc;
                const int s = it % n_stages;
                if (!mbar_wait(&full[s], (it / n_stages) & 1)) {
                    report_timeout(a.status);
                    dead = true;
                    break;
                }
                const uint8_t *rowp = stages + (size_t)s * kStageBytes + (size_t)row_in_tile * kSlabBytes;
                const int nsl = min(kSlabsPerStage, dslabs - kc * kSlabsPerStage);
                for (int sl = 0; sl < nsl; ++sl) {
                    const float *qbase = qs + (kc * kSlabsPerStage + sl) * kSlabElems;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float4 k4 = *reinterpret_cast<const float4 *>(
                            rowp + (size_t)sl * kRows * kSlabBytes + ((c ^ swz) << 4));
#pragma unroll
                        for (int q = 0; q < QB; ++q) {
                            const float4 q4 = *reinterpret_cast<const float4 *>(qbase + (size_t)q * dpad + c * 4);
                            acc[q][0] = fmaf(q4.x, k4.x, acc[q][0]);
                            acc[q][1] = fmaf(q4.y, k4.y, acc[q][1]);
                            acc[q][2] = fmaf(q4.z, k4.z, acc[q][2]);
                            acc[q][3] = fmaf(q4.w, k4.w, acc[q][3]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
            }
            if (dead) break;

            const long long row = (long long)(cta + tl * G) * kRows + row_in_tile;
            float sc[QB];
            bool take[QB];
            bool any = false;
#pragma unroll
            for (int q = 0; q < QB; ++q) {
                sc[q] = (acc[q][0] + acc[q][1]) + (acc[q][2] + acc[q][3]);
                take[q] = q < a.B && row < a.N && sc[q] >= my_sel[q].tau && (want[q] < 0 || tok == want[q]);
                any |= take[q];
            }
            if (__any_sync(0xFFFFFFFFu, any)) {
                // Rare path: pull the grid-wide filter, re-test, queue, publish ours.
                if (lane < QB && lane < a.B) my_sel[lane].tau = peek_tau(&a.gtau[lane], my_sel[lane].tau);
                __syncwarp();
#pragma unroll
                for (int q = 0; q < QB; ++q)
                    warp_topn_push(&my_sel[q], a.top_n, lane, take[q] && sc[q] >= my_sel[q].tau, sc[q], (uint32_t)row);
                if (lane < QB && lane < a.B) my_sel[lane].tau = share_tau(&a.gtau[lane], my_sel[lane].tau);
                __syncwarp();
            }
        }
        for (int q = 0; q < QB; ++q)
            if (my_sel[q].count > 0) warp_topn_merge(&my_sel[q], a.top_n, lane);
    }
    __syncthreads();

    if (warp < kConsumerWarps) {
        for (int q = warp; q < min(QB, a.B); q += kConsumerWarps) {
            unsigned long long m = sel[q].list[lane];
            for (int w = 1; w < kConsumerWarps; ++w)
                m = warp_merge_top32(m, sel[w * QB + q].list[lane], lane);
            if (lane >= a.top_n) m = 0ull;
            a.cand[((size_t)cta * a.cand_batch + q) * kCandStride + lane] = m;
        }
    }
}

template <int QB>
size_t smem_bytes(int d, int *stages_out)
{
    const int dpad = ((d + kSlabElems - 1) / kSlabElems) * kSlabElems;
    size_t fixed = 1024 + sizeof(WarpTopN) * kConsumerWarps * QB + 2 * kMaxStages * sizeof(uint64_t) +
                   sizeof(float) * (size_t)QB * dpad;
    int stages = (int)((227 * 1024 - (long long)fixed) / kStageBytes);
    if (stages > kMaxStages) stages = kMaxStages;
    *stages_out = stages;
    return fixed + (size_t)(stages > 0 ? stages : 0) * kStageBytes;
}

template <int QB>
cudaError_t launch_one(const CUtensorMap &map, ScanArgs a, int grid, cudaStream_t stream)
{
    int stages = 0;
    const size_t smem = smem_bytes<QB>(a.d, &stages);
    if (stages < 2) return cudaErrorInvalidValue;
    a.stages = stages;
    auto kernel = scan_f32_kernel<QB>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kernel<<<grid, kThreads, smem, stream>>>(map, a);
    return cudaGetLastError();
}

}  // namespace

int scan_f32_tile_rows(int) { return kRows; }
int scan_f32_queries_per_launch(int d, int) { return d <= 1024 ? 8 : 4; }

cudaError_t launch_scan_f32(const CUtensorMap &map, const ScanArgs &a, int grid, cudaStream_t stream)
{
    return scan_f32_queries_per_launch(a.d, a.B) == 8 ? launch_one<8>(map, a, grid, stream)
                                                       : launch_one<4>(map, a, grid, stream);
}

}  // namespace dresd
