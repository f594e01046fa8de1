// K2+K3 for fp32 datastores -- Eq. 3 of the paper for every key, s_i = q . k_i,
// in plain fp32 FMA (tensor cores would round fp32 operands to 10-11 mantissa
// bits, far outside the 1e-5 score tolerance), fused with the per-CTA top-n.
//
// Same skeleton as the 16-bit streaming kernel: a producer thread streams
// 128-row key tiles into shared memory with TMA (128-byte swizzle, two
// 32-float slabs per stage) through an mbarrier ring; eight consumer warps in
// two groups: a thread owns one row of the tile and half of the launch's
// queries (two warps per scheduler hide the latency of the shared-memory reads
// that one warp alone left exposed), reads the row with conflict-free LDS.128
// against queries broadcast from shared memory, and keeps four partial sums per
// query so that the accumulation error stays near d/4 ulps.  Up to QB queries per launch.
// The running top-n lists are shared by the CTA (one per query): survivors of
// the filter are queued with a shared-memory atomic, a named barrier per tile
// publishes them, and a queue that reaches 16 entries is folded by one warp
// (the warps fold different queries at once).  Per-warp lists would cost a small
// store four cold starts per query instead of one; the one cold start left is
// bounded by taking the n-th largest of 32 group maxima of the first tile as the
// first filter score (n rows reach it, so the final n-th best does too).
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kQueryGroups = 2;                   // warp groups; each takes QB / 2 of the queries
constexpr int kRows = 128;                        // rows per stage, one per thread of a group
constexpr int kConsumerWarps = kQueryGroups * kRows / 32;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kSlabBytes = 128;                   // 32 floats
constexpr int kSlabElems = 32;
constexpr int kSlabsPerStage = 2;
constexpr int kStageBytes = kRows * kSlabsPerStage * kSlabBytes;   // 32 KB
constexpr int kMaxStages = 6;

struct SelFlags {
    int need_merge;
    int overflow;
};
__device__ __forceinline__ void consumer_bar()
{
    asm volatile("bar.sync 2, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

template <int QB>
__global__ void __launch_bounds__(kThreads, 1)
scan_f32_kernel(const __grid_constant__ CUtensorMap keys_map, const ScanArgs a)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    uint8_t *stages = base;
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(stages + (size_t)n_stages * kStageBytes);   // [QB], CTA-wide
    uint64_t *full = reinterpret_cast<uint64_t *>(sel + QB);
    uint64_t *empty = full + kMaxStages;
    SelFlags *flags = reinterpret_cast<SelFlags *>(empty + kMaxStages);   // [3], rotating
    float *qs = reinterpret_cast<float *>(flags + 4);              // [QB][dpad]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const int dpad = dslabs * kSlabElems;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kConsumerWarps);
        }
        for (int i = 0; i < 3; ++i) {
            flags[i].need_merge = 0;
            flags[i].overflow = 0;
        }
        mbar_fence_init();
    }
    if (warp < kConsumerWarps)
        for (int q = warp; q < QB; q += kConsumerWarps) {
            warp_topn_init(&sel[q], lane);
            if (lane == 0 && q < a.B) sel[q].tau = peek_tau(&a.gtau[q], -INFINITY);
        }
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
        constexpr int QT = QB / kQueryGroups;         // queries per thread
        const int row_in_tile = tid & (kRows - 1);    // 0..127
        const int q0 = (tid / kRows) * QT;            // this thread's first query
        const uint32_t swz = (uint32_t)(row_in_tile & 7);
        // A warp whose wait expired goes "dead": it does no more work and no more waits,
        // but keeps taking part in every barrier so that nobody is left behind.
        bool dead = false;
        int round = 0;                                 // barrier-A count: selects the flag slot
        SelFlags *fl = &flags[0];
        int want[QT];                                  // first-token filter, -1 = off
#pragma unroll
        for (int j = 0; j < QT; ++j) want[j] = (a.first_col && q0 + j < a.B) ? a.want_first[q0 + j] : -1;
        for (int tl = 0; tl < my_tiles; ++tl) {
            // this row's first stored token, requested before the tile is waited for
            const long long row = (long long)(cta + tl * G) * kRows + row_in_tile;
            const int tok = (a.first_col && row < a.N) ? a.first_col[row] : 0;
            float acc[QT][4];
#pragma unroll
            for (int j = 0; j < QT; ++j)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[j][i] = 0.f;
            for (int kc = 0; kc < kch; ++kc) {
                const int it = tl * kch + kc;
                const int s = it % n_stages;
                if (!dead && !mbar_wait(&full[s], (it / n_stages) & 1)) {
                    report_timeout(a.status);
                    dead = true;
                }
                dead = __any_sync(0xFFFFFFFFu, dead);
                if (dead) continue;
                const uint8_t *rowp = stages + (size_t)s * kStageBytes + (size_t)row_in_tile * kSlabBytes;
                const int nsl = min(kSlabsPerStage, dslabs - kc * kSlabsPerStage);
                for (int sl = 0; sl < nsl; ++sl) {
                    const float *qbase = qs + (size_t)q0 * dpad + (kc * kSlabsPerStage + sl) * kSlabElems;
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const float4 k4 = *reinterpret_cast<const float4 *>(
                            rowp + (size_t)sl * kRows * kSlabBytes + ((c ^ swz) << 4));
#pragma unroll
                        for (int j = 0; j < QT; ++j) {
                            const float4 q4 = *reinterpret_cast<const float4 *>(qbase + (size_t)j * dpad + c * 4);
                            acc[j][0] = fmaf(q4.x, k4.x, acc[j][0]);
                            acc[j][1] = fmaf(q4.y, k4.y, acc[j][1]);
                            acc[j][2] = fmaf(q4.z, k4.z, acc[j][2]);
                            acc[j][3] = fmaf(q4.w, k4.w, acc[j][3]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
            }
            // every fourth tile, pull the grid-wide filter (other CTAs may know a better n-th best)
            if ((tl & 3) == 0 && tid < a.B && tid < QB) sel[tid].tau = peek_tau(&a.gtau[tid], sel[tid].tau);

            float sc[QT];
#pragma unroll
            for (int j = 0; j < QT; ++j) sc[j] = (acc[j][0] + acc[j][1]) + (acc[j][2] + acc[j][3]);
            if (tl == 0) {
                // Cold start: 32 groups of 4 rows per query; the n-th largest group maximum is reached by
                // n rows of this tile and becomes the first filter score, so that about n rows are queued
                // instead of all 128 (four overflow rounds of barriers and merges otherwise).
#pragma unroll
                for (int j = 0; j < QT; ++j) {
                    const int q = q0 + j;
                    const bool valid = !dead && q < a.B && row < a.N && sc[j] > -INFINITY &&      // false for NaN
                                       (want[j] < 0 || tok == want[j]);
                    uint32_t key = valid ? float_to_ordered(sc[j] + 0.0f) : 0u;
                    key = __reduce_max_sync(0xFu << (lane & ~3), key);
                    // the queue is still empty: its first 128 bytes take the group maxima
                    if ((lane & 3) == 0)
                        reinterpret_cast<uint32_t *>(sel[q].queue)[(warp & 3) * 8 + (lane >> 2)] = key;
                }
                consumer_bar();
                for (int q = warp; q < QB; q += kConsumerWarps) {
                    if (q >= a.B || sel[q].tau > -INFINITY) continue;                              // warp-uniform
                    unsigned long long x = reinterpret_cast<const uint32_t *>(sel[q].queue)[lane];
                    __syncwarp();
                    x = warp_sort_desc(x, lane);
                    const uint32_t nth = (uint32_t)shfl_u64(x, a.top_n - 1);
                    if (lane == 0 && nth) sel[q].tau = share_tau(&a.gtau[q], ordered_to_float(nth));
                }
                consumer_bar();
            }
            uint32_t pend = 0u;                        // queries for which this row is (still) a candidate
#pragma unroll
            for (int j = 0; j < QT; ++j) {
                const int q = q0 + j;
                const bool take = !dead && q < a.B && row < a.N && sc[j] >= sel[q].tau && (want[j] < 0 || tok == want[j]);
                pend |= take ? (1u << j) : 0u;
            }
            // Queue the survivors; when a queue is full the candidate waits (`pend`) until the CTA
            // has folded the queues, so that adversarial row orders stay exact.
            while (true) {
                // claim the slots first (independent shared-memory atomics in flight together), then fill them
                int slot[QT];
#pragma unroll
                for (int j = 0; j < QT; ++j) {
                    const int q = q0 + j;
                    if (((pend >> j) & 1u) && !(sc[j] >= sel[q].tau)) pend &= ~(1u << j);   // the filter has tightened
                    slot[j] = ((pend >> j) & 1u) ? atomicAdd(&sel[q].count, 1) : 0;
                }
#pragma unroll
                for (int j = 0; j < QT; ++j) {
                    const int q = q0 + j;
                    if ((pend >> j) & 1u) {
                        if (slot[j] < kQueueCap) {
                            sel[q].queue[slot[j]] = pack_candidate(sc[j], (uint32_t)row);
                            if (slot[j] + 1 >= kMergeLevel) fl->need_merge = 1;
                            pend &= ~(1u << j);
                        } else {
                            fl->overflow = 1;
                        }
                    }
                }
                consumer_bar();                         // A: every push of this pass is visible
                const int need = fl->need_merge, over = fl->overflow;
                // Flags rotate over three slots: the slot of the previous pass was read by everyone
                // before arriving at A and is not written again before the next A.
                if (tid == 0) {
                    SelFlags *prev = &flags[(round + 2) % 3];
                    prev->need_merge = 0;
                    prev->overflow = 0;
                }
                round += 1;
                fl = &flags[round % 3];
                if (!(need | over)) break;
                for (int q = warp; q < QB; q += kConsumerWarps) {
                    if (sel[q].count > 0) {
                        warp_topn_merge(&sel[q], a.top_n, lane);
                        if (lane == 0 && q < a.B) sel[q].tau = share_tau(&a.gtau[q], sel[q].tau);
                    }
                }
                consumer_bar();                         // C: lists, counts and tau are settled
                if (!over) break;
            }
        }
        // flush and publish this CTA's lists
        consumer_bar();
        for (int q = warp; q < min(QB, a.B); q += kConsumerWarps) {
            if (sel[q].count > 0) warp_topn_merge(&sel[q], a.top_n, lane);
            unsigned long long m = sel[q].list[lane];
            if (lane >= a.top_n) m = 0ull;
            a.cand[((size_t)cta * a.cand_batch + q) * kCandStride + lane] = m;
        }
    }
}

template <int QB>
size_t smem_bytes(int d, int *stages_out)
{
    const int dpad = ((d + kSlabElems - 1) / kSlabElems) * kSlabElems;
    size_t fixed = 1024 + sizeof(WarpTopN) * QB + 2 * kMaxStages * sizeof(uint64_t) + 4 * sizeof(SelFlags) +
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
