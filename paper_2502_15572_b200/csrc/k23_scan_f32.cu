// K2+K3 for fp32 datastores -- Eq. 3 of the paper for every key, s_i = q . k_i,
// in plain fp32 FMA (tensor cores would round fp32 operands to 10-11 mantissa
// bits, far outside the 1e-5 score tolerance), fused with the per-CTA top-n.
//
// Same skeleton as the 16-bit streaming kernel: a producer thread streams key
// tiles into shared memory with TMA (128-byte swizzle, one 32-float slab of 512
// rows per stage) through an mbarrier ring; four consumer warps score them.
// The loop is register-tiled: a thread owns FOUR rows of the tile and all QB
// queries of the launch, so that per four elements of k it issues 4 LDS.128 of
// its rows and QB broadcast LDS.128 of the queries for 16 QB FMAs.  With one row
// per thread (the first form) the loop was bound by shared-memory instruction
// issue, 5 LDS.128 per 16 FMAs: 2.5 TB/s on a large store at any batch.  Four
// partial sums per (row, query), advanced in pairs by packed FMAs (fma.rn.f32x2),
// keep the accumulation error near d/4 ulps.
// QB is the batch rounded up to 1, 2, 4 or 8: a single query pays for one.  Eight
// queries are split over two groups of four warps (the same rows, four queries each):
// 128 accumulators per thread would leave no registers for the loads in flight.
//
// The running top-n lists are shared by the CTA (one per query): survivors of
// the filter are queued with a shared-memory atomic, a named barrier per tile
// publishes them, and a queue that reaches 16 entries is folded by one warp
// (the warps fold different queries at once).  The cold start is bounded by
// taking the n-th largest of 32 group maxima of the first tile as the first
// filter score (n rows reach it, so the final n-th best does too).
#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kGroupWarps = 4;
constexpr int kRowsPerThread = 4;
constexpr int kLanes = kGroupWarps * 32;                     // 128 threads share the rows of a tile
constexpr int kRows = kLanes * kRowsPerThread;               // 512 rows per tile
constexpr int kBoxRows = 256;                                // a TMA box is at most 256 rows tall
constexpr int groups_of(int QB) { return QB > 4 ? 2 : 1; }   // query groups (each: kGroupWarps warps)
constexpr int kSlabBytes = 128;                              // 32 floats
constexpr int kSlabElems = 32;
constexpr int kStageBytes = kRows * kSlabBytes;              // one slab of the tile: 64 KB
constexpr int kMaxStages = 3;

struct SelFlags {
    int need_merge;
    int overflow;
};
template <int NTHREADS> __device__ __forceinline__ void consumer_bar()
{
    asm volatile("bar.sync 2, %0;" ::"n"(NTHREADS) : "memory");
}

template <int QB>
__global__ void __launch_bounds__((groups_of(QB) * kGroupWarps + 1) * 32, 1)
scan_f32_kernel(const __grid_constant__ CUtensorMap keys_map, const ScanArgs a)
{
    constexpr int kConsumerWarps = groups_of(QB) * kGroupWarps;
    constexpr int kThreads = (kConsumerWarps + 1) * 32;
    constexpr int QT = QB / groups_of(QB);                   // queries per thread
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int n_stages = a.stages;
    uint8_t *stages = base;
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(stages + (size_t)n_stages * kStageBytes);   // [QB], CTA-wide
    uint64_t *full = reinterpret_cast<uint64_t *>(sel + QB);
    uint64_t *empty = full + kMaxStages;
    SelFlags *flags = reinterpret_cast<SelFlags *>(empty + kMaxStages);   // [3], rotating
    float *qs = reinterpret_cast<float *>(                         // [QB][dpad], read as float4
        (reinterpret_cast<uintptr_t>(flags + 4) + 15) & ~static_cast<uintptr_t>(15));

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const int dpad = dslabs * kSlabElems;

    if (tid == 0) {
        tma_prefetch_desc(&keys_map);
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

    const int my_tiles = cta < a.n_tiles ? (a.n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * dslabs;                // one slab of one tile per stage
    const long long wl = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;   // bound of every wait below

    if (warp == kConsumerWarps) {
        if (lane == 0) {
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
                const int tile = cta + (it / dslabs) * G;
                const int sl = it % dslabs;
                mbar_arrive_expect_tx(&full[s], (uint32_t)kStageBytes);     // rows past N arrive as zeros
                uint8_t *dst = stages + (size_t)s * kStageBytes;
                if (!debug_check(s >= 0 && s < n_stages && tile >= 0 && (long long)tile * kRows < a.N + kRows, a.status, 21)) break;
                // Test hook: CTA 0 "loses" the copies of one stage, so that the waits on it run out.
                const bool lose = a.debug_lose_stage > 0 && cta == 0 && it == a.debug_lose_stage - 1;
                for (int h = 0; h < kRows / kBoxRows && !lose; ++h)
                    tma_load_2d(dst + (size_t)h * kBoxRows * kSlabBytes, &keys_map, sl * kSlabElems,
                                tile * kRows + h * kBoxRows, &full[s]);
                issued = it + 1;
            }
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
        }
    } else {
        constexpr int R = kRowsPerThread;
        // this thread's rows of a tile: rt, rt + 128, rt + 256, rt + 384 (the same swizzle phase);
        // its queries: q0 .. q0 + QT - 1
        const int rt = tid & (kLanes - 1), q0 = (tid / kLanes) * QT;
        const uint32_t swz = (uint32_t)(rt & 7);
        // A warp whose wait expired goes "dead": it does no more work and no more waits,
        // but keeps taking part in every barrier so that nobody is left behind.
        bool dead = false;
        int round = 0;                                 // barrier-A count: selects the flag slot
        SelFlags *fl = &flags[0];
        int want[QT];                                  // first-token filter, -1 = off
#pragma unroll
        for (int j = 0; j < QT; ++j) want[j] = (a.first_col && q0 + j < a.B) ? a.want_first[q0 + j] : -1;
        for (int tl = 0; tl < my_tiles; ++tl) {
            const long long row0 = (long long)(cta + tl * G) * kRows + rt;
            // the rows' first stored tokens, requested before the tile is waited for
            int tok[R];
#pragma unroll
            for (int ri = 0; ri < R; ++ri) {
                const long long row = row0 + ri * kLanes;
                tok[ri] = (a.first_col && row < a.N) ? a.first_col[row] : 0;
            }
            // four partial sums per (row, query), held as two pairs: one packed FMA (two IEEE fp32
            // FMAs in one instruction) advances a pair
            float2 acc[R][QT][2];
#pragma unroll
            for (int ri = 0; ri < R; ++ri)
#pragma unroll
                for (int q = 0; q < QT; ++q)
#pragma unroll
                    for (int i = 0; i < 2; ++i) acc[ri][q][i] = make_float2(0.f, 0.f);
            for (int sl = 0; sl < dslabs; ++sl) {
                const int it = tl * dslabs + sl;
                const int s = it % n_stages;
                if (!dead && !mbar_wait(&full[s], (it / n_stages) & 1, wl)) {
                    report_timeout(a.status);
                    dead = true;
                }
                dead = __any_sync(0xFFFFFFFFu, dead);
                if (dead) continue;
                const uint8_t *rowp = stages + (size_t)s * kStageBytes + (size_t)rt * kSlabBytes;
                const float *qbase = qs + (size_t)q0 * dpad + sl * kSlabElems;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    float4 k4[R];
#pragma unroll
                    for (int ri = 0; ri < R; ++ri)
                        k4[ri] = *reinterpret_cast<const float4 *>(rowp + (size_t)ri * kLanes * kSlabBytes + ((c ^ swz) << 4));
#pragma unroll
                    for (int q = 0; q < QT; ++q) {
                        const float4 q4 = *reinterpret_cast<const float4 *>(qbase + (size_t)q * dpad + c * 4);
#pragma unroll
                        for (int ri = 0; ri < R; ++ri) {
                            acc[ri][q][0] = __ffma2_rn(make_float2(q4.x, q4.y), make_float2(k4[ri].x, k4[ri].y), acc[ri][q][0]);
                            acc[ri][q][1] = __ffma2_rn(make_float2(q4.z, q4.w), make_float2(k4[ri].z, k4[ri].w), acc[ri][q][1]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);
            }
            // every fourth tile, pull the grid-wide filter (other CTAs may know a better n-th best)
            if ((tl & 3) == 0 && tid < a.B && tid < QB) sel[tid].tau = peek_tau(&a.gtau[tid], sel[tid].tau);

            float sc[R][QT];
            uint32_t okbits = 0u;                      // bit ri * QT + j: the row may be a result of query q0 + j
#pragma unroll
            for (int ri = 0; ri < R; ++ri)
#pragma unroll
                for (int q = 0; q < QT; ++q) {
                    sc[ri][q] = (acc[ri][q][0].x + acc[ri][q][0].y) + (acc[ri][q][1].x + acc[ri][q][1].y);
                    const bool ok = !dead && q0 + q < a.B && row0 + ri * kLanes < a.N && sc[ri][q] > -INFINITY &&   // false for NaN
                                    (want[q] < 0 || tok[ri] == want[q]);
                    okbits |= ok ? (1u << (ri * QT + q)) : 0u;
                }
            if (tl == 0) {
                // Cold start: 32 groups of 16 rows per query (a thread's four rows and those of its three
                // neighbours); the n-th largest group maximum is reached by n rows of this tile and becomes
                // the first filter score, so that about n rows are queued instead of all 512.
#pragma unroll
                for (int q = 0; q < QT; ++q) {
                    uint32_t key = 0u;
#pragma unroll
                    for (int ri = 0; ri < R; ++ri)
                        if ((okbits >> (ri * QT + q)) & 1u) key = max(key, float_to_ordered(sc[ri][q] + 0.0f));
                    key = __reduce_max_sync(0xFu << (lane & ~3), key);
                    // the queue is still empty: its first 128 bytes take the group maxima
                    if ((lane & 3) == 0)
                        reinterpret_cast<uint32_t *>(sel[q0 + q].queue)[(warp & (kGroupWarps - 1)) * 8 + (lane >> 2)] = key;
                }
                consumer_bar<kConsumerWarps * 32>();
                for (int q = warp; q < QB; q += kConsumerWarps) {
                    if (q >= a.B || sel[q].tau > -INFINITY) continue;                              // warp-uniform
                    unsigned long long x = reinterpret_cast<const uint32_t *>(sel[q].queue)[lane];
                    __syncwarp();
                    x = warp_sort_desc(x, lane);
                    const uint32_t nth = (uint32_t)shfl_u64(x, a.top_n - 1);
                    if (lane == 0 && nth) sel[q].tau = share_tau(&a.gtau[q], ordered_to_float(nth));
                }
                consumer_bar<kConsumerWarps * 32>();
            }
            uint32_t pend = 0u;                        // (row, query) pairs that are (still) candidates
#pragma unroll
            for (int ri = 0; ri < R; ++ri)
#pragma unroll
                for (int q = 0; q < QT; ++q)
                    if (((okbits >> (ri * QT + q)) & 1u) && sc[ri][q] >= sel[q0 + q].tau) pend |= 1u << (ri * QT + q);
            // Queue the survivors; when a queue is full the candidate waits (`pend`) until the CTA
            // has folded the queues, so that adversarial row orders stay exact.
            while (true) {
                uint32_t todo = pend;
                while (todo) {                          // rare once the filter is warm
                    const int b = __ffs(todo) - 1;
                    todo &= todo - 1;
                    const int ri = b / QT, q = q0 + b % QT;
                    float s = 0.f;                      // the pair's score without dynamic register indexing
#pragma unroll
                    for (int i = 0; i < R; ++i)
#pragma unroll
                        for (int j = 0; j < QT; ++j)
                            if (i * QT + j == b) s = sc[i][j];
                    if (!(s >= sel[q].tau)) {           // the filter has tightened
                        pend &= ~(1u << b);
                        continue;
                    }
                    const int slot = atomicAdd(&sel[q].count, 1);
                    if (slot < kQueueCap) {
                        sel[q].queue[slot] = pack_candidate(s, (uint32_t)(row0 + ri * kLanes));
                        if (slot + 1 >= kMergeLevel) fl->need_merge = 1;
                        pend &= ~(1u << b);
                    } else {
                        fl->overflow = 1;
                    }
                }
                consumer_bar<kConsumerWarps * 32>();                         // A: every push of this pass is visible
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
                consumer_bar<kConsumerWarps * 32>();                         // C: lists, counts and tau are settled
                if (!over) break;
            }
        }
        // flush and publish this CTA's lists
        consumer_bar<kConsumerWarps * 32>();
        for (int q = warp; q < min(QB, a.B); q += kConsumerWarps) {
            if (sel[q].count > 0) warp_topn_merge(&sel[q], a.top_n, lane);
            unsigned long long m = sel[q].list[lane];
            if (lane >= a.top_n) m = 0ull;
            if (debug_check(q < a.cand_batch && (m == 0ull || (long long)candidate_id(m) < a.N), a.status, 24))
                a.cand[((size_t)cta * a.cand_batch + q) * kCandStride + lane] = m;
        }
    }
}

template <int QB>
size_t smem_bytes(int d, int *stages_out)
{
    const int dpad = ((d + kSlabElems - 1) / kSlabElems) * kSlabElems;
    size_t fixed = 1024 + sizeof(WarpTopN) * QB + 2 * kMaxStages * sizeof(uint64_t) + 4 * sizeof(SelFlags) + 16 +
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
    kernel<<<grid, (groups_of(QB) * kGroupWarps + 1) * 32, smem, stream>>>(map, a);
    return cudaGetLastError();
}

}  // namespace

int scan_f32_tile_rows(int) { return kRows; }
int scan_f32_box_rows(int) { return kBoxRows; }
// the queries of a launch sit in shared memory beside at least two 64 KB stages
int scan_f32_queries_per_launch(int d, int) { return d <= 1024 ? 8 : 4; }

cudaError_t launch_scan_f32(const CUtensorMap &map, const ScanArgs &a, int grid, cudaStream_t stream)
{
    const int cap = scan_f32_queries_per_launch(a.d, a.B);
    if (a.B <= 1) return launch_one<1>(map, a, grid, stream);
    if (a.B <= 2) return launch_one<2>(map, a, grid, stream);
    if (a.B <= 4 || cap == 4) return launch_one<4>(map, a, grid, stream);
    return launch_one<8>(map, a, grid, stream);
}

}  // namespace dresd
