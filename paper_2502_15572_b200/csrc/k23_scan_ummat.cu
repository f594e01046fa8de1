// K2+K3 for 17-64 queries on 16-bit keys of 129-256 elements -- Eq. 3 of the paper for
// every key, fused with the per-CTA top-n, with the operand roles of the tensor-core
// instruction swapped: the QUERIES are the M = 128 operand (two rows per query: q = hi +
// lo/scale) and the KEYS are the N = 256 operand.
//
// Why: a tcgen05.mma retires in a time that depends little on its width (about 160 cycles at
// N = 128, 215-250 at N = 256).  With the keys as the M = 128 operand and 64 queries as
// N = 128, a 128-key tile of 256 elements costs 16 instructions = 2.6 k cycles, more than
// the 2.3-2.7 k cycles in which HBM delivers the tile: the instruction stream, not the memory
// stream, set the pace.  With 256 keys per instruction the same 16 instructions cover twice
// the keys.
//
// Accumulator layout: TMEM lane = operand row, column = key.  The operand rows come in 16-row
// blocks (rows 0-7 hi, rows 8-15 lo of 8 queries), and the epilogue reads 16-lane x 256-bit
// fragments, in which one thread holds hi . k and lo . k of the same query and key: a score is
// one FMA.  A thread owns one query per block and walks keys; the running n-th best score of
// its queries sits in registers.
//
// One persistent CTA per SM, ten warps: warp 0 = TMA producer (a stage is one 64-element slab
// of a 256-key tile: two 16 KB boxes), warp 1 = TMEM allocation + MMA issue (two accumulator
// buffers of 256 columns), warps 2-9 = epilogue (lane group = 16 queries, two warps per lane
// group split the 256 keys).  Selection state, grid-wide filter, probe mode and first-token
// filter are those of the other tcgen05 kernel.  Every wait is bounded.
#include <type_traits>

#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kEpiWarps = 8;
constexpr int kThreads = (2 + kEpiWarps) * 32;
constexpr int kTileKeys = 256;                             // keys per tile = N of the instruction
constexpr int kOpRows = 128;                               // query operand rows = M
constexpr int kNQ = kOpRows / 2;                           // queries (padded)
constexpr int kSlabBytes = 128;
constexpr int kSlabElems = 64;
constexpr int kBoxBytes = 128 * kSlabBytes;                // one TMA box: 128 rows x 64 elements
constexpr int kStageBytes = 2 * kBoxBytes;                 // 256 keys x 64 elements
constexpr int kQSlabBytes = kOpRows * kSlabBytes;          // 16 KB
constexpr int kMaxStages = 6;
constexpr int kAccCols = kTileKeys;
constexpr int kTmemCols = 2 * kAccCols;

// 16 lanes x 256 bits per repetition: thread t gets, per 8-column group, the columns
// 2 (t & 3) + {0, 1} of lane (t >> 2) in registers 0-1 and of lane 8 + (t >> 2) in registers 2-3.
__device__ __forceinline__ void tmem_ld_frag1(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x1.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_frag8(uint32_t taddr, uint32_t *r)      // 8 groups = 64 columns
{
    asm volatile(
        "tcgen05.ld.sync.aligned.16x256b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}

__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory"); }

struct EpiFlags {
    int need_merge;
    int overflow;
};

// Shared-memory carve-up (dynamic shared memory must start on a 1024-byte boundary).
struct Layout {
    int stages_off, qres_off, sel_off, tau_off, want_off, tok_off, best_off, bar_off, total;
};
__host__ __device__ inline Layout make_layout(int n_stages, int dslabs)
{
    Layout l;
    l.stages_off = 0;
    l.qres_off = n_stages * kStageBytes;
    l.sel_off = l.qres_off + dslabs * kQSlabBytes;
    l.tau_off = l.sel_off + (int)sizeof(WarpTopN) * kNQ;
    l.want_off = l.tau_off + (int)sizeof(float) * kNQ;
    l.tok_off = l.want_off + (int)sizeof(int) * kNQ;
    l.best_off = l.tok_off + (int)sizeof(int) * kTileKeys;
    l.bar_off = l.best_off + (int)sizeof(unsigned long long) * kNQ;
    l.total = l.bar_off + (int)sizeof(uint64_t) * (2 * kMaxStages + 5) + 8 + (int)sizeof(EpiFlags) * 3;
    return l;
}

template <typename T>
__global__ void __launch_bounds__(kThreads, 1)
scan_ummat_kernel(const __grid_constant__ CUtensorMap keys_map, const __grid_constant__ CUtensorMap q_map,
                  const ScanArgs a)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    if (smem_u32(smem) & 1023u) {                          // the swizzled tiles need it; never expected
        if (threadIdx.x == 0) report_timeout(a.status);
        return;
    }
    const int n_stages = a.stages;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const Layout L = make_layout(n_stages, dslabs);
    uint8_t *stages = smem + L.stages_off;
    uint8_t *qres = smem + L.qres_off;                      // resident query operand, [dslabs][128 rows][128 B]
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(smem + L.sel_off);
    float *tau = reinterpret_cast<float *>(smem + L.tau_off);
    int *want_s = reinterpret_cast<int *>(smem + L.want_off);            // first-token filter per query, -1 = off
    int *tok_s = reinterpret_cast<int *>(smem + L.tok_off);              // first stored token of the tile's keys
    unsigned long long *best = reinterpret_cast<unsigned long long *>(smem + L.best_off);   // probe: per query
    uint64_t *full = reinterpret_cast<uint64_t *>(smem + L.bar_off);
    uint64_t *empty = full + kMaxStages;
    uint64_t *tfull = empty + kMaxStages;                   // [2] accumulator ready
    uint64_t *tempty = tfull + 2;                           // [2] accumulator drained
    uint64_t *qbar = tempty + 2;                            // query operand landed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(qbar + 1);
    EpiFlags *flags = reinterpret_cast<EpiFlags *>(tmem_slot + 2);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int my_tiles = cta < a.n_tiles ? (a.n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * dslabs;
    const long long wl = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;   // bound of every wait below

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], 1);
            mbar_init(&tempty[b], kEpiWarps);
        }
        mbar_init(qbar, 1);
        for (int i = 0; i < 3; ++i) {
            flags[i].need_merge = 0;
            flags[i].overflow = 0;
        }
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    // Everything above is independent of the preceding kernel; what follows reads its output.
    pdl_wait();
    pdl_launch_dependents();
    if (warp >= 2) {
        for (int q = warp - 2; q < kNQ; q += kEpiWarps) {
            warp_topn_init(&sel[q], lane);
            // start from whatever the grid already knows; padding queries never pass
            if (lane == 0) {
                tau[q] = (q < a.B && !a.no_select) ? peek_tau(&a.gtau[q], -INFINITY) : INFINITY;
                want_s[q] = (a.first_col && q < a.B) ? a.want_first[q] : -1;
                best[q] = 0ull;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------------------------- producer ----------------------------------
        if (lane == 0) {
            tma_prefetch_desc(&keys_map);
            tma_prefetch_desc(&q_map);
            mbar_arrive_expect_tx(qbar, (uint32_t)(dslabs * kQSlabBytes));
            for (int s = 0; s < dslabs; ++s)
                tma_load_2d(qres + (size_t)s * kQSlabBytes, &q_map, s * kSlabElems, 0, qbar);
            int issued = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
                const int tile = (cta + (it / dslabs) * G) * a.tile_stride;
                const int ks = it % dslabs;
                uint8_t *dst = stages + (size_t)s * kStageBytes;
                if (!debug_check(s >= 0 && s < n_stages && dst + kStageBytes <= qres && tile >= 0 &&
                                     (long long)tile * kTileKeys < a.N + kTileKeys, a.status, 11))
                    break;
                // rows past N read as zeros (a box may start past the end)
                mbar_arrive_expect_tx(&full[s], (uint32_t)kStageBytes);
                // Test hook: CTA 0 "loses" the copies of one stage, so that the waits on it run out.
                if (a.debug_lose_stage > 0 && cta == 0 && it == a.debug_lose_stage - 1) {
                    issued = it + 1;
                    continue;
                }
                tma_load_2d(dst, &keys_map, ks * kSlabElems, tile * kTileKeys, &full[s]);
                tma_load_2d(dst + kBoxBytes, &keys_map, ks * kSlabElems, tile * kTileKeys + 128, &full[s]);
                issued = it + 1;
            }
            // Do not leave while copies into this CTA's shared memory are in flight.
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
            if (!mbar_wait(qbar, 0, wl)) report_timeout(a.status);
        }
    } else if (warp == 1) {
        // ---------------------------------- MMA issuer ----------------------------------
        if (lane == 0) {
            constexpr uint32_t kFmt = std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
            // A = queries (M = 128 operand rows), B = keys (N = 256), both K-major, fp32 accumulate
            constexpr uint32_t idesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((uint32_t)(kTileKeys >> 3) << 17) |
                                       ((uint32_t)(kOpRows >> 4) << 24);
            bool ok = true;
            if (my_tiles > 0) ok = mbar_wait(qbar, 0, wl);
            for (int tl = 0; tl < my_tiles && ok; ++tl) {
                const int acc = tl & 1, use = tl >> 1;
                if (use >= 1 && !mbar_wait(&tempty[acc], (use - 1) & 1, wl)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
                for (int ks = 0; ks < dslabs; ++ks) {
                    const int it = tl * dslabs + ks;
                    const int s = it % n_stages;
                    if (!mbar_wait(&full[s], (it / n_stages) & 1, wl)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_desc(smem_u32(qres + (size_t)ks * kQSlabBytes));
                    const uint64_t b_desc = make_desc(smem_u32(stages + (size_t)s * kStageBytes));
                    // 4 x K=16 inside the 128-byte swizzle row, +32 bytes each; a last slab that the row
                    // fills only in part (zeros beyond d) needs only the steps that hold data
                    const int ksteps = min(4, (a.d - ks * kSlabElems + 15) / 16);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (k < ksteps) umma_f16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (ks | k) != 0);
                    tc_commit(&empty[s]);            // slab reusable once these MMAs have read it
                }
                if (!ok) break;
                tc_commit(&tfull[acc]);              // accumulator complete
            }
            if (!ok) report_timeout(a.status);
        }
    } else {
        // ---------------------------------- epilogue ----------------------------------
        // The query operand is laid out in 16-row blocks (rows 0-7: hi of 8 queries, rows 8-15:
        // their lo), and the accumulators are read as 16-lane x 256-bit fragments: thread t of a
        // warp then holds, for query (t >> 2) of the block, hi AND lo of the key columns
        // 8 g + 2 (t & 3) + {0, 1} of every 8-column group g -- a score is one FMA, no shuffle.
        // Warp w owns TMEM lanes 32 (w & 3)..+31 = two blocks = 16 queries; the two warps of a
        // lane group take 128 keys each, in four units (block, 64 keys) of 16 scores per thread.
        const int ew = warp - 2;                            // 0..7
        const int lane_grp = warp & 3;
        const int half = ew >> 2;
        const int et = ew * 32 + lane;                      // 0..255
        const int qq0 = lane_grp * 16 + (lane >> 2);        // this thread's query in block 0 (block 1: + 8)
        const int col0 = 2 * (lane & 3);                    // its first column in every 8-column group
        const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(half * 128);
        const float inv = a.lo_inv_scale;
        // a round is asked for when a queue of 32 holds this many: 24 measured 1-4 % ahead of 16 (fewer rounds)
        const int mlevel = a.merge_level > 0 ? a.merge_level : 24;
        const bool filtered = a.first_col != nullptr;
        const int want0 = want_s[qq0], want1 = want_s[qq0 + 8];
        // A warp whose wait expired goes "dead": it does no more work and no more
        // waits, but keeps taking part in every barrier so that nobody is left behind.
        bool dead = false;
        int round = 0;                                      // barrier-A count: selects the flag slot
        EpiFlags *fl = &flags[0];

        for (int tl = 0; tl < my_tiles; ++tl) {
            const int acc = tl & 1, use = tl >> 1;
            const long long tile_key0 = (long long)(cta + tl * G) * a.tile_stride * kTileKeys;
            // key of slot i (group g = i >> 1, e = i & 1) of unit u: key0 + 64 (u & 1) + 8 g + e
            const long long key0 = tile_key0 + half * 128 + col0;
            // first stored token of the tile's keys (filtered calls), requested before the wait
            int tk = -1;
            if (filtered && tile_key0 + et < a.N) tk = a.first_col[tile_key0 + et];
            if (!dead && !mbar_wait(&tfull[acc], use & 1, wl)) {
                report_timeout(a.status);
                dead = true;
            }
            dead = __any_sync(0xFFFFFFFFu, dead);
            tc_fence_after();
            // every fourth tile, pull the grid-wide filter (other CTAs may know a better n-th best)
            if ((tl & 3) == 0 && et < a.B && !a.no_select) tau[et] = peek_tau(&a.gtau[et], tau[et]);
            if (filtered) {
                tok_s[et] = tk;                             // readers of the previous tile are past its barrier A
                epi_bar();
            }
            const uint32_t acc_addr = lane_addr + (uint32_t)(acc * kAccCols);
            auto unit_addr = [&](int u) -> uint32_t {       // block u >> 1 (16 lanes further), keys 64 (u & 1)..
                return acc_addr + ((uint32_t)((u >> 1) * 16) << 16) + (uint32_t)(64 * (u & 1));
            };
            // slots of unit u whose key exists and carries the wanted first token
            auto slot_mask = [&](int u) -> uint32_t {
                const long long k0 = key0 + 64 * (u & 1);
                uint32_t m = 0u;
                if (k0 + 64 <= a.N) {
                    m = 0xFFFFu;
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i) m |= (k0 + 8 * (i >> 1) + (i & 1) < a.N) ? (1u << i) : 0u;
                }
                const int want = (u >> 1) ? want1 : want0;
                if (filtered && want >= 0) {
                    const int2 *t2 = reinterpret_cast<const int2 *>(tok_s + half * 128 + 64 * (u & 1) + col0);
                    uint32_t match = 0u;
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const int2 t = t2[4 * g];                    // keys 8g + col0, + 1 of the unit
                        match |= (t.x == want ? 1u : 0u) << (2 * g) | (t.y == want ? 1u : 0u) << (2 * g + 1);
                    }
                    m &= match;
                }
                return m;
            };
            if (a.probe_max) {
                // Probe pass: no filtering and no lists -- only the best key of the tile per query.
                // The n-th largest of all tiles' bests is a valid filter: at least n keys reach it.
                for (int blk = 0; blk < 2; ++blk) {
                    unsigned long long bv = 0ull;
                    if (!dead) {
                        for (int u = 2 * blk; u < 2 * blk + 2; ++u) {
                            uint32_t r[32];
                            tmem_ld_frag8(unit_addr(u), r);
                            tmem_ld_wait();
                            const uint32_t okm = slot_mask(u);
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const int g = i >> 1, e = i & 1;
                                const float s = fmaf(__uint_as_float(r[4 * g + 2 + e]), inv, __uint_as_float(r[4 * g + e]));
                                if (((okm >> i) & 1u) && s > -INFINITY)              // false for NaN
                                    bv = umax64(bv, pack_candidate(s, (uint32_t)(key0 + 64 * (u & 1) + 8 * g + e)));
                            }
                        }
                    }
                    bv = umax64(bv, shfl_xor_u64(bv, 1));
                    bv = umax64(bv, shfl_xor_u64(bv, 2));
                    if ((lane & 3) == 0 && bv) atomicMax(&best[qq0 + 8 * blk], bv);
                }
                epi_bar();                                   // both halves have contributed
                if (et < a.B) {
                    const unsigned long long v = best[et];
                    best[et] = 0ull;
                    if (v && sel[et].count < kQueueCap) sel[et].queue[sel[et].count++] = v;
                }
                epi_bar();                                   // `best` may be written for the next tile
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[acc]);
                continue;
            }
            // Main pass.  A warp walks its four units; a candidate that finds its query's queue
            // full is remembered (`pend`), the warp stops at that unit, and after the CTA has
            // merged the queues it resumes there -- so adversarial key orders stay exact.
            int next_unit = 0;
            uint32_t pend = 0u;
            bool resume = false;
            // scores of one unit against the filter, survivors queued; true = stop here (queue full)
            auto process = [&](int u, const uint32_t (&r)[32], float tau_r) -> bool {
                const int q = qq0 + 8 * (u >> 1);
                if (!resume && !a.no_fast_reject) {
                    // Fast rejection: hi + lo/S for two keys at a time (packed fp32, the same rounding as the
                    // exact step below), plus -tau; the sign bit of that sum is clear exactly when the score
                    // reaches the filter (a sum of two floats is never rounded across zero).  The sign bits
                    // are ANDed; a warp in which no key of the unit reaches its query's filter is done with it.
                    const float2 iv = make_float2(inv, inv), nt = make_float2(-tau_r, -tau_r);
                    uint32_t neg = 0x80000000u;
#pragma unroll
                    for (int g = 0; g < 8; ++g) {
                        const float2 s2 = __ffma2_rn(make_float2(__uint_as_float(r[4 * g + 2]), __uint_as_float(r[4 * g + 3])), iv,
                                                     make_float2(__uint_as_float(r[4 * g]), __uint_as_float(r[4 * g + 1])));
                        const float2 t2 = __fadd2_rn(s2, nt);
                        neg &= __float_as_uint(t2.x) & __float_as_uint(t2.y);
                    }
                    if (!__any_sync(0xFFFFFFFFu, (neg & 0x80000000u) == 0u)) return false;
                }
                uint32_t m = 0u;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int g = i >> 1, e = i & 1;
                    const float s = fmaf(__uint_as_float(r[4 * g + 2 + e]), inv, __uint_as_float(r[4 * g + e]));
                    m |= (s >= tau_r) ? (1u << i) : 0u;
                }
                if (resume) {
                    m &= pend;                              // only what was left over in this unit
                    pend = 0u;
                    resume = false;
                } else if (m) {
                    m &= slot_mask(u);
                }
                // Cold part (rare once the filter is warm): a warp-uniform loop over the
                // 8-column groups with a survivor in some lane; the group is re-read.
                uint32_t wm = __reduce_or_sync(0xFFFFFFFFu, m);
                if (wm == 0u) return false;
                while (wm) {
                    const int g = (__ffs(wm) - 1) >> 1;
                    wm &= ~(3u << (2 * g));
                    uint32_t v[4];                          // hi, hi, lo, lo of my two columns of the group
                    tmem_ld_frag1(unit_addr(u) + (uint32_t)(8 * g), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        if ((m >> (2 * g + e)) & 1u) {
                            const float s = fmaf(__uint_as_float(v[2 + e]), inv, __uint_as_float(v[e]));
                            const int slot = atomicAdd(&sel[q].count, 1);
                            if (slot < kQueueCap) {
                                sel[q].queue[slot] = pack_candidate(s, (uint32_t)(key0 + 64 * (u & 1) + 8 * g + e));
                                if (slot + 1 >= mlevel) fl->need_merge = 1;
                            } else {
                                pend |= 1u << (2 * g + e);
                                fl->overflow = 1;
                            }
                        }
                    }
                }
                if (__any_sync(0xFFFFFFFFu, pend != 0u)) {
                    resume = true;
                    return true;
                }
                return false;
            };
            bool first_round = true;
            while (true) {
                const float tau0 = tau[qq0], tau1 = tau[qq0 + 8];
                if (!dead && first_round) {
                    // all four units, the fragment of the next one in flight while this one is scored
                    uint32_t ra[32], rb[32];
                    tmem_ld_frag8(unit_addr(0), ra);
                    next_unit = 4;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        tmem_ld_wait();
                        if (u + 1 < 4) tmem_ld_frag8(unit_addr(u + 1), (u & 1) ? ra : rb);
                        if (process(u, (u & 1) ? rb : ra, (u >> 1) ? tau1 : tau0)) {
                            next_unit = u;
                            break;
                        }
                    }
                    tmem_ld_wait();                         // nothing in flight towards registers past this point
                } else if (!dead) {
                    int u = next_unit;
                    for (; u < 4; ++u) {                    // warp-uniform
                        uint32_t r[32];
                        tmem_ld_frag8(unit_addr(u), r);
                        tmem_ld_wait();
                        if (process(u, r, (u >> 1) ? tau1 : tau0)) break;
                    }
                    next_unit = u;
                }
                first_round = false;
                epi_bar();                                   // A: every push of this round is visible
                const int need = fl->need_merge, over = fl->overflow;
                // Flags rotate over three slots: the slot of the previous round was read by
                // everyone before arriving at A and is not written again before the next A.
                if (et == 0) {
                    EpiFlags *prev = &flags[(round + 2) % 3];
                    prev->need_merge = 0;
                    prev->overflow = 0;
                }
                round += 1;
                fl = &flags[round % 3];
                if (!(need | over)) break;
                for (int qq = ew; qq < kNQ; qq += kEpiWarps) {
                    if (sel[qq].count > 0) {
                        warp_topn_merge(&sel[qq], a.top_n, lane);
                        if (lane == 0 && qq < a.B) tau[qq] = share_tau(&a.gtau[qq], sel[qq].tau);
                    }
                }
                epi_bar();                                   // C: lists, counts and tau are settled
                if (!over) break;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty[acc]);
        }
        // flush and publish this CTA's lists
        epi_bar();
        for (int qq = ew; qq < kNQ; qq += kEpiWarps) {
            if (sel[qq].count > 0) warp_topn_merge(&sel[qq], a.top_n, lane);
            if (qq < a.B) {
                unsigned long long m = sel[qq].list[lane];
                if (lane >= a.top_n) m = 0ull;
                if (debug_check(qq < a.cand_batch && (m == 0ull || (long long)candidate_id(m) < a.N), a.status, 14))
                    a.cand[((size_t)cta * a.cand_batch + qq) * kCandStride + lane] = m;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// This kernel serves 17-64 queries on rows of three or four 64-element slabs (129-256 elements):
// its cost does not depend on the batch (the operand always has 128 rows), and from 17 queries on it
// beats the form with the keys as M (10M x 256 bf16: 0.75 against 0.90 ms at 17-32 queries; 9-16
// queries measured equal or slightly worse, 0.742-0.748 against 0.736-0.738 ms).
// On narrower rows it works too but measured no better than the other tcgen05 kernel (the
// epilogue, ~2.7 k cycles per 256 keys, is then slower than the memory stream in both).
bool scan_ummat_eligible(int d, int B)
{
    const int dslabs = (d + kSlabElems - 1) / kSlabElems;
    return B > 16 && B <= kNQ && dslabs >= 3 && dslabs <= 4;
}

cudaError_t launch_scan_ummat(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a_in, int grid,
                              cudaStream_t stream)
{
    ScanArgs a = a_in;
    if (a.tile_stride < 1) a.tile_stride = 1;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    int stages = kMaxStages;
    while (stages >= 2 && make_layout(stages, dslabs).total > 227 * 1024) --stages;
    if (stages < 2) return cudaErrorInvalidValue;
    a.stages = stages;
    const size_t smem = (size_t)make_layout(stages, dslabs).total;
    cudaError_t e;
    if (a.dtype == kF16) {
        auto k = scan_ummat_kernel<__half>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return launch_dependent(k, dim3(grid), dim3(kThreads), smem, stream, kmap, qmap, a);
    } else {
        auto k = scan_ummat_kernel<__nv_bfloat16>;
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        return launch_dependent(k, dim3(grid), dim3(kThreads), smem, stream, kmap, qmap, a);
    }
}

}  // namespace dresd
