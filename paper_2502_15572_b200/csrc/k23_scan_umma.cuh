// K2+K3 (tensor-core path, 16-bit keys) -- the kernel template; instantiated and launched from
// k23_scan_umma.cu and k23_scan_umma_merged.cu.  Eq. 3 of the paper for every key and
// up to 64 queries at once on the 5th-generation tensor cores, fused with the
// per-CTA top-n selection.  Still HBM-bound (B flop/byte is far left of the
// ridge): tensor cores are used so that the arithmetic of B queries hides
// under ONE pass over the keys.
//
// One persistent CTA per SM, ten or eleven warps:
//   warp 0    producer: one thread streams 128-row x 64-column key slabs
//             (16 KB, 128-byte swizzle) with TMA through an mbarrier ring and,
//             when the query operand is too large to stay resident, the
//             matching query slab next to each key slab;
//   warp 1    allocates TMEM; one thread issues tcgen05.mma (M = 128 key rows,
//             N = 2 columns per query: q = hi + lo/scale, K = 16 per
//             instruction, fp32 accumulators in TMEM, two accumulator buffers
//             so that the epilogue of tile t overlaps the MMAs of tile t+1);
//             tcgen05.commit releases shared-memory stages and publishes
//             finished accumulators; where the instruction stream would set the pace, a
//             second issuing thread (warp 10) takes half of the instructions (see
//             threads_of() below);
//   warps 2-9 epilogue: each thread owns one key row of the tile and half of
//             the queries' accumulator columns (two warps share a TMEM lane group),
//             reads them with tcgen05.ld and rejects the sub-tile with a packed
//             sign-bit test of score - tau when no row reaches any filter; else
//             the exact step combines hi and lo, compares with the CTA's running
//             n-th best per query and queues the survivors; queues are folded into
//             sorted 32-lane lists with shuffle-based bitonic merges, in rounds that
//             the warps hold on demand (they do not meet at every tile).
// Forms (template parameters): TSUB sub-tiles per tile (narrow rows; 33-64 queries on wide
// rows), DUAL accumulator sets with two issuing threads (wide rows), PACK2 (64-byte keys,
// two per row), MERGED (one accumulator column per query), HALVES (hi columns, then lo columns).
// Every wait is bounded; TMEM is freed on every path.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "internal.h"

namespace dresd {
namespace {

constexpr int kEpiWarps = 8;
// Two threads issue the MMAs where the instruction stream would otherwise set the pace (one
// tcgen05.mma per ~85 ns from one thread = 4 KB of keys, level with what HBM delivers): on narrow rows they
// take alternate sub-tiles; on wide rows alternate 64-element slabs, into two
// accumulator sets that the epilogue adds.
constexpr bool dual_possible(int tsub, int ncols) { return tsub == 1 && 4 * ncols <= 512; }
// MMA-issuing threads: a thread issues a tcgen05.mma about every 85 ns whatever its shape, so narrow
// rows (sub-tiles with accumulators of their own) and wide rows with two accumulator sets spread
// their instructions over two threads.  (Four threads, one per sub-tile, measured slower: 0.97
// against 0.73 ms on 23M x 64 fp16 keys with 64 queries.)
constexpr int issuers_of(int tsub, bool dual, bool merged = false)
{
    return (tsub > 1 || dual) ? 2 : 1;
}
constexpr int threads_of(int tsub, bool dual, bool merged = false, int epi_warps = kEpiWarps)
{
    return (2 + epi_warps + issuers_of(tsub, dual, merged) - 1) * 32;
}
constexpr int kTileRows = 128;
constexpr int kSlabBytes = 128;
constexpr int kSlabElems = 64;
constexpr int kKeyStageBytes = kTileRows * kSlabBytes;     // 16 KB
constexpr int kMaxStages = 12;
constexpr int kResidentLimit = 64 * 1024;                  // query operand kept in smem up to this size

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld16p(uint32_t taddr, uint32_t *r)
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t *r)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr));
}
// C consecutive accumulator columns of this thread's TMEM lane -> registers (C = 4, 8, 16, 32, 64).
template <int C> __device__ __forceinline__ void tmem_ld_n(uint32_t taddr, uint32_t *r)
{
    if constexpr (C == 4) {
        tmem_ld4(taddr, r);
    } else if constexpr (C == 8) {
        tmem_ld8(taddr, r);
    } else {
#pragma unroll
        for (int c = 0; c < C / 16; ++c) tmem_ld16p(taddr + 16 * c, r + 16 * c);
    }
}
template <int CW> __device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[CW])
{
    tmem_ld_n<CW>(taddr, r);
}
// Column-wise maximum over the 32 lanes of a warp for C values per lane, with C-1
// exchanges in total instead of 5 per value: at each step a lane keeps one half of its
// values and hands the other half to its partner.  Afterwards v[0] of lane l holds the
// maximum of column l >> (5 - log2 C) (the lanes of such a group all hold it).
template <int C, int O> struct WarpColumnMax {
    template <int N> static __device__ __forceinline__ void run(unsigned long long (&v)[N], int lane)
    {
        if constexpr (O >= 1) {
            const bool upper = (lane & O) != 0;
            if constexpr (C > 1) {
#pragma unroll
                for (int i = 0; i < C / 2; ++i) {
                    const unsigned long long send = upper ? v[i] : v[i + C / 2];
                    const unsigned long long keep = upper ? v[i + C / 2] : v[i];
                    v[i] = umax64(keep, shfl_xor_u64(send, O));
                }
                WarpColumnMax<C / 2, O / 2>::run(v, lane);
            } else {
                v[0] = umax64(v[0], shfl_xor_u64(v[0], O));
                WarpColumnMax<1, O / 2>::run(v, lane);
            }
        }
    }
};
// *p = max(*p, v) for floats shared by several warps (no NaN): non-negative floats order like
// signed integers, negative ones inversely like unsigned integers.
__device__ __forceinline__ void raise_float(float *p, float v)
{
    if (v >= 0.f) atomicMax(reinterpret_cast<int *>(p), __float_as_int(v));
    else atomicMin(reinterpret_cast<unsigned int *>(p), __float_as_uint(v));
}
template <int EW> __device__ __forceinline__ void epi_bar_n() { asm volatile("bar.sync 1, %0;" ::"n"(EW * 32) : "memory"); }

struct EpiFlags {
    int need_merge;
    int overflow;
};

// First-token windows of a filtered launch over a store sorted by first token (Section 3.5:
// only keys whose value starts with x_{t+1} can be drafted).  Entry b belongs to query b; it
// has tiles only when b is the first query that names its token, so that every window is
// scanned once.  lo/hi are key indices, tile0 the window's first tile, prefix the running
// tile count: CTA c takes the tiles c, c + G, ... of the concatenated windows.
struct Windows {
    int on;                          // 0: scan the whole store (a query without a token, or no index)
    int total;
    int tile0[kMaxBatch], lo[kMaxBatch], hi[kMaxBatch];
    int prefix[kMaxBatch + 1];
    unsigned long long qmask[kMaxBatch];   // operand column pairs (queries) that name the window's token
};

// The accumulator columns of this warp's QW queries -> registers.  Layouts of a sub-tile's NCOLS columns:
//   pairs  (PACK2 and the 8-bit copy)   query j: columns 2j (hi) and 2j+1 (lo);  CW = 2 QW consecutive columns
//   HALVES (16-bit keys, two columns)   query j: column j (hi) and column NQ + j (lo): r[0..QW) = hi, r[QW..2QW) = lo
//   MERGED (one column per query)       query j: column j;  CW = QW
// With two accumulator sets, set B (NCOLS columns further) is added to set A -- the sum of the even and of the
// odd slabs' partial products.  Loads are issued only; the caller waits.
template <int CW, int QW, int NQ, int NCOLS, bool DUAL, bool HALVES>
__device__ __forceinline__ void tmem_ld_acc(uint32_t addr, uint32_t (&r)[CW])
{
    if constexpr (HALVES) {
        tmem_ld_n<QW>(addr, r);
        tmem_ld_n<QW>(addr + NQ, r + QW);
    } else {
        tmem_ld_n<CW>(addr, r);
    }
    if constexpr (DUAL) {
        constexpr int PART = HALVES ? QW : CW;        // consecutive columns per load
        constexpr int CH = PART < 16 ? PART : 16;     // set B in chunks: 16 registers, not CW more
#pragma unroll
        for (int c = 0; c < CW / CH; ++c) {
            uint32_t r2[CH];
            const int first = c * CH;                  // register index of the chunk
            const uint32_t col = HALVES ? (uint32_t)(first < QW ? first : NQ + first - QW) : (uint32_t)first;
            tmem_ld_n<CH>(addr + NCOLS + col, r2);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < CH; ++i)
                r[first + i] = __float_as_uint(__uint_as_float(r[first + i]) + __uint_as_float(r2[i]));
        }
    }
}

// The exact selection step of the forms with a fast rejection (HALVES, MERGED) for ONE sub-tile of one
// warp: the columns are read again, compared with the filter scores, and the survivors queued.  Kept
// out of line on purpose: it runs for a few per cent of the sub-tiles, and a single copy that all
// warps and sub-tiles share stays in the instruction cache, where copies inlined into every
// unrolled sub-tile were fetched cold each time (measured: 0.74 -> 1.38 ms per call when the
// rare path was unrolled in place).  `allow` = the queries this thread's row may feed (window,
// range and, on a resumed round, the candidates that found their queue full); returns the
// queries whose candidate found the queue full now.
template <int CW, int QW, int NQ, int NCOLS, bool DUAL, bool MERGED>
static __device__ __noinline__ uint32_t epi_select(uint32_t addr, const float *tau_q, const int *want_q, int tok,
                                                   uint32_t wild, int filtered, uint32_t allow, float inv,
                                                   WarpTopN *sel_q, uint32_t row, EpiFlags *fl, int mlevel)
{
    uint32_t r[CW];
    tmem_ld_acc<CW, QW, NQ, NCOLS, DUAL, !MERGED>(addr, r);
    tmem_ld_wait();
    auto score = [&](int j) -> float {
        if constexpr (MERGED) return __uint_as_float(r[j]) * inv;
        else return fmaf(__uint_as_float(r[QW + j]), inv, __uint_as_float(r[j]));
    };
    uint32_t mask = 0u;
#pragma unroll
    for (int j4 = 0; j4 < QW / 4; ++j4) {
        const float4 t = reinterpret_cast<const float4 *>(tau_q)[j4];
        const float tt[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) mask |= (score(4 * j4 + i) >= tt[i]) ? (1u << (4 * j4 + i)) : 0u;
    }
    if (filtered) {                                     // Section 3.5: drafts must start with x_{t+1}
        uint32_t match = wild;
#pragma unroll
        for (int j4 = 0; j4 < QW / 4; ++j4) {
            const int4 w = reinterpret_cast<const int4 *>(want_q)[j4];
            match |= ((tok == w.x ? 1u : 0u) | (tok == w.y ? 2u : 0u) | (tok == w.z ? 4u : 0u) | (tok == w.w ? 8u : 0u))
                     << (4 * j4);
        }
        mask &= match;
    }
    mask &= allow;
    uint32_t pend = 0u;
    uint32_t wm = __reduce_or_sync(0xFFFFFFFFu, mask);
    while (wm) {                                        // warp-uniform: tcgen05.ld needs the whole warp
        const int j = __ffs(wm) - 1;
        wm &= wm - 1;
        // the registers cannot be indexed by a run-time j: the score's columns are read once more
        uint32_t v0, v1 = 0u;
        tmem_ld1(addr + (uint32_t)j, v0);
        if constexpr (!MERGED) tmem_ld1(addr + (uint32_t)(NQ + j), v1);
        if constexpr (DUAL) {
            uint32_t w0, w1 = 0u;
            tmem_ld1(addr + (uint32_t)j + NCOLS, w0);
            if constexpr (!MERGED) tmem_ld1(addr + (uint32_t)(NQ + j) + NCOLS, w1);
            tmem_ld_wait();
            v0 = __float_as_uint(__uint_as_float(v0) + __uint_as_float(w0));
            v1 = __float_as_uint(__uint_as_float(v1) + __uint_as_float(w1));
        } else {
            tmem_ld_wait();
        }
        const float sc = MERGED ? __uint_as_float(v0) * inv : fmaf(__uint_as_float(v1), inv, __uint_as_float(v0));
        if ((mask >> j) & 1u) {
            const int slot = atomicAdd(&sel_q[j].count, 1);
            if (slot < kQueueCap) {
                sel_q[j].queue[slot] = pack_candidate(sc, row);
                if (slot + 1 >= mlevel) fl->need_merge = 1;
            } else {
                pend |= 1u << j;
                fl->overflow = 1;
            }
        }
    }
    return pend;
}

// PACK2 (8-bit keys of 64 elements): a 128-byte row of the store holds TWO keys.  Query j then
// owns four operand rows -- (h1|0), (h2|0), (0|h1), (0|h2) -- i.e. two "virtual" queries 2j, 2j+1
// that score the even and the odd key of a row; both feed the lists and the filter of query j,
// and a candidate's id is 2 * row + parity.  tau[] is kept per virtual query (two equal
// entries per query) so that the hot loop is the same code.
//
// MERGED: ONE accumulator column per query instead of two.  The operand then holds hi' = S hi in its
// first NQ rows and lo' = S (q - hi) in the next NQ (S = 2^11 for fp16, 2^8 for bf16: both terms
// exact, neither subnormal), every k-step issues two instructions -- keys x hi', keys x lo' -- into
// the SAME columns, and the accumulator is S times the score.  Half the accumulator columns means
// half the TMEM reads and compares of the epilogue, at twice the instructions: the form for
// batches whose epilogue, not the instruction stream, sets the pace (more than 16 queries).
//
// HALVES: two columns per query, but the hi columns of all queries first and the lo columns after them
// (K1 writes the operand rows in that order), so that hi and lo of NEIGHBOURING queries sit in neighbouring
// registers and packed fp32 instructions can combine them: the same one-and-a-half instructions per score
// fast rejection -- fma.f32x2 (hi + lo/S), add.f32x2 (-tau), sign bits ANDed -- for every two-column form.
// EW epilogue warps (8, or 16: four per TMEM lane group, a quarter of the columns each).
template <typename T, int NCOLS, int TSUB, bool PACK2 = false, bool DUAL = false, bool MERGED = false,
          bool HALVES = false, int EW = kEpiWarps>
__global__ void __launch_bounds__(threads_of(TSUB, DUAL, MERGED, EW), 1)
scan_umma_kernel(const __grid_constant__ CUtensorMap keys_map, const __grid_constant__ CUtensorMap q_map,
                 const ScanArgs a, const int q_resident, const int gs)
{
    constexpr int NQ = MERGED ? NCOLS : NCOLS / 2;          // queries (padded)
    constexpr int CPQ = MERGED ? 1 : 2;                     // accumulator columns per query
    static_assert(!(MERGED && PACK2), "the packed 8-bit layout keeps two columns per query");
    static_assert(!(HALVES && (MERGED || PACK2)), "hi block | lo block: a layout of the plain two-column forms");
    constexpr bool FAST = MERGED || HALVES;                 // forms with the packed sign-bit rejection
    static_assert(!DUAL || dual_possible(TSUB, NCOLS), "two accumulator sets: wide rows only");
    constexpr int kAccCols = TSUB * NCOLS * (DUAL ? 2 : 1); // one accumulator buffer
    constexpr int kTmemCols = 2 * kAccCols < 32 ? 32 : 2 * kAccCols;
    static_assert(kTmemCols <= 512, "TMEM has 512 columns");
    constexpr int kQSlabBytes = 2 * NQ * kSlabBytes;        // operand rows: two per query in either layout
    extern __shared__ uint8_t smem_raw[];
    uint8_t *base = reinterpret_cast<uint8_t *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    // A tile is TSUB sub-tiles of 128 rows.  A pipeline stage (one full/empty barrier
    // pair, one wait and one commit) holds a GROUP of slabs: for TSUB == 1, `gs`
    // consecutive 64-column slabs of the tile; for TSUB > 1 (narrow rows) the whole
    // tile, i.e. all slabs of all its sub-tiles.
    const int n_stages = a.stages;
    const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
    const int gpt = (dslabs + gs - 1) / gs;                 // groups per tile (narrow rows: gs = dslabs, one group)
    const int slab_bytes = kKeyStageBytes + (q_resident ? 0 : kQSlabBytes);
    // TSUB > 1: a group holds the slabs sl0 .. sl0+gs-1 of ALL sub-tiles, [sub][slab], then (query operand
    // not resident) the gs operand slabs, which the sub-tiles share -- one operand slab per TSUB key slabs
    const int stage_bytes = TSUB > 1 ? gs * (TSUB * kKeyStageBytes + (q_resident ? 0 : kQSlabBytes)) : gs * slab_bytes;
    uint8_t *stages = base;
    uint8_t *qres = stages + (size_t)n_stages * stage_bytes;                 // resident query operand
    WarpTopN *sel = reinterpret_cast<WarpTopN *>(qres + (q_resident ? (size_t)dslabs * kQSlabBytes : 0));
    float *tau = reinterpret_cast<float *>(sel + NQ);
    float *ntau = tau + NQ;                                 // -tau (MERGED: -S tau), what the fast rejection adds to a score
    int *want_s = reinterpret_cast<int *>(ntau + NQ);       // first-token filter per query, -1 = off
    unsigned long long *tilemax = reinterpret_cast<unsigned long long *>(want_s + NQ);   // probe: [sub][lane group][query]
    uint64_t *full = reinterpret_cast<uint64_t *>(tilemax + 4 * TSUB * NQ);
    uint64_t *empty = full + kMaxStages;
    uint64_t *tfull = empty + kMaxStages;                   // [2] accumulator ready
    uint64_t *tempty = tfull + 2;                           // [2] accumulator drained
    uint64_t *qbar = tempty + 2;                            // resident query operand landed
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(qbar + 1);
    EpiFlags *flags = reinterpret_cast<EpiFlags *>(tmem_slot + 2);
    int *done_warps = &flags[3].need_merge;                 // epilogue warps that are through all their tiles
    Windows *win = reinterpret_cast<Windows *>(flags + 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    // the filter score of operand query q (and, MERGED, its negative in accumulator units: exact, S is a power of two)
    const float acc_scale = 1.0f / a.lo_inv_scale;
    auto set_tau = [&](int q, float t) {
        tau[q] = t;
        if constexpr (MERGED) ntau[q] = -t * acc_scale;
        else if constexpr (HALVES) ntau[q] = -t;
    };
    const long long wl = a.wait_cycles > 0 ? a.wait_cycles : kWaitCycles;   // bound of every wait below
    constexpr int kRowsPerTile = kTileRows * TSUB;
    // Narrow rows: the sub-tiles of a tile have accumulators of their own, so two threads (warps 1
    // and 10) issue the MMAs of alternate sub-tiles; each commits to the barriers for its share.
    constexpr int kIssuers = issuers_of(TSUB, DUAL, MERGED);
    constexpr int kIssuer2Warp = 2 + EW;

    if (tid == 0) {
        tma_prefetch_desc(&keys_map);                       // kernel parameters: nothing to wait for
        tma_prefetch_desc(&q_map);
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kIssuers);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&tfull[b], kIssuers);
            mbar_init(&tempty[b], EW);
        }
        mbar_init(qbar, 1);
        for (int i = 0; i < 4; ++i) {
            flags[i].need_merge = 0;
            flags[i].overflow = 0;
        }
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    // Everything above is independent of the preceding kernel; what follows reads its output
    // (the query operand, the reset filter words).
    pdl_wait();
    pdl_launch_dependents();
    if (warp >= 2 && warp < kIssuer2Warp) {
        for (int q = warp - 2; q < NQ; q += EW) {
            warp_topn_init(&sel[q], lane);
            // start from whatever the grid already knows; padding columns never pass
            if (lane == 0) {
                const int rq = PACK2 ? q >> 1 : q;          // the query this column pair belongs to
                set_tau(q, (rq < a.B && !a.no_select) ? peek_tau(&a.gtau[rq], -INFINITY) : INFINITY);
                want_s[q] = (a.first_col && rq < a.B) ? a.want_first[rq] : -1;
            }
        }
    }
    // Sorted store and a token for every query: scan those tokens' windows only.
    const bool windowed = a.win_start != nullptr && a.first_col != nullptr && a.tile_stride == 1 && !a.probe_max;
    if (windowed) {
        if (tid < kMaxBatch) {
            int t0 = 0, nt = 0, lo = 0, hi = 0;
            unsigned long long qm = 0ull;
            if (tid < a.B) {
                const int tok = a.want_first[tid];
                bool owner = tok >= 0 && tok < a.win_vocab;          // no row holds a token >= win_vocab
                for (int b = 0; b < tid && owner; ++b) owner = a.want_first[b] != tok;
                if (owner) {
                    if (debug_check(tok >= 0 && tok + 1 <= a.win_vocab, a.status, 3)) {
                        lo = a.win_start[tok];
                        hi = a.win_start[tok + 1];
                    }
                    if (hi > lo) {
                        constexpr int kKeysPerTile = PACK2 ? 2 * kRowsPerTile : kRowsPerTile;
                        t0 = lo / kKeysPerTile;
                        nt = (hi - 1) / kKeysPerTile - t0 + 1;
                        // every key of the window starts with `tok`: the token test is this constant mask
                        for (int q = tid; q < a.B; ++q)
                            if (a.want_first[q] == tok) qm |= PACK2 ? 3ull << (2 * q) : 1ull << q;
                    }
                }
            }
            win->tile0[tid] = t0;
            win->lo[tid] = lo;
            win->hi[tid] = hi;
            win->qmask[tid] = qm;
            win->prefix[tid + 1] = nt;                               // counts; summed below
        }
        __syncthreads();
        if (tid == 0) {
            int sum = 0, wild = 0;
            win->prefix[0] = 0;
            for (int b = 0; b < a.B; ++b) {                          // entries beyond B are never looked at
                sum += win->prefix[b + 1];
                win->prefix[b + 1] = sum;
                if (a.want_first[b] < 0) wild = 1;                   // that query needs every row
            }
            win->total = sum;
            win->on = !wild;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const bool win_on = windowed && win->on;
    const int n_tiles = win_on ? win->total : a.n_tiles;
    const int my_tiles = cta < n_tiles ? (n_tiles - cta + G - 1) / G : 0;
    const int n_it = my_tiles * gpt;

    if (warp == 0) {
        // ---------------------------------- producer ----------------------------------
        if (lane == 0) {
            if (q_resident) {
                mbar_arrive_expect_tx(qbar, (uint32_t)(dslabs * kQSlabBytes));
                for (int s = 0; s < dslabs; ++s)
                    tma_load_2d(qres + (size_t)s * kQSlabBytes, &q_map, s * kSlabElems, 0, qbar);
            }
            int issued = 0, wk = 0;
            for (int it = 0; it < n_it; ++it) {
                const int s = it % n_stages;
                if (it >= n_stages && !mbar_wait(&empty[s], ((it / n_stages) - 1) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
                int tile = (cta + (it / gpt) * G) * a.tile_stride;
                if (win_on) {                                    // tile of the concatenated windows -> tile of the store
                    while (win->prefix[wk + 1] <= tile) ++wk;
                    tile = win->tile0[wk] + (tile - win->prefix[wk]);
                }
                uint8_t *dst = stages + (size_t)s * stage_bytes;
                // debug build: the ring slot lies inside the stage area, the tile inside the key matrix
                if (!debug_check(s >= 0 && s < n_stages && dst + stage_bytes <= qres && tile >= 0 &&
                                     (long long)tile * kRowsPerTile < a.N + kRowsPerTile, a.status, 1))
                    break;
                // Test hook: CTA 0 "loses" the copies of one stage (they are announced to the barrier
                // but never issued), so that every wait that depends on it runs out.
                const bool lose = a.debug_lose_stage > 0 && cta == 0 && it == a.debug_lose_stage - 1;
                if constexpr (TSUB > 1) {
                    // the group's slabs of every sub-tile (rows past N read as zeros), then its operand slabs
                    const int sl0 = (it % gpt) * gs;
                    const int nsl = min(gs, dslabs - sl0);
                    mbar_arrive_expect_tx(&full[s], (uint32_t)(nsl * (TSUB * kKeyStageBytes + (q_resident ? 0 : kQSlabBytes))));
                    for (int sub = 0; sub < TSUB && !lose; ++sub)
                        for (int j = 0; j < nsl; ++j)
                            tma_load_2d(dst + (size_t)(sub * gs + j) * kKeyStageBytes, &keys_map, (sl0 + j) * kSlabElems,
                                        tile * kRowsPerTile + sub * kTileRows, &full[s]);
                    if (!q_resident)
                        for (int j = 0; j < nsl && !lose; ++j)
                            tma_load_2d(dst + (size_t)TSUB * gs * kKeyStageBytes + (size_t)j * kQSlabBytes, &q_map,
                                        (sl0 + j) * kSlabElems, 0, &full[s]);
                } else {
                    const int sl0 = (it % gpt) * gs;
                    const int nsl = min(gs, dslabs - sl0);
                    mbar_arrive_expect_tx(&full[s], (uint32_t)(nsl * slab_bytes));
                    for (int j = 0; j < nsl && !lose; ++j) {
                        tma_load_2d(dst + (size_t)j * slab_bytes, &keys_map, (sl0 + j) * kSlabElems,
                                    tile * kTileRows, &full[s]);
                        if (!q_resident)
                            tma_load_2d(dst + (size_t)j * slab_bytes + kKeyStageBytes, &q_map,
                                        (sl0 + j) * kSlabElems, 0, &full[s]);
                    }
                }
                issued = it + 1;
            }
            // Do not leave while copies into this CTA's shared memory are in flight.
            for (int it = max(0, issued - n_stages); it < issued; ++it)
                if (!mbar_wait(&full[it % n_stages], (it / n_stages) & 1, wl)) {
                    report_timeout(a.status);
                    break;
                }
            if (q_resident && !mbar_wait(qbar, 0, wl)) report_timeout(a.status);
        }
    } else if (warp == 1 || warp >= kIssuer2Warp) {
        // ---------------------------------- MMA issuer ----------------------------------
        const int issuer = warp == 1 ? 0 : warp - kIssuer2Warp + 1;
        if (lane == 0 && issuer < kIssuers) {
            // operand formats: kind::f16 -- 0 = fp16, 1 = bf16; kind::f8f6f4 -- 0 = E4M3
            constexpr bool kIs8 = std::is_same<T, E4M3Keys>::value;
            constexpr uint32_t kFmt = std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
            constexpr uint32_t idesc = (1u << 4) | (kFmt << 7) | (kFmt << 10) | ((uint32_t)(NCOLS >> 3) << 17) |
                                       ((uint32_t)(kTileRows >> 4) << 24);
            bool ok = true;
            if (q_resident && my_tiles > 0) ok = mbar_wait(qbar, 0, wl);
            for (int tl = 0; tl < my_tiles && ok; ++tl) {
                const int acc = tl & 1, use = tl >> 1;
                if (use >= 1 && !mbar_wait(&tempty[acc], (use - 1) & 1, wl)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
                for (int g = 0; g < gpt; ++g) {
                    const int it = tl * gpt + g;
                    const int s = it % n_stages;
                    if (!mbar_wait(&full[s], (it / n_stages) & 1, wl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st_addr = smem_u32(stages + (size_t)s * stage_bytes);
                    if constexpr (TSUB > 1) {
                        const int sl0 = g * gs;
                        const int nsl = min(gs, dslabs - sl0);
                        for (int sub = issuer; sub < TSUB; sub += kIssuers)
                            for (int jj = 0; jj < nsl; ++jj) {
                                const int j = sl0 + jj;                       // slab of the row
                                const uint64_t a_desc = make_desc(st_addr + (uint32_t)((sub * gs + jj) * kKeyStageBytes));
                                const uint64_t b_desc = make_desc(
                                    q_resident ? smem_u32(qres + (size_t)j * kQSlabBytes)
                                               : st_addr + (uint32_t)(TSUB * gs * kKeyStageBytes + jj * kQSlabBytes));
                                // a last slab that the row fills only in part (zeros beyond d) needs only
                                // the 32-byte steps that hold data
                                const int ksteps = min(4, (a.d - j * kSlabElems + 15) / 16);
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    if (k >= ksteps) break;
                                    if constexpr (kIs8) {
                                        umma_f8(d_tmem + (uint32_t)(sub * NCOLS), a_desc + 2 * k, b_desc + 2 * k, idesc,
                                                (j + k) != 0);
                                    } else {
                                        umma_f16(d_tmem + (uint32_t)(sub * NCOLS), a_desc + 2 * k, b_desc + 2 * k, idesc,
                                                 (j + k) != 0);
                                        if constexpr (MERGED)   // the lo' rows, NQ operand rows further, same columns
                                            umma_f16(d_tmem + (uint32_t)(sub * NCOLS), a_desc + 2 * k,
                                                     b_desc + (uint64_t)((NQ * kSlabBytes) >> 4) + 2 * k, idesc, 1);
                                    }
                                }
                            }
                    } else {
                        const int sl0 = g * gs;
                        const int nsl = min(gs, dslabs - sl0);
                        for (int j = 0; j < nsl; ++j) {
                            if (DUAL && ((sl0 + j) & 1) != issuer) continue;      // the other thread's slab
                            const uint32_t a_addr = st_addr + (uint32_t)(j * slab_bytes);
                            const uint32_t b_addr = q_resident ? smem_u32(qres + (size_t)(sl0 + j) * kQSlabBytes)
                                                               : a_addr + kKeyStageBytes;
                            const uint64_t a_desc = make_desc(a_addr), b_desc = make_desc(b_addr);
                            const int ksteps = min(4, (a.d - (sl0 + j) * kSlabElems + 15) / 16);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {  // 4 x K=16 inside the 128-byte swizzle row: +32 bytes each
                                if (k >= ksteps) break;
                                // a set starts afresh with the first step of its first slab (slab 0 or 1)
                                const uint32_t d_set = d_tmem + (DUAL ? (uint32_t)(issuer * NCOLS) : 0u);
                                const bool accumulate = (DUAL ? (sl0 + j - issuer) : (sl0 + j)) + k != 0;
                                if constexpr (kIs8) {
                                    umma_f8(d_set, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                                } else {
                                    umma_f16(d_set, a_desc + 2 * k, b_desc + 2 * k, idesc, accumulate);
                                    if constexpr (MERGED)
                                        umma_f16(d_set, a_desc + 2 * k, b_desc + (uint64_t)((NQ * kSlabBytes) >> 4) + 2 * k,
                                                 idesc, 1);
                                }
                            }
                        }
                    }
                    tc_commit(&empty[s]);             // group reusable once these MMAs have read it
                }
                if (!ok) break;
                tc_commit(&tfull[acc]);               // accumulator complete
            }
            if (!ok) report_timeout(a.status);
        }
    } else if (warp < kIssuer2Warp) {
        // ---------------------------------- epilogue ----------------------------------
        // Eight warps: warp w may read TMEM lanes 32*(w&3)..+31 (one key row per thread and
        // sub-tile); the two warps that share a lane group split the accumulator columns.
        constexpr int CW = NCOLS / (EW / 4);                // columns per warp
        constexpr int QW = CW / CPQ;                        // queries per warp
        const int ew = warp - 2;                            // 0..7
        const int lane_grp = warp & 3;
        const int half = ew >> 2;
        const int et = ew * 32 + lane;
        // Few queries on narrow rows (all of them within one warp's columns, several sub-tiles per
        // tile): the two warps of a lane group split the SUB-TILES instead, so that neither spends
        // its time on columns of padding.
        const bool split_subs = EW == 8 && TSUB >= 2 && (PACK2 ? 2 * a.B : a.B) <= QW;
        const int qbase = split_subs ? 0 : half * QW;
        // a warp whose columns are all padding (few queries, one sub-tile per tile) only keeps the barriers
        const bool no_cols = qbase >= (PACK2 ? 2 * a.B : a.B);
        const uint32_t lane_addr = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(qbase * (HALVES ? 1 : CPQ));
        const float inv = a.lo_inv_scale;
        // a round is asked for when a queue of 32 holds this many: 24 measured 1-4 % ahead of 16 (fewer rounds)
        const int mlevel = a.merge_level > 0 ? a.merge_level : 24;
        // score of this warp's j-th query from the registers of ld_cols: hi + lo / S, or acc / S
        auto score_at = [&](const uint32_t (&r)[CW], int j) -> float {
            if constexpr (MERGED) return __uint_as_float(r[j]) * inv;
            else if constexpr (HALVES) return fmaf(__uint_as_float(r[QW + j]), inv, __uint_as_float(r[j]));
            else return fmaf(__uint_as_float(r[2 * j + 1]), inv, __uint_as_float(r[2 * j]));
        };
        // accumulator reads (issued only; the caller waits): with two sets, set B (NCOLS columns further)
        // is added to set A -- the sum of the even and of the odd slabs' partial products
        auto ld_cols = [&](uint32_t addr, uint32_t (&r)[CW]) { tmem_ld_acc<CW, QW, NQ, NCOLS, DUAL, HALVES>(addr, r); };
        // the same score re-read from TMEM: `addr` = the sub-tile's first column of this warp, j = its query
        auto ld_score = [&](uint32_t addr, int j) -> float {
            if constexpr (MERGED) {
                uint32_t v0;
                tmem_ld1(addr + (uint32_t)j, v0);
                if constexpr (DUAL) {
                    uint32_t w0;
                    tmem_ld1(addr + (uint32_t)j + NCOLS, w0);
                    tmem_ld_wait();
                    return (__uint_as_float(v0) + __uint_as_float(w0)) * inv;
                }
                tmem_ld_wait();
                return __uint_as_float(v0) * inv;
            } else if constexpr (HALVES) {
                uint32_t v0, v1;
                tmem_ld1(addr + (uint32_t)j, v0);
                tmem_ld1(addr + (uint32_t)(NQ + j), v1);
                if constexpr (DUAL) {
                    uint32_t w0, w1;
                    tmem_ld1(addr + (uint32_t)j + NCOLS, w0);
                    tmem_ld1(addr + (uint32_t)(NQ + j) + NCOLS, w1);
                    tmem_ld_wait();
                    v0 = __float_as_uint(__uint_as_float(v0) + __uint_as_float(w0));
                    v1 = __float_as_uint(__uint_as_float(v1) + __uint_as_float(w1));
                }
                tmem_ld_wait();
                return fmaf(__uint_as_float(v1), inv, __uint_as_float(v0));
            } else {
                uint32_t v0, v1;
                tmem_ld2(addr + (uint32_t)(2 * j), v0, v1);
                if constexpr (DUAL) {
                    uint32_t w0, w1;
                    tmem_ld2(addr + (uint32_t)(2 * j) + NCOLS, w0, w1);
                    tmem_ld_wait();
                    v0 = __float_as_uint(__uint_as_float(v0) + __uint_as_float(w0));
                    v1 = __float_as_uint(__uint_as_float(v1) + __uint_as_float(w1));
                }
                tmem_ld_wait();
                return fmaf(__uint_as_float(v1), inv, __uint_as_float(v0));
            }
        };
        const float4 *tau4 = reinterpret_cast<const float4 *>(tau + qbase);
        const int4 *want4 = reinterpret_cast<const int4 *>(want_s + qbase);
        const bool filtered = a.first_col != nullptr && !win_on;    // windows carry their token
        uint32_t wmatch = 0xFFFFFFFFu;                      // this warp's queries that the tile's window serves
        uint32_t wild = 0u;                                 // this warp's queries without a token filter
        for (int j = 0; j < QW; ++j) wild |= (want_s[qbase + j] < 0) ? (1u << j) : 0u;
        // A warp whose wait expired goes "dead": it does no more work and no more
        // waits, but keeps taking part in every barrier so that nobody is left behind.
        bool dead = false;
        int round = 0;                                      // barrier-A count: selects the flag slot
        EpiFlags *fl = &flags[0];
        // Cold start.  While a query has no filter score, every row is a candidate and the 32-entry
        // queues overflow round after round (a 512-row tile: 16 rounds of barriers and merges, ~4 us).
        // So on the first tile of a scan, and of every window, the tile is cut into 32 groups of rows
        // per query; the n-th largest of the 32 group maxima is reached by n rows of the tile (one per
        // group), hence by the final n-th best too, and becomes the filter score before the tile is
        // scored in earnest: about n rows then pass, one merge instead of sixteen.
        uint32_t active = 0u;                               // this warp's column pairs that belong to real queries
        for (int j = 0; j < QW; ++j)
            if ((PACK2 ? (qbase + j) >> 1 : qbase + j) < a.B && !a.no_select) active |= 1u << j;
        // Rounds.  Survivors go to per-query queues with atomic slot claims; folding the queues into the
        // sorted lists needs the whole CTA: barrier A (every push so far is visible), the flags of the
        // round, the folds (a warp per query), barrier C (lists, counts and filter scores settled).  A
        // round is held when a queue has reached the merge level or overflowed.  Warps do NOT meet at
        // every tile: a warp looks at the flag words at the end of a tile and while it waits for an
        // accumulator, and goes to barrier A when one is set -- so that the occasional warp with
        // survivors to queue does not hold up the seven others tile after tile.  All warps take part in
        // every round (bar.sync counts them), whichever tile each is at; they are never more than two
        // tiles apart (two accumulator buffers).  Token windows and the probe pass, whose tiles have
        // barriers of their own, keep a round per tile.
        const bool free_run = !win_on && !a.probe_max && !a.round_per_tile;
        int last_over = 0, last_done = 0;
        auto round_wanted = [&]() -> bool {
            return (*reinterpret_cast<volatile int *>(&fl->need_merge) | *reinterpret_cast<volatile int *>(&fl->overflow)) != 0;
        };
        auto one_round = [&]() -> int {
            epi_bar_n<EW>();                                       // A: every push so far is visible
            const int need = fl->need_merge, over = fl->overflow;
            last_done = *reinterpret_cast<volatile int *>(done_warps);
            last_over = over;
            // Flags rotate over three slots: the slot of the previous round was read by
            // everyone before arriving at A and is not written again before the next A.
            if (et == 0) {
                EpiFlags *prev = &flags[(round + 2) % 3];
                prev->need_merge = 0;
                prev->overflow = 0;
            }
            round += 1;
            fl = &flags[round % 3];
            if (need | over) {
                for (int q = ew; q < NQ; q += EW) {
                    if (sel[q].count > 0) {
                        warp_topn_merge(&sel[q], a.top_n, lane);
                        if (lane == 0 && q < a.B) {
                            const float t = share_tau(&a.gtau[q], sel[q].tau);
                            if constexpr (PACK2) tau[2 * q] = tau[2 * q + 1] = t;
                            else set_tau(q, t);
                        }
                    }
                }
            }
            // C: lists, counts and filter scores are settled.  Free-running warps hold it in every round, so
            // that nobody leaves a round (and counts itself done) before all have read its flags.
            if ((need | over) || free_run) epi_bar_n<EW>();
            return over;
        };
        auto attend_rounds = [&]() {
            while (one_round()) {}
        };
        int wk = 0, wk_seen = -1;
        for (int tl = 0; tl < my_tiles; ++tl) {
            const int acc = tl & 1, use = tl >> 1;
            long long tile = (long long)(cta + tl * G) * a.tile_stride;
            long long klo = 0, khi = PACK2 ? 2 * a.N : a.N;  // keys of this tile that count
            if (win_on) {
                while (win->prefix[wk + 1] <= tile) ++wk;
                tile = win->tile0[wk] + (tile - win->prefix[wk]);
                klo = win->lo[wk];
                khi = win->hi[wk];
                wmatch = (uint32_t)(win->qmask[wk] >> qbase);
            }
            const bool cold_tile = !a.no_select && !a.probe_max && (tl == 0 || wk != wk_seen);   // same in all warps
            wk_seen = wk;
            const long long row0 = tile * kRowsPerTile + lane_grp * 32 + lane;
            // first stored token of this thread's rows (filtered calls), requested before the wait
            // (PACK2: of the row's two keys -- first_col is indexed by key, two per row)
            int tok[TSUB], tok1[TSUB];
#pragma unroll
            for (int sub = 0; sub < TSUB; ++sub) {
                const long long r = row0 + sub * kTileRows;
                tok[sub] = tok1[sub] = 0;
                if (filtered && r < a.N) {
                    if constexpr (PACK2) {
                        const int2 t = *reinterpret_cast<const int2 *>(a.first_col + 2 * r);
                        tok[sub] = t.x;
                        tok1[sub] = t.y;
                    } else {
                        if (debug_check(r >= 0 && r < a.N, a.status, 2)) tok[sub] = a.first_col[r];
                    }
                }
            }
            // every fourth tile, pull the grid-wide filter (other CTAs may know a better n-th best); the
            // word comes from L2, so it is requested before the wait for the accumulator and used after it
            const bool pull = (tl & 3) == 0 && et < a.B && !a.no_select;
            unsigned int gword = 0u;
            if (pull) gword = *reinterpret_cast<const volatile unsigned int *>(&a.gtau[et]);
            // The wait is decided warp-wide (votes): what follows -- rounds with their CTA barriers, tcgen05.ld --
            // needs the whole warp, so no lane may leave the loop, or enter a round, on its own view of the barrier.
            if (!__all_sync(0xFFFFFFFFu, dead || mbar_try_wait(&tfull[acc], use & 1))) {
                const long long t0 = clock64();
                while (!__all_sync(0xFFFFFFFFu, mbar_try_wait(&tfull[acc], use & 1))) {
                    // a warp that waits at the round's barrier holds its accumulator buffer, which this
                    // wait may depend on: rounds are attended from here too
                    if (free_run && __any_sync(0xFFFFFFFFu, round_wanted())) attend_rounds();
                    if (__any_sync(0xFFFFFFFFu, clock64() - t0 > wl)) {
                        if (lane == 0) report_timeout(a.status);
                        dead = true;
                        break;
                    }
                }
            }
            tc_fence_after();
            if (pull && gword) {
                const float g = ordered_to_float(gword);
                if constexpr (PACK2) {
                    if (g > tau[2 * et]) tau[2 * et] = tau[2 * et + 1] = g;
                } else {
                    if (g > tau[et]) set_tau(et, g);
                }
            }
            const uint32_t acc_addr = lane_addr + (uint32_t)(acc * kAccCols);
            if (a.probe_max) {
                // Probe pass: no filtering and no lists -- only the best row of each sub-tile
                // per query (at most 32 per CTA, so they fit the queue as they are).  The n-th
                // largest of all CTAs' bests is a valid filter: at least n rows reach it.
#pragma unroll
                for (int sub = 0; sub < TSUB; ++sub) {
                    if ((split_subs && (sub & 1) != half) || no_cols) continue;
                    const long long row = row0 + sub * kTileRows;
                    const bool row_ok = row < a.N;
                    unsigned long long *slot = tilemax + (size_t)(sub * 4 + lane_grp) * NQ + qbase;
                    if (!dead) {
                        uint32_t r[CW];
                        ld_cols(acc_addr + (uint32_t)(sub * NCOLS), r);
                        tmem_ld_wait();
                        // per-query maximum over the warp's 32 rows.  Only the SCORES matter here (the probe
                        // yields a filter score, never a result row), so the maximum is one redux.sync per
                        // query on the order-preserving integer image of the score; the row that goes with
                        // it is any row of this sub-tile and lane group (distinct per entry, never returned).
                        // Lane j keeps query j's maximum and stores it after the loop: no store inside the
                        // loop, so that the reductions of different queries overlap.
                        int wants[QW];
#pragma unroll
                        for (int j4 = 0; j4 < QW / 4; ++j4) {
                            const int4 w = want4[j4];
                            wants[4 * j4] = w.x; wants[4 * j4 + 1] = w.y; wants[4 * j4 + 2] = w.z; wants[4 * j4 + 3] = w.w;
                        }
                        uint32_t mine = 0u;
#pragma unroll
                        for (int j = 0; j < QW; ++j) {
                            const float s = score_at(r, j);
                            const int tkj = (PACK2 && ((qbase + j) & 1)) ? tok1[sub] : tok[sub];
                            const bool ok = row_ok && (wants[j] < 0 || tkj == wants[j]) && s > -INFINITY;   // false for NaN
                            const uint32_t best = __reduce_max_sync(0xFFFFFFFFu, ok ? float_to_ordered(s + 0.0f) : 0u);
                            if (lane == j) mine = best;
                        }
                        if (lane < QW) {
                            const uint32_t id = PACK2 ? (uint32_t)(2 * row + ((qbase + lane) & 1)) : (uint32_t)row;
                            slot[lane] = mine ? ((unsigned long long)mine << 32) | (0xFFFFFFFFu - id) : 0ull;
                        }
                    } else if (lane < QW) {
                        slot[lane] = 0ull;
                    }
                }
                epi_bar_n<EW>();                                   // all lane groups have written
                // a lane per (query of this warp, sub-tile): the best of the four lane groups joins the queue
                {
                    const int q = ew + EW * (lane / TSUB), sub = lane % TSUB;
                    if (q < a.B) {
                        const unsigned long long *m = tilemax + (size_t)(sub * 4) * NQ + (PACK2 ? 2 * q : q);
                        unsigned long long v = umax64(umax64(m[0], m[NQ]), umax64(m[2 * NQ], m[3 * NQ]));
                        if constexpr (PACK2)               // the odd keys of the same rows
                            v = umax64(v, umax64(umax64(m[1], m[NQ + 1]), umax64(m[2 * NQ + 1], m[3 * NQ + 1])));
                        if (v) {
                            const int at = atomicAdd(&sel[q].count, 1);
                            if (at < kQueueCap) sel[q].queue[at] = v;
                            else atomicSub(&sel[q].count, 1);
                        }
                    }
                }
                epi_bar_n<EW>();                                   // slots may be rewritten for the next tile
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&tempty[acc]);
                continue;
            }
            auto okmask_of = [&](long long row) -> uint32_t {   // columns whose key lies in the window (or the store)
                if constexpr (PACK2)
                    return ((2 * row >= klo && 2 * row < khi) ? 0x55555555u : 0u) |
                           ((2 * row + 1 >= klo && 2 * row + 1 < khi) ? 0xAAAAAAAAu : 0u);
                else
                    return (row >= klo && row < khi) ? 0xFFFFFFFFu : 0u;
            };
            if (cold_tile) {
                constexpr int kGroupRows = 4 * TSUB;        // 32 groups over the tile's 128 * TSUB rows
                constexpr int kGroupsPerUnit = 32 / kGroupRows;
                epi_bar_n<EW>();                                  // tau[] is settled: every warp sees the same cold queries
                uint32_t todo = 0u;
                for (uint32_t m = active & wmatch; m; m &= m - 1) {
                    const int j = __ffs(m) - 1;
                    if (!(tau[qbase + j] > -INFINITY)) todo |= 1u << j;
                }
#pragma unroll
                for (int sub = 0; sub < TSUB; ++sub) {
                    if ((split_subs && (sub & 1) != half) || no_cols) continue;
                    const uint32_t ok = okmask_of(row0 + sub * kTileRows);
                    const int slot = (sub * 4 + lane_grp) * kGroupsPerUnit + lane / kGroupRows;
                    for (uint32_t m = todo; m; m &= m - 1) {            // warp-uniform
                        const int j = __ffs(m) - 1;
                        uint32_t key = 0u;
                        if (!dead) {
                            const float sc = ld_score(acc_addr + (uint32_t)(sub * NCOLS), j);
                            bool valid = ((ok >> j) & 1u) && sc > -INFINITY;            // false for NaN
                            if (filtered) {
                                const int w = want_s[qbase + j];
                                const int tkj = (PACK2 && (j & 1)) ? tok1[sub] : tok[sub];
                                valid = valid && (w < 0 || tkj == w);
                            }
                            key = valid ? float_to_ordered(sc + 0.0f) : 0u;
                            const uint32_t grp = ((1u << kGroupRows) - 1u) << (lane & ~(kGroupRows - 1));
                            key = __reduce_max_sync(grp, key);
                        }
                        // the queue is empty on a cold tile: its first 128 bytes take the group maxima
                        if (lane % kGroupRows == 0) reinterpret_cast<uint32_t *>(sel[qbase + j].queue)[slot] = key;
                    }
                }
                epi_bar_n<EW>();
                const unsigned long long wq = win_on ? win->qmask[wk] : ~0ull;
                for (int q = ew; q < NQ; q += EW) {
                    const int rq = PACK2 ? q >> 1 : q;
                    if (rq >= a.B || !((wq >> q) & 1ull) || tau[q] > -INFINITY) continue;   // warp-uniform
                    unsigned long long x = reinterpret_cast<const uint32_t *>(sel[q].queue)[lane];
                    __syncwarp();
                    x = warp_sort_desc(x, lane);
                    const uint32_t nth = (uint32_t)shfl_u64(x, a.top_n - 1);
                    if (lane == 0 && nth) {
                        const float t = share_tau(&a.gtau[rq], ordered_to_float(nth));
                        if constexpr (PACK2) {               // the even and the odd keys feed one query
                            raise_float(&tau[2 * rq], t);
                            raise_float(&tau[2 * rq + 1], t);
                        } else {
                            set_tau(q, t);
                        }
                    }
                }
                epi_bar_n<EW>();
            }
            uint32_t pending[TSUB];                         // queries whose candidate found the queue full
#pragma unroll
            for (int sub = 0; sub < TSUB; ++sub) pending[sub] = 0u;
            bool first = true;
            int must = 0;                                   // the last round left an overflow: the next one is attended too
            while (true) {
#pragma unroll
                for (int sub = 0; sub < TSUB; ++sub) {
                    const long long row = row0 + sub * kTileRows;
                    const uint32_t okmask = okmask_of(row);
                    // warp-uniform decision: tcgen05.ld needs the whole warp
                    if (dead || no_cols || (split_subs && (sub & 1) != half) ||
                        !(first || __any_sync(0xFFFFFFFFu, pending[sub] != 0u)))
                        continue;
                    if constexpr (FAST) {
                        // Fast rejection, one instruction per score (one and a half with two columns per query):
                        // score + (-tau) has its sign bit clear exactly when the score reaches the filter (the
                        // sum of two floats is never rounded across zero); packed fp32 instructions take two
                        // queries at a time -- MERGED: accumulator + (-S tau); HALVES: hi + lo/S, rounded as in
                        // the exact step, then + (-tau) -- and the sign bits are ANDed three words per
                        // instruction.  A warp in which no row reaches any filter -- the usual case once the
                        // filter is warm -- is done with the sub-tile.
                        if (first) {
                            uint32_t r[CW];
                            ld_cols(acc_addr + (uint32_t)(sub * NCOLS), r);
                            tmem_ld_wait();
                            uint32_t neg = 0x80000000u;
                            const float4 *nt4 = reinterpret_cast<const float4 *>(ntau + qbase);
                            const float2 iv = make_float2(inv, inv);
#pragma unroll
                            for (int j4 = 0; j4 < QW / 4; ++j4) {
                                const float4 t = nt4[j4];
                                float2 s0 = make_float2(__uint_as_float(r[4 * j4]), __uint_as_float(r[4 * j4 + 1]));
                                float2 s1 = make_float2(__uint_as_float(r[4 * j4 + 2]), __uint_as_float(r[4 * j4 + 3]));
                                if constexpr (HALVES) {
                                    s0 = __ffma2_rn(make_float2(__uint_as_float(r[QW + 4 * j4]), __uint_as_float(r[QW + 4 * j4 + 1])), iv, s0);
                                    s1 = __ffma2_rn(make_float2(__uint_as_float(r[QW + 4 * j4 + 2]), __uint_as_float(r[QW + 4 * j4 + 3])), iv, s1);
                                }
                                const float2 x = __fadd2_rn(s0, make_float2(t.x, t.y));
                                const float2 y = __fadd2_rn(s1, make_float2(t.z, t.w));
                                neg &= __float_as_uint(x.x) & __float_as_uint(x.y);
                                neg &= __float_as_uint(y.x) & __float_as_uint(y.y);
                            }
                            if (!__any_sync(0xFFFFFFFFu, (neg & 0x80000000u) == 0u)) continue;
                        }
                        pending[sub] = epi_select<CW, QW, NQ, NCOLS, DUAL, MERGED>(
                            acc_addr + (uint32_t)(sub * NCOLS), tau + qbase, want_s + qbase, tok[sub], wild, filtered ? 1 : 0,
                            first ? (okmask & wmatch) : pending[sub], inv, sel + qbase, (uint32_t)row, fl, mlevel);
                        continue;
                    }
                    uint32_t r[CW];
                    ld_cols(acc_addr + (uint32_t)(sub * NCOLS), r);
                    tmem_ld_wait();
                    // Hot part, branch-free and compact: one bit per query whose score
                    // reaches the filter.
                    uint32_t mask = 0u;
#pragma unroll
                    for (int j4 = 0; j4 < QW / 4; ++j4) {
                        const float4 t = tau4[j4];
                        const float tt[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const int j = 4 * j4 + i;
                            mask |= (score_at(r, j) >= tt[i]) ? (1u << j) : 0u;
                        }
                    }
                    if (filtered) {                         // Section 3.5: drafts must start with x_{t+1}
                        uint32_t match = wild;
                        // column pairs alternate between the row's even and odd key when packed (qbase is even)
                        const int tk = tok[sub], tko = PACK2 ? tok1[sub] : tok[sub];
#pragma unroll
                        for (int j4 = 0; j4 < QW / 4; ++j4) {
                            const int4 w = want4[j4];
                            match |= ((tk == w.x ? 1u : 0u) | (tko == w.y ? 2u : 0u) | (tk == w.z ? 4u : 0u) |
                                      (tko == w.w ? 8u : 0u)) << (4 * j4);
                        }
                        mask &= match;
                    }
                    mask &= first ? (okmask & wmatch) : pending[sub];
                    pending[sub] = 0u;
                    // Cold part (rare once the filter is warm), kept out of the hot code:
                    // a warp-uniform loop over the queries that have a survivor in some
                    // lane; the two accumulator columns are re-read from TMEM.
                    uint32_t wm = __reduce_or_sync(0xFFFFFFFFu, mask);
                    while (wm) {
                        const int j = __ffs(wm) - 1;
                        wm &= wm - 1;
                        const float s = ld_score(acc_addr + (uint32_t)(sub * NCOLS), j);
                        if ((mask >> j) & 1u) {
                            const int q = PACK2 ? (qbase + j) >> 1 : qbase + j;
                            const uint32_t id = PACK2 ? (uint32_t)(2 * row + ((qbase + j) & 1)) : (uint32_t)row;
                            const int slot = atomicAdd(&sel[q].count, 1);
                            if (slot < kQueueCap) {
                                sel[q].queue[slot] = pack_candidate(s, id);
                                if (slot + 1 >= mlevel) fl->need_merge = 1;
                            } else {
                                pending[sub] |= 1u << j;
                                fl->overflow = 1;
                            }
                        }
                    }
                }
                first = false;
                bool mine = false;
#pragma unroll
                for (int sub = 0; sub < TSUB; ++sub) mine = mine || pending[sub] != 0u;
                mine = __any_sync(0xFFFFFFFFu, mine);
                // Nobody has asked for a round (no queue reached the merge level, none overflowed): on to
                // the next tile without a barrier.
                if (free_run && !must && !mine && !round_wanted()) break;
                must = one_round();
                if (!must) break;
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty[acc]);
        }
        // Through all tiles.  Other warps may still ask for rounds: they are attended until every warp is here.
        if (free_run) {
            if (lane == 0) atomicAdd(done_warps, 1);
            while (true) {
                one_round();
                if (last_done == EW && !last_over) break;
            }
        } else {
            epi_bar_n<EW>();
        }
        // flush and publish this CTA's lists
        for (int q = ew; q < NQ; q += EW) {
            if (sel[q].count > 0) warp_topn_merge(&sel[q], a.top_n, lane);
            if (q < a.B) {
                unsigned long long m = sel[q].list[lane];
                if (lane >= a.top_n) m = 0ull;
                // debug build: the list lies in this launch's part of the candidate array, its rows in the store
                if (debug_check(q < a.cand_batch && (m == 0ull || (long long)candidate_id(m) < (PACK2 ? 2 * a.N + 1 : a.N)),
                                a.status, 4))
                    a.cand[((size_t)cta * a.cand_batch + q) * kCandStride + lane] = m;
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
}  // namespace dresd
