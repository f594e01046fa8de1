// K2+K3 (tensor-core path, 16-bit keys and their 8-bit copy): planning and launch of
// scan_umma_kernel (k23_scan_umma.cuh) in its two-columns-per-query forms.  The one-column
// ("merged") forms are instantiated in k23_scan_umma_merged.cu.
#include "k23_scan_umma.cuh"
#include "k23_scan_umma_plan.h"

namespace dresd {
namespace {

template <typename T, int NCOLS, int TSUB, bool PACK2 = false>
cudaError_t launch_one(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                       int grid, cudaStream_t stream)
{
    // 16-bit keys, one key per row: the operand rows come as hi block | lo block (K1 layout 4)
    constexpr bool HALVES = !PACK2 && !std::is_same<T, E4M3Keys>::value;
    if constexpr (2 * TSUB * NCOLS > 512) {
        return cudaErrorInvalidValue;
    } else {
        const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
        if constexpr (dual_possible(TSUB, NCOLS)) {
            if (umma_dual_pays(dslabs, NCOLS)) {
                auto kernel = scan_umma_kernel<T, NCOLS, TSUB, PACK2, true, false, HALVES>;
                cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
                if (e != cudaSuccess) return e;
                return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, true)), p.smem, stream, kmap, qmap, a,
                                        p.q_resident, p.gs);
            }
        }
        if constexpr (HALVES && TSUB > 1 && NCOLS == 128) {
            // 33-64 queries, two sub-tiles per tile: sixteen selection warps (four per TMEM lane group, a
            // quarter of the queries each) hide more of the epilogue's latency than eight.  Interleaved A/B,
            // 3 GB stores, 8 -> 16 warps: d = 128 0.638 -> 0.632 ms (n = 32: 0.738 -> 0.676), d = 512
            // 0.693 -> 0.671, d = 2048 0.634 -> 0.616, d = 1024 with 40 queries and n = 32 0.682 -> 0.640;
            // with 17-32 queries (64 columns) eight warps stay ahead (d = 128: 0.521 against 0.540).
            if (a.epi_warps != 8) {
                auto kernel = scan_umma_kernel<T, NCOLS, TSUB, PACK2, false, false, HALVES, 16>;
                cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
                if (e != cudaSuccess) return e;
                return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, false, false, 16)), p.smem, stream, kmap,
                                        qmap, a, p.q_resident, p.gs);
            }
        }
        auto kernel = scan_umma_kernel<T, NCOLS, TSUB, PACK2, false, false, HALVES>;
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
        if (e != cudaSuccess) return e;
        return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, false)), p.smem, stream, kmap, qmap, a,
                                p.q_resident, p.gs);
    }
}

template <typename T, int NCOLS, bool PACK2 = false>
cudaError_t launch_tsub(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                        int grid, cudaStream_t stream)
{
    switch (p.tsub) {
    case 4: return launch_one<T, NCOLS, 4, PACK2>(kmap, qmap, a, p, grid, stream);
    case 2: return launch_one<T, NCOLS, 2, PACK2>(kmap, qmap, a, p, grid, stream);
    default: return launch_one<T, NCOLS, 1, PACK2>(kmap, qmap, a, p, grid, stream);
    }
}

}  // namespace

// ---- planning (shared with the merged forms) ----------------------------------------------
int umma_queries_padded(int B) { return B <= 8 ? 8 : B <= 16 ? 16 : B <= 32 ? 32 : 64; }

// Narrow rows (one or two 64-element slabs): several 128-row sub-tiles per tile so that a
// pipeline stage is 32-64 KB and the per-tile barrier round trips are amortised.
int umma_tsub_of(int d, int ncols)
{
    const int dslabs = (d + kSlabElems - 1) / kSlabElems;
    // 33-64 queries (two columns each) on rows wider than 256: the 16 KB operand slab does not stay in
    // shared memory (128 rows x d) and would come from L2 once per 16 KB key slab; with two sub-tiles per
    // tile one operand slab serves 32 KB of keys (and the two sub-tiles have an MMA-issuing thread each)
    if (dslabs > 4 && ncols == 128) return 2;
    if (dslabs > 2) return 1;
    int t = 4 / dslabs;                              // 4 slabs per stage
    while (2 * t * ncols > 512) t >>= 1;             // two accumulator buffers in 512 TMEM columns
    return t;
}

// Measured against one issuer on 3 GB stores.  Up to 8 queries: rows of 3-6 slabs 5-14 % faster (d = 256:
// 0.775 -> 0.739 ms on 10M rows), 15 and more slabs 2-6 % faster, 7-12 slabs 4-10 % slower.  9-16 queries:
// faster at every width (d = 512: 0.51 -> 0.45 ms).  17-64 queries (rows wider than 256): 10-25 % faster.
// Rows of 3-4 slabs with more than 16 queries normally run the kernel with the keys as N; when they come
// here (token windows, "keys_as_m") they keep one accumulator set, whose sums are bit-identical to that kernel's.
bool umma_dual_pays(int dslabs, int ncols)
{
    if (ncols >= 64) return dslabs > 4;
    if (ncols == 32) return true;                     // 9-16 queries: 6-20 % faster at every width measured
    return dslabs <= 6 || dslabs >= 15;               // up to 8 queries: 7-12 slabs measured 4-10 % slower
}

UmmaPlan umma_make_plan(int d, int B, bool merged)
{
    UmmaPlan p{};
    const int nq = umma_queries_padded(B);
    p.ncols = merged ? nq : 2 * nq;
    p.tsub = umma_tsub_of(d, p.ncols);
    const int dslabs = (d + kSlabElems - 1) / kSlabElems;
    const size_t op_slab = (size_t)2 * nq * kSlabBytes;             // one 64-element slab of the query operand
    const size_t qbytes = (size_t)dslabs * op_slab;
    p.q_resident = qbytes <= (size_t)kResidentLimit;
    const size_t fixed = 1024 + (p.q_resident ? qbytes : 0) + sizeof(WarpTopN) * nq +
                         (2 * sizeof(float) + sizeof(int) + 4 * p.tsub * sizeof(unsigned long long)) * nq +
                         sizeof(uint64_t) * (2 * kMaxStages + 5) + 64 + sizeof(Windows);
    const size_t slab = kKeyStageBytes + (p.q_resident ? 0 : op_slab);
    if (p.tsub > 1) {
        // narrow rows: the whole tile is one group; wide rows (operand not resident): one slab index per group
        p.gs = dslabs <= 2 ? dslabs : 1;
        const size_t group = (size_t)p.gs * (p.tsub * kKeyStageBytes + (p.q_resident ? 0 : op_slab));
        long long s = ((long long)227 * 1024 - (long long)fixed) / (long long)group;
        p.stages = (int)(s > kMaxStages ? kMaxStages : s);
        p.smem = fixed + (size_t)(p.stages > 0 ? p.stages : 0) * group;
        return p;
    } else {
        // Largest slab group (fewest barrier round trips per tile) that still leaves
        // at least three groups in flight.
        for (int gs = 4; gs >= 1; --gs) {
            if (gs > dslabs && gs > 1) continue;          // three-slab rows: one group of three per tile
            long long s = ((long long)227 * 1024 - (long long)fixed) / (long long)(gs * slab);
            if (s > kMaxStages) s = kMaxStages;
            p.gs = gs;
            p.stages = (int)s;
            if (s >= 3) break;
        }
    }
    p.smem = fixed + (size_t)(p.stages > 0 ? p.stages : 0) * p.gs * slab;
    return p;
}

// One accumulator column per query: for more than 32 queries on rows of at most 64 elements (one
// slab), where the epilogue -- the compares per key and query -- sets the pace.  Measured on 3 GB
// fp16 stores, two columns -> one column per query: d = 64, 64 queries 0.90 -> 0.68 ms; d = 32,
// 64 queries 1.72 -> 1.04.  With 17-32 queries the two-column form (hi block | lo block, one
// instruction per K-step instead of two) is the faster one since its rejection test went to packed
// arithmetic: d = 64, 17 / 24 / 32 queries 0.61 / 0.65 / 0.66 -> 0.54 / 0.58 / 0.58 ms, 46.3M rows at
// 32 queries 1.24 -> 1.05; d = 48 0.80 -> 0.70; d = 32 0.88 -> 0.85 (interleaved A/B).  From two slabs
// per row on, twice the instructions cost more than half the columns save (d = 128, 64 queries:
// 0.58 against 0.64 ms; d = 512: 0.73 against 0.93).
bool scan_umma_merged_eligible(int d, int B, int dtype)
{
    return dtype != kE4M3 && B > 32 && d <= kSlabElems;
}

int scan_umma_tile_rows(int d, int B, int keys_as_m, int merged)
{
    if (!keys_as_m && scan_ummat_eligible(d, B)) return 256;        // keys are the N = 256 operand there
    const int nq = umma_queries_padded(B);
    return kTileRows * umma_tsub_of(d, merged ? nq : 2 * nq);
}
int scan_umma_operand_rows(int B) { return 2 * umma_queries_padded(B); }

cudaError_t launch_scan_umma(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a_in, int grid,
                             cudaStream_t stream)
{
    if (!a_in.keys_as_m && a_in.dtype != kE4M3 && scan_ummat_eligible(a_in.d, a_in.B))
        return launch_scan_ummat(kmap, qmap, a_in, grid, stream);
    if (a_in.merged) return launch_scan_umma_merged(kmap, qmap, a_in, grid, stream);
    if (a_in.pack2 && a_in.dtype != kE4M3) return launch_scan_umma_pack16(kmap, qmap, a_in, grid, stream);
    ScanArgs a = a_in;
    if (a.tile_stride < 1) a.tile_stride = 1;
    const bool h = a.dtype == kF16, q8 = a.dtype == kE4M3;
    const bool pack2 = q8 && a.pack2;
    const UmmaPlan p = umma_make_plan(a.d, pack2 ? 2 * a.B : a.B, false);   // two operand-row pairs per query when packed
    if (p.stages < 2) return cudaErrorInvalidValue;
    a.stages = p.stages;
#define DRESD_GO(N_)                                                                          \
    if (pack2) return launch_tsub<E4M3Keys, N_, true>(kmap, qmap, a, p, grid, stream);        \
    return q8 ? launch_tsub<E4M3Keys, N_>(kmap, qmap, a, p, grid, stream)                     \
           : h ? launch_tsub<__half, N_>(kmap, qmap, a, p, grid, stream)                      \
               : launch_tsub<__nv_bfloat16, N_>(kmap, qmap, a, p, grid, stream)
    switch (p.ncols) {
    case 16: DRESD_GO(16);
    case 32: DRESD_GO(32);
    case 64: DRESD_GO(64);
    default: DRESD_GO(128);
    }
#undef DRESD_GO
}

}  // namespace dresd
