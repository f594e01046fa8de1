// K2+K3 (tensor-core path, 16-bit keys): the forms of scan_umma_kernel with ONE accumulator
// column per query (see k23_scan_umma.cuh), for 17-64 queries.
#include "k23_scan_umma.cuh"
#include "k23_scan_umma_plan.h"

namespace dresd {
namespace {

template <typename T, int NCOLS, int TSUB>
cudaError_t launch_one(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                       int grid, cudaStream_t stream)
{
    if constexpr (2 * TSUB * NCOLS > 512) {
        return cudaErrorInvalidValue;
    } else {
        const int dslabs = (a.d + kSlabElems - 1) / kSlabElems;
        if constexpr (dual_possible(TSUB, NCOLS)) {
            // wide rows: the two issuing threads take alternate slabs (twice the instructions of the
            // two-column form, so a second issuer pays at every width that has more than one slab group)
            if (dslabs > 2) {
                auto kernel = scan_umma_kernel<T, NCOLS, TSUB, false, true, true>;
                cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
                if (e != cudaSuccess) return e;
                return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, true, true)), p.smem, stream, kmap, qmap, a,
                                        p.q_resident, p.gs);
            }
        }
        if constexpr (NCOLS == 64 && TSUB == 4) {
            // Sixteen epilogue warps (four per TMEM lane group, a quarter of the queries each) where the tile
            // has four sub-tiles: the epilogue is bound by latency, not by issue slots (the schedulers
            // issue 37 % of the time with eight), and twice the warps hide more of it.  Interleaved A/B,
            // 3 GB fp16 stores, 8 -> 16 warps: d = 64, 64 queries 0.778 -> 0.746 ms, with n = 32
            // 0.916 -> 0.807, 40 queries 0.734 -> 0.692; d = 32 1.132 -> 1.096.
            if (a.epi_warps != 8) {
                auto kernel = scan_umma_kernel<T, NCOLS, TSUB, false, false, true, false, 16>;
                cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
                if (e != cudaSuccess) return e;
                return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, false, true, 16)), p.smem, stream, kmap,
                                        qmap, a, p.q_resident, p.gs);
            }
        }
        auto kernel = scan_umma_kernel<T, NCOLS, TSUB, false, false, true>;
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
        if (e != cudaSuccess) return e;
        return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, false, true)), p.smem, stream, kmap, qmap, a,
                                p.q_resident, p.gs);
    }
}

template <typename T, int NCOLS>
cudaError_t launch_tsub(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                        int grid, cudaStream_t stream)
{
    switch (p.tsub) {
    case 4: return launch_one<T, NCOLS, 4>(kmap, qmap, a, p, grid, stream);
    case 2: return launch_one<T, NCOLS, 2>(kmap, qmap, a, p, grid, stream);
    default: return launch_one<T, NCOLS, 1>(kmap, qmap, a, p, grid, stream);
    }
}

}  // namespace

cudaError_t launch_scan_umma_merged(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a_in, int grid,
                                    cudaStream_t stream)
{
    ScanArgs a = a_in;
    if (a.tile_stride < 1) a.tile_stride = 1;
    if (a.dtype != kF16 && a.dtype != kBF16) return cudaErrorInvalidValue;
    const UmmaPlan p = umma_make_plan(a.d, a.B, true);
    if (p.stages < 2) return cudaErrorInvalidValue;
    a.stages = p.stages;
    const bool h = a.dtype == kF16;
    switch (p.ncols) {
    case 32: return h ? launch_tsub<__half, 32>(kmap, qmap, a, p, grid, stream)
                      : launch_tsub<__nv_bfloat16, 32>(kmap, qmap, a, p, grid, stream);
    case 64: return h ? launch_tsub<__half, 64>(kmap, qmap, a, p, grid, stream)
                      : launch_tsub<__nv_bfloat16, 64>(kmap, qmap, a, p, grid, stream);
    default: return cudaErrorInvalidValue;      // up to 16 queries keep two columns per query
    }
}

}  // namespace dresd
