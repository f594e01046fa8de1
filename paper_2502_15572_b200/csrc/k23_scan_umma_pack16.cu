// K2+K3 (tensor-core path): 16-bit keys of 32 elements.  Such a key is 64 bytes -- half a 128-byte
// shared-memory row, so that half of every pipeline stage would be padding and too few bytes of
// real data in flight to cover the HBM latency (3.5 TB/s at any batch).  The store is therefore
// scanned as N/2 rows of TWO keys (the PACK2 forms of scan_umma_kernel, shared with the 8-bit
// copy of 64-element keys): query j owns the operand rows (hi|0), (lo|0), (0|hi), (0|lo), two
// column pairs that score the even and the odd key of a row.  The zero halves add exact zeros,
// so scores are bit-identical to the unpacked scan.
#include "k23_scan_umma.cuh"
#include "k23_scan_umma_plan.h"

namespace dresd {
namespace {

template <typename T, int NCOLS, int TSUB>
cudaError_t launch_one(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                       int grid, cudaStream_t stream)
{
    auto kernel = scan_umma_kernel<T, NCOLS, TSUB, true, false, false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(kernel, dim3(grid), dim3(threads_of(TSUB, false)), p.smem, stream, kmap, qmap, a,
                            p.q_resident, p.gs);
}

template <typename T>
cudaError_t launch_cols(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a, const UmmaPlan &p,
                        int grid, cudaStream_t stream)
{
    // one 64-element slab per row: four sub-tiles per tile, two with 128 accumulator columns
    if (p.ncols == 16 && p.tsub == 4) return launch_one<T, 16, 4>(kmap, qmap, a, p, grid, stream);
    if (p.ncols == 32 && p.tsub == 4) return launch_one<T, 32, 4>(kmap, qmap, a, p, grid, stream);
    if (p.ncols == 64 && p.tsub == 4) return launch_one<T, 64, 4>(kmap, qmap, a, p, grid, stream);
    if (p.ncols == 128 && p.tsub == 2) return launch_one<T, 128, 2>(kmap, qmap, a, p, grid, stream);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_scan_umma_pack16(const CUtensorMap &kmap, const CUtensorMap &qmap, const ScanArgs &a_in, int grid,
                                    cudaStream_t stream)
{
    ScanArgs a = a_in;
    if (a.tile_stride < 1) a.tile_stride = 1;
    if ((a.dtype != kF16 && a.dtype != kBF16) || a.d != kSlabElems || !a.pack2) return cudaErrorInvalidValue;
    const UmmaPlan p = umma_make_plan(a.d, 2 * a.B, false);     // two operand-row pairs per query
    if (p.stages < 2) return cudaErrorInvalidValue;
    a.stages = p.stages;
    return a.dtype == kF16 ? launch_cols<__half>(kmap, qmap, a, p, grid, stream)
                           : launch_cols<__nv_bfloat16>(kmap, qmap, a, p, grid, stream);
}

}  // namespace dresd
