// Launch plan of the tcgen05 scan kernel (keys as the M operand), shared by the files that
// instantiate its forms.
#pragma once
#include <cstddef>

namespace dresd {

struct UmmaPlan {
    int ncols, tsub, stages, q_resident, gs;
    size_t smem;
};
int umma_queries_padded(int B);                 // 8, 16, 32 or 64
int umma_tsub_of(int d, int ncols);             // 128-row sub-tiles per tile
bool umma_dual_pays(int dslabs, int ncols);     // two MMA-issuing threads on alternate slabs
UmmaPlan umma_make_plan(int d, int B, bool merged);

}  // namespace dresd
