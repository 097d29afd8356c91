// Instantiations of the fused step kernel for one first-moment width (SOLO_BM).
#include "solo_dispatch.h"

#ifndef SOLO_BM
#error "compile with -DSOLO_BM=2|3|4|8"
#endif

#define SOLO_CAT_(a, b) a##b
#define SOLO_CAT(a, b) SOLO_CAT_(a, b)

namespace solo {

StepKernel SOLO_CAT(step_kernel_bm, SOLO_BM)(int bv_index, bool cta_group) {
    static const StepKernel table[4][2] = {
        {solo_step_kernel<SOLO_BM, 2, false>, solo_step_kernel<SOLO_BM, 2, true>},
        {solo_step_kernel<SOLO_BM, 3, false>, solo_step_kernel<SOLO_BM, 3, true>},
        {solo_step_kernel<SOLO_BM, 4, false>, solo_step_kernel<SOLO_BM, 4, true>},
        {solo_step_kernel<SOLO_BM, 8, false>, solo_step_kernel<SOLO_BM, 8, true>},
    };
    if (bv_index < 0 || bv_index > 3) return nullptr;
    return table[bv_index][cta_group ? 1 : 0];
}

}  // namespace solo
