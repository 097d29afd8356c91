// The sixteen-elements-per-thread kernels: 2-bit first moment, 2/3/4-bit second moment, block 128,
// fp32 or bf16 parameters, plain step.  (With wider first moments the nearest-level search over
// sixteen elements costs more than the shared per-thread work saves: measured slower than the
// eight-per-thread kernel, so those widths are not instantiated.)
#include "solo_dispatch.h"
#include "solo_fast16.cuh"

namespace solo {

StepKernel fast16_kernel(int bits_m, int bits_v, bool param_bf16) {
    if (bits_m != 2) return nullptr;
    switch (bits_v) {
        case 2: return param_bf16 ? solo_step_fast16_kernel<2, 2, true> : solo_step_fast16_kernel<2, 2, false>;
        case 3: return param_bf16 ? solo_step_fast16_kernel<2, 3, true> : solo_step_fast16_kernel<2, 3, false>;
        case 4: return param_bf16 ? solo_step_fast16_kernel<2, 4, true> : solo_step_fast16_kernel<2, 4, false>;
        default: return nullptr;
    }
}

size_t fast16_kernel_smem(int bits_m, int bits_v) {
    if (bits_m != 2) return 0;
    switch (bits_v) {
        case 2: return sizeof(Fast16Shared<2, 2>);
        case 3: return sizeof(Fast16Shared<2, 3>);
        case 4: return sizeof(Fast16Shared<2, 4>);
        default: return 0;
    }
}

}  // namespace solo
