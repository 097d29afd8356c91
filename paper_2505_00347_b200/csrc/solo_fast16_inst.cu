// The sixteen-elements-per-thread kernels: 2/3/4-bit states except 4-bit / 4-bit (measured slower
// than the eight-per-thread kernel: 223 vs 236 Gparams/s), block 128, fp32 or bf16 parameters, plain
// step.
#include "solo_dispatch.h"
#include "solo_fast16.cuh"

namespace solo {

#define SOLO_K16(BM, BV) (param_bf16 ? solo_step_fast16_kernel<BM, BV, true> : solo_step_fast16_kernel<BM, BV, false>)

StepKernel fast16_kernel(int bits_m, int bits_v, bool param_bf16) {
    switch (bits_m * 10 + bits_v) {
        case 22: return SOLO_K16(2, 2);
        case 23: return SOLO_K16(2, 3);
        case 24: return SOLO_K16(2, 4);
        case 32: return SOLO_K16(3, 2);
        case 33: return SOLO_K16(3, 3);
        case 34: return SOLO_K16(3, 4);
        case 42: return SOLO_K16(4, 2);
        case 43: return SOLO_K16(4, 3);
        default: return nullptr;
    }
}

size_t fast16_kernel_smem(int bits_m, int bits_v, bool param_bf16) {
    switch (bits_m * 10 + bits_v) {
        case 22: return param_bf16 ? sizeof(Fast16Shared<2, 2, true>) : sizeof(Fast16Shared<2, 2, false>);
        case 23: return param_bf16 ? sizeof(Fast16Shared<2, 3, true>) : sizeof(Fast16Shared<2, 3, false>);
        case 24: return param_bf16 ? sizeof(Fast16Shared<2, 4, true>) : sizeof(Fast16Shared<2, 4, false>);
        case 32: return param_bf16 ? sizeof(Fast16Shared<3, 2, true>) : sizeof(Fast16Shared<3, 2, false>);
        case 33: return param_bf16 ? sizeof(Fast16Shared<3, 3, true>) : sizeof(Fast16Shared<3, 3, false>);
        case 34: return param_bf16 ? sizeof(Fast16Shared<3, 4, true>) : sizeof(Fast16Shared<3, 4, false>);
        case 42: return param_bf16 ? sizeof(Fast16Shared<4, 2, true>) : sizeof(Fast16Shared<4, 2, false>);
        case 43: return param_bf16 ? sizeof(Fast16Shared<4, 3, true>) : sizeof(Fast16Shared<4, 3, false>);
        default: return 0;
    }
}

}  // namespace solo
