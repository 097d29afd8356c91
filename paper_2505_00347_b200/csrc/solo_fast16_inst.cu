// The sixteen-elements-per-thread kernels for one block size (SOLO_G = 4, 8, 16 lanes per block:
// blocks of 64, 128, 256 elements): 2/3/4-bit states, fp32 or bf16 parameters, with the modes of the
// step fixed at compile time (the paper's plain step) or read from the arguments.
#include "solo_dispatch.h"
#include "solo_fast16.cuh"

#ifndef SOLO_G
#error "compile with -DSOLO_G=4|8|16"
#endif

#define SOLO_CAT_(a, b) a##b
#define SOLO_CAT(a, b) SOLO_CAT_(a, b)

namespace solo {

#define SOLO_K16(BM, BV)                                                                                          \
    (plain ? (param_bf16 ? solo_step_fast16_kernel<BM, BV, true, SOLO_G, true> : solo_step_fast16_kernel<BM, BV, false, SOLO_G, true>) \
           : (param_bf16 ? solo_step_fast16_kernel<BM, BV, true, SOLO_G, false> : solo_step_fast16_kernel<BM, BV, false, SOLO_G, false>))
#define SOLO_S16(BM, BV) \
    (param_bf16 ? sizeof(Fast16Shared<BM, BV, true, SOLO_G>) : sizeof(Fast16Shared<BM, BV, false, SOLO_G>))

StepKernel SOLO_CAT(fast16_kernel_g, SOLO_G)(int bits_m, int bits_v, bool param_bf16, bool plain) {
    switch (bits_m * 10 + bits_v) {
        case 22: return SOLO_K16(2, 2);
        case 23: return SOLO_K16(2, 3);
        case 24: return SOLO_K16(2, 4);
        case 32: return SOLO_K16(3, 2);
        case 33: return SOLO_K16(3, 3);
        case 34: return SOLO_K16(3, 4);
        case 42: return SOLO_K16(4, 2);
        case 43: return SOLO_K16(4, 3);
        case 44: return SOLO_K16(4, 4);
        default: return nullptr;
    }
}

size_t SOLO_CAT(fast16_smem_g, SOLO_G)(int bits_m, int bits_v, bool param_bf16) {
    switch (bits_m * 10 + bits_v) {
        case 22: return SOLO_S16(2, 2);
        case 23: return SOLO_S16(2, 3);
        case 24: return SOLO_S16(2, 4);
        case 32: return SOLO_S16(3, 2);
        case 33: return SOLO_S16(3, 3);
        case 34: return SOLO_S16(3, 4);
        case 42: return SOLO_S16(4, 2);
        case 43: return SOLO_S16(4, 3);
        case 44: return SOLO_S16(4, 4);
        default: return 0;
    }
}

}  // namespace solo
