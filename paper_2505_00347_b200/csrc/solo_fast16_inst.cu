// The sixteen-elements-per-thread kernels for one block size (SOLO_G = 4, 8, 16 lanes per block:
// blocks of 64, 128, 256 elements) and one set of modes (SOLO_MODES = 0: the paper's plain step, fixed
// at compile time; 1, 2: read from the arguments, see solo_fast16.cuh): 2/3/4-bit states, fp32 or bf16
// parameters.
#include "solo_dispatch.h"
#include "solo_fast16.cuh"

#ifndef SOLO_G
#error "compile with -DSOLO_G=4|8|16"
#endif
#ifndef SOLO_MODES
#error "compile with -DSOLO_MODES=0|1|2"
#endif

#define SOLO_CAT_(a, b) a##b
#define SOLO_CAT(a, b) SOLO_CAT_(a, b)
#define SOLO_CAT4(a, b, c, d) SOLO_CAT(SOLO_CAT(a, b), SOLO_CAT(c, d))

namespace solo {

#define SOLO_K16(BM, BV) \
    (param_bf16 ? solo_step_fast16_kernel<BM, BV, true, SOLO_G, SOLO_MODES> : solo_step_fast16_kernel<BM, BV, false, SOLO_G, SOLO_MODES>)
#define SOLO_S16(BM, BV) \
    (param_bf16 ? sizeof(Fast16Shared<BM, BV, true, SOLO_G>) : sizeof(Fast16Shared<BM, BV, false, SOLO_G>))

StepKernel SOLO_CAT4(fast16_kernel_g, SOLO_G, _m, SOLO_MODES)(int bits_m, int bits_v, bool param_bf16) {
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

#if SOLO_MODES == 0
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
#endif

}  // namespace solo
