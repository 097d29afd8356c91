// Instantiations of the streamlined step kernel for one first-moment width (SOLO_BM = 2, 3, 4, 8).
#include "solo_dispatch.h"
#include "solo_fast.cuh"

#ifndef SOLO_BM
#error "compile with -DSOLO_BM=2|3|4|8"
#endif

#define SOLO_CAT_(a, b) a##b
#define SOLO_CAT(a, b) SOLO_CAT_(a, b)

namespace solo {

#define SOLO_ROW(BV, PBF, PLAIN)                                                                            \
    {solo_step_fast_kernel<SOLO_BM, BV, 8, PBF, PLAIN>, solo_step_fast_kernel<SOLO_BM, BV, 16, PBF, PLAIN>, \
     solo_step_fast_kernel<SOLO_BM, BV, 32, PBF, PLAIN>, solo_step_fast_kernel<SOLO_BM, BV, 256, PBF, PLAIN>}
#define SOLO_PLANE(PBF, PLAIN) \
    {SOLO_ROW(2, PBF, PLAIN), SOLO_ROW(3, PBF, PLAIN), SOLO_ROW(4, PBF, PLAIN), SOLO_ROW(8, PBF, PLAIN)}

StepKernel SOLO_CAT(fast_kernel_bm, SOLO_BM)(int bv_index, int block, bool param_bf16, bool plain) {
    static const StepKernel table[2][2][4][4] = {
        {SOLO_PLANE(false, false), SOLO_PLANE(true, false)},
        {SOLO_PLANE(false, true), SOLO_PLANE(true, true)},
    };
    const int g = block == 64 ? 0 : block == 128 ? 1 : block == 256 ? 2 : block == 2048 ? 3 : -1;
    if (bv_index < 0 || bv_index > 3 || g < 0) return nullptr;
    return table[plain ? 1 : 0][param_bf16 ? 1 : 0][bv_index][g];
}

#if SOLO_BM == 2
// Exhaustive check of the error model used above: for every binary32 x with bit pattern
// in [lo, hi] (positive, finite) the largest value of
//   |lg2.approx(x) - log2_sp(x)| - (LG2_REL / 2) |log2_sp(x)|
// is written (as a maximum over the launch) to *out_max_excess, which starts at -1.
__global__ void fast_log_check_kernel(uint32_t lo, uint32_t hi, float* out_max_excess) {
    float worst = -1.0f;
    for (uint64_t b = (uint64_t)lo + blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; b <= hi;
         b += (uint64_t)gridDim.x * blockDim.x) {
        const float x = __uint_as_float((uint32_t)b);
        const float exact = log2_sp(x);
        const float ex = fabsf(lg2_approx(x) - exact) - (0.5f * LG2_REL) * fabsf(exact);
        worst = fmaxf(worst, ex);
    }
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, 16));
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, 8));
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, 4));
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, 2));
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, 1));
    if ((threadIdx.x & 31) == 0 && worst > 0.0f)
        atomicMax(reinterpret_cast<int*>(out_max_excess), __float_as_int(worst));
}

cudaError_t launch_fast_log_check(uint32_t lo, uint32_t hi, float* out_max_excess, cudaStream_t stream) {
    fast_log_check_kernel<<<148 * 8, 256, 0, stream>>>(lo, hi, out_max_excess);
    return cudaGetLastError();
}
float fast_log_abs_bound() { return LG2_ABS; }
size_t fast_kernel_smem(int bits_m, int bits_v) {
    const bool m8 = bits_m == 8, v8 = bits_v == 8;
    return m8 ? (v8 ? sizeof(FastSharedT<2, 2>) : sizeof(FastSharedT<2, 1>))
              : (v8 ? sizeof(FastSharedT<1, 2>) : sizeof(FastSharedT<1, 1>));
}
#endif

}  // namespace solo
