// Kernel lookup by (bits_m, bits_v, block kind).  The step kernel is instantiated
// once per first-moment width in its own translation unit (solo_step_inst.cu compiled
// with -DSOLO_BM=2,3,4,8) so that the instantiations build in parallel.
#pragma once
#include <cuda_runtime.h>

#include "solo_device.cuh"

namespace solo {

using StepKernel = void (*)(const StepArgs);

// Per-translation-unit tables: index [bv_index][cta_group], bv_index 0..3 for 2,3,4,8 bits.
StepKernel step_kernel_bm2(int bv_index, bool cta_group);
StepKernel step_kernel_bm3(int bv_index, bool cta_group);
StepKernel step_kernel_bm4(int bv_index, bool cta_group);
StepKernel step_kernel_bm8(int bv_index, bool cta_group);

inline int bits_index(int bits) {
    switch (bits) {
        case 2: return 0;
        case 3: return 1;
        case 4: return 2;
        case 8: return 3;
        default: return -1;
    }
}

StepKernel step_kernel(int bits_m, int bits_v, bool cta_group);

// Streamlined kernel (2/3/4/8-bit states, block 64, 128, 256 or 2048, fp32 or bf16 parameters); null
// outside that domain.  The caller additionally requires the logarithmic second-moment
// quantizer, nearest rounding of the first moment and eps >= 1e-12.
// `plain`: no L2 term in the gradient, no AdaBelief, base from the quantile, xi drawn (the
// paper's step as it stands); that instantiation carries no code for the other modes.
StepKernel fast_kernel_bm2(int bv_index, int block, bool param_bf16, bool plain);
StepKernel fast_kernel_bm3(int bv_index, int block, bool param_bf16, bool plain);
StepKernel fast_kernel_bm4(int bv_index, int block, bool param_bf16, bool plain);
StepKernel fast_kernel_bm8(int bv_index, int block, bool param_bf16, bool plain);
StepKernel fast_kernel(int bits_m, int bits_v, int block, bool param_bf16, bool plain);
// Sixteen elements per thread: 2/3/4-bit states, blocks of 64, 128 or 256, fp32 or bf16 parameters, the
// quantile rank of p = 0.1 or no quantile (fixed base, baseline codebook); `modes`: 0 as `plain` for
// fast_kernel, 1 the modes fast_kernel reads at run time, 2 those plus Eq. 5 rounding and the baseline
// second-moment codebooks; full tiles
// of aligned tensors only (the rest is left to a launch of the streamlined or of the general kernel with
// StepArgs::only_partial).  Launched with CTA16 = 128 threads.
// Null / 0 for other widths and block sizes.  One translation unit per block size and set of modes.
constexpr int CTA16 = 128;         // threads per CTA of that kernel
StepKernel fast16_kernel_g4_m0(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g4_m1(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g4_m2(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g8_m0(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g8_m1(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g8_m2(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g16_m0(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g16_m1(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel_g16_m2(int bits_m, int bits_v, bool param_bf16);
size_t fast16_smem_g4(int bits_m, int bits_v, bool param_bf16);
size_t fast16_smem_g8(int bits_m, int bits_v, bool param_bf16);
size_t fast16_smem_g16(int bits_m, int bits_v, bool param_bf16);
StepKernel fast16_kernel(int bits_m, int bits_v, int block, bool param_bf16, int modes);
size_t fast16_kernel_smem(int bits_m, int bits_v, int block, bool param_bf16);
// Dynamic shared memory the streamlined kernel for these widths is launched with.
size_t fast_kernel_smem(int bits_m, int bits_v);
// Resident CTAs per SM of a step kernel launched with `dyn_smem` bytes of dynamic shared memory
// (cached per device and kernel; opts the kernel in to that much shared memory), 0 on error.
int kernel_occupancy(StepKernel k, size_t dyn_smem, int threads = CTA);

// Exhaustive comparison of the hardware lg2 approximation with log2_sp (tests).
cudaError_t launch_fast_log_check(uint32_t lo, uint32_t hi, float* out_max_excess, cudaStream_t stream);
float fast_log_abs_bound();

cudaError_t launch_dequant(int bits, const DequantArgs& a, unsigned grid, cudaStream_t stream);

}  // namespace solo
