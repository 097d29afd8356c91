// The sixteen-elements-per-thread kernel for the paper's default configuration.
#include "solo_dispatch.h"
#include "solo_fast16.cuh"

namespace solo {

StepKernel fast16_kernel() { return solo_step_fast16_kernel; }
size_t fast16_kernel_smem() { return sizeof(Fast16Shared); }

}  // namespace solo
