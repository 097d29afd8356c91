// Kernel lookup tables and the dequantization launcher.
#include "solo_dispatch.h"

#include <map>
#include <utility>
#include <mutex>

namespace solo {

StepKernel step_kernel(int bits_m, int bits_v, bool cta_group) {
    const int bv = bits_index(bits_v);
    switch (bits_m) {
        case 2: return step_kernel_bm2(bv, cta_group);
        case 3: return step_kernel_bm3(bv, cta_group);
        case 4: return step_kernel_bm4(bv, cta_group);
        case 8: return step_kernel_bm8(bv, cta_group);
        default: return nullptr;
    }
}

StepKernel fast_kernel(int bits_m, int bits_v, int block, bool param_bf16, bool plain) {
    const int bv = bits_index(bits_v);
    if (bv < 0) return nullptr;
    switch (bits_m) {
        case 2: return fast_kernel_bm2(bv, block, param_bf16, plain);
        case 3: return fast_kernel_bm3(bv, block, param_bf16, plain);
        case 4: return fast_kernel_bm4(bv, block, param_bf16, plain);
        case 8: return fast_kernel_bm8(bv, block, param_bf16, plain);
        default: return nullptr;
    }
}

StepKernel fast16_kernel(int bits_m, int bits_v, int block, bool param_bf16, int modes) {
#define SOLO_PICK16(G)                                                                   \
    (modes == 0 ? fast16_kernel_g##G##_m0(bits_m, bits_v, param_bf16)                    \
                : modes == 1 ? fast16_kernel_g##G##_m1(bits_m, bits_v, param_bf16)       \
                             : fast16_kernel_g##G##_m2(bits_m, bits_v, param_bf16))
    switch (block) {
        case 64: return SOLO_PICK16(4);
        case 128: return SOLO_PICK16(8);
        case 256: return SOLO_PICK16(16);   // twenty-five selection rounds
        default: return nullptr;
    }
#undef SOLO_PICK16
}

size_t fast16_kernel_smem(int bits_m, int bits_v, int block, bool param_bf16) {
    switch (block) {
        case 64: return fast16_smem_g4(bits_m, bits_v, param_bf16);
        case 128: return fast16_smem_g8(bits_m, bits_v, param_bf16);
        case 256: return fast16_smem_g16(bits_m, bits_v, param_bf16);
        default: return 0;
    }
}

int kernel_occupancy(StepKernel k, size_t dyn_smem, int threads) {
    static std::mutex mu;
    static std::map<std::pair<int, const void*>, int> cache;    // per device: the opt-in below is per context
    if (!k) return 0;
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    std::lock_guard<std::mutex> lk(mu);
    const auto key = std::make_pair(device, (const void*)k);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int n = 0;
    if ((dyn_smem > 0 &&
         cudaFuncSetAttribute((const void*)k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn_smem) != cudaSuccess) ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k, threads, dyn_smem) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return 0;
    }
    cache[key] = n;
    return n;
}

cudaError_t launch_dequant(int bits, const DequantArgs& a, unsigned grid, cudaStream_t stream) {
    switch (bits) {
        case 2: solo_dequant_kernel<2><<<grid, CTA, 0, stream>>>(a); break;
        case 3: solo_dequant_kernel<3><<<grid, CTA, 0, stream>>>(a); break;
        case 4: solo_dequant_kernel<4><<<grid, CTA, 0, stream>>>(a); break;
        case 8: solo_dequant_kernel<8><<<grid, CTA, 0, stream>>>(a); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace solo
