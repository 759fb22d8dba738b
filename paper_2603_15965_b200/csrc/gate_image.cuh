// Preparation kernel shared by the tensor-core routers: an fp32 weight matrix [d, C] (input-major) is split into three
// bf16 terms per value and written as the K-major operand images the tcgen05 kernels load by TMA.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "sm100_ptx.cuh"

namespace molora {

// Preparation: fp32 G [d, C] -> per 64-wide k chunk the image [3*CP][64] bf16 (row = term * CP + adapter).
template <int CP>
__global__ void __launch_bounds__(256) gate_umma_split_kernel(const float* __restrict__ G, int d, int C,
                                                              __nv_bfloat16* __restrict__ img)
{
    // An earlier gate call may still be reading the images this kernel rewrites: wait for it.  The gate kernel
    // that follows is launched programmatically: from here on it may run its set-up and its x loads, and it
    // waits only before it reads the images written here.
    ptx::grid_dependency_sync();
    const int64_t total = (int64_t)d * CP;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(e % CP);
        const int64_t k = e / CP;
        const float v = c < C ? __ldg(G + k * C + c) : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        const float r1 = v - __bfloat162float(hi);
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        __nv_bfloat16* base = img + (k / 64) * (3 * CP * 64) + (k % 64);
        base[(0 * CP + c) * 64] = hi;
        base[(1 * CP + c) * 64] = mid;
        base[(2 * CP + c) * 64] = lo;
    }
}

}  // namespace molora
