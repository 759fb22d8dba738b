// Warp-level butterfly reduce-scatter of a per-lane register array.
#pragma once
#include <cuda_runtime.h>

namespace molora {

// Sums v[0..NV) element-wise over the 32 lanes of a warp.  While more than one value is left, each
// step halves the array: a lane keeps the half selected by one bit of its lane index and receives
// the partner's copy of that half, so NV-1 shuffles (not 5*NV) do the whole reduction.
//   NV >= 32: on return lane L holds the NV/32 finished sums of indices reduce_scatter_base<NV>(L) + j
//             in v[0 .. NV/32).
//   NV <  32: the last log2(32/NV) steps are plain xor-adds; lanes L with L % (32/NV) == 0 (and their
//             neighbours) hold the one finished sum of index reduce_scatter_base<NV>(L) in v[0].
// Every index expression is a compile-time constant after unrolling, so v stays in registers.
template <int NV, int OFF>
struct ReduceScatterStep {
    static __device__ __forceinline__ void run(float* v, int lane)
    {
        if constexpr (NV >= 2) {
            constexpr int H = NV / 2;
            const bool upper = (lane & OFF) != 0;
#pragma unroll
            for (int i = 0; i < H; ++i) {
                const float send = upper ? v[i] : v[i + H];
                const float keep = upper ? v[i + H] : v[i];
                v[i] = keep + __shfl_xor_sync(0xFFFFFFFFu, send, OFF);
            }
            if constexpr (OFF > 1) ReduceScatterStep<H, OFF / 2>::run(v, lane);
        } else {
            v[0] += __shfl_xor_sync(0xFFFFFFFFu, v[0], OFF);
            if constexpr (OFF > 1) ReduceScatterStep<1, OFF / 2>::run(v, lane);
        }
    }
};

template <int NV>
__device__ __forceinline__ void warp_reduce_scatter(float* v, int lane)
{
    static_assert(NV >= 1 && (NV & (NV - 1)) == 0, "NV must be a power of two");
    ReduceScatterStep<NV, 16>::run(v, lane);
}

// First index of the sums lane `lane` holds after warp_reduce_scatter<NV>.
template <int NV>
__device__ __forceinline__ int reduce_scatter_base(int lane)
{
    int base = 0, n = NV;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        if (n >= 2) {
            n >>= 1;
            if (lane & off) base += n;
        }
    }
    return base;
}

}  // namespace molora
