// Token-to-adapter grouping (Section 3.3 steps 1-3, Algorithm 2): histogram of r, exclusive scan into
// segment offsets, STABLE permutation.  The paper allocates positions with atomicAdd, which leaves the
// order inside a group to the hardware; here every position is computed from warp ballots/matches and
// prefix sums only, so counts, offsets and perm are unique and bit-reproducible.
#include "common.cuh"

namespace molora {

constexpr int kGroupThreads = 1024;
constexpr int kGroupWarps = kGroupThreads / 32;

// One CTA, three phases in shared memory.  Warp w owns the contiguous token range
// [w*chunk, (w+1)*chunk) and walks it 32 tokens at a time, so "warp index, then iteration, then lane"
// is ascending token order:
//   1. hist[w][c]  = tokens of adapter c in warp w's range (match_any groups equal adapters in a step;
//                    the lowest lane of each group adds the group's size -- distinct addresses, no atomics)
//   2. hist[w][c] <- exclusive prefix over w;  seg[c] = exclusive prefix of the totals over c
//   3. second walk: position = seg[c] + hist[w][c] + (rank of the lane inside its match group);
//      the group leader then advances hist[w][c] by the group's size.
__global__ void __launch_bounds__(kGroupThreads) group_single_cta_kernel(const int32_t* __restrict__ r, int64_t N,
                                                                         int C, int32_t* __restrict__ counts,
                                                                         int32_t* __restrict__ offsets,
                                                                         int32_t* __restrict__ perm,
                                                                         uint32_t* dev_status)
{
    __shared__ int hist[kGroupWarps][MOLORA_MAX_ADAPTERS];
    __shared__ int seg[MOLORA_MAX_ADAPTERS + 1];
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const unsigned lt_mask = (1u << lane) - 1u;

    const int64_t chunk = ceil_div64(ceil_div64(N, kGroupWarps), 32) * 32;
    const int64_t begin = (int64_t)warp * chunk;
    const int64_t end = begin + chunk < N ? begin + chunk : N;

    for (int c = lane; c < C; c += 32) hist[warp][c] = 0;
    __syncwarp();

    bool bad = false;
    for (int64_t i0 = begin; i0 < end; i0 += 32) {
        const int64_t i = i0 + lane;
        const int v = i < end ? __ldg(r + i) : -1;
        const bool routed = v >= 0 && v < C;
        bad |= (v < -1) || (v >= C);
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, routed ? v : -1);
        if (routed && lane == __ffs(peers) - 1) hist[warp][v] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();

    // exclusive prefix over warps, per adapter; totals are the histogram
    for (int c = threadIdx.x; c < C; c += kGroupThreads) {
        int run = 0;
#pragma unroll 8
        for (int w = 0; w < kGroupWarps; ++w) {
            const int t = hist[w][c];
            hist[w][c] = run;
            run += t;
        }
        counts[c] = run;
        seg[c + 1] = run;   // shifted by one: turned into the inclusive prefix below
    }
    __syncthreads();

    // exclusive prefix over adapters (C <= 256): warp 0, eight consecutive adapters per lane
    if (warp == 0) {
        int local[8];
        int sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = lane * 8 + j;
            local[j] = c < C ? seg[c + 1] : 0;
            sum += local[j];
        }
        int incl = sum;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        int run = incl - sum;   // exclusive prefix of this lane's first adapter
        if (lane == 0) seg[0] = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int c = lane * 8 + j;
            run += local[j];
            if (c < C) seg[c + 1] = run;
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c <= C; c += kGroupThreads) offsets[c] = seg[c];

    // stable scatter
    for (int64_t i0 = begin; i0 < end; i0 += 32) {
        const int64_t i = i0 + lane;
        const int v = i < end ? __ldg(r + i) : -1;
        const bool routed = v >= 0 && v < C;
        const unsigned peers = __match_any_sync(0xFFFFFFFFu, routed ? v : -1);
        if (routed) {
            const int pos = seg[v] + hist[warp][v] + __popc(peers & lt_mask);
            perm[pos] = (int32_t)i;
        }
        __syncwarp();
        if (routed && lane == __ffs(peers) - 1) hist[warp][v] += __popc(peers);
        __syncwarp();
    }
    if (dev_status != nullptr && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(dev_status, MOLORA_DEV_BAD_ROUTE);
}

size_t group_workspace_bytes(int64_t /*N*/, int32_t /*C*/) { return 0; }

molora_status_t launch_group(const int32_t* r, int64_t N, int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm,
                             void* /*ws*/, size_t /*ws_bytes*/, uint32_t* dev_status, cudaStream_t s)
{
    group_single_cta_kernel<<<1, kGroupThreads, 0, s>>>(r, N, C, counts, offsets, perm, dev_status);
    return cuda_ok(cudaGetLastError());
}

}  // namespace molora
