// Token-to-adapter grouping (Section 3.3 steps 1-3, Algorithm 2): histogram of r, exclusive scan into
// segment offsets, STABLE permutation.  The paper allocates positions with atomicAdd, which leaves the
// order inside a group to the hardware; here every position is computed from warp ballots/matches and
// prefix sums only, so counts, offsets and perm are unique and bit-reproducible.
//
// One launch: a thread-block cluster of S <= 8 CTAs (1024 threads each) splits the tokens into S * 32
// contiguous warp ranges, so "CTA rank, then warp, then iteration, then lane" is ascending token order.
//   1. hist[w][c]  = tokens of adapter c in warp w's range (equal adapters of a 32-token step are grouped
//                    by ballot / match; the lowest lane of a group adds its size -- distinct addresses,
//                    no atomics)
//   2. hist[w][c] <- exclusive prefix over the CTA's warps; tot[c] = the CTA's histogram
//   3. hardware cluster barrier; every CTA reads all S histograms through distributed shared memory:
//      counts[c] = their sum, lower[c] = sum over lower-ranked CTAs, seg[c] = exclusive prefix of counts
//   4. second walk: position = seg[c] + lower[c] + hist[w][c] + (rank of the lane inside its group);
//      the group leader then advances hist[w][c].
// A final cluster barrier keeps every CTA's shared memory alive until all peers have read it.
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kGroupThreads = 1024;
constexpr int kGroupWarps = kGroupThreads / 32;
constexpr int kGroupMaxCluster = 8;
constexpr int kGroupCached = 4;      // 32-token steps of a warp kept in registers

__global__ void __launch_bounds__(kGroupThreads) group_cluster_kernel(const int32_t* __restrict__ r, int64_t N, int C,
                                                                     int32_t* __restrict__ counts,
                                                                     int32_t* __restrict__ offsets,
                                                                     int32_t* __restrict__ perm, uint32_t* dev_status)
{
    __shared__ int hist[kGroupWarps][MOLORA_MAX_ADAPTERS];
    __shared__ int tot_all[kGroupMaxCluster][MOLORA_MAX_ADAPTERS];   // every CTA's histogram, pushed by its owner
    __shared__ int seg[MOLORA_MAX_ADAPTERS + 1];      // global exclusive prefix of counts
    __shared__ int lower[MOLORA_MAX_ADAPTERS];        // tokens of adapter c in lower-ranked CTAs
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const unsigned lt_mask = (1u << lane) - 1u;
    const uint32_t S = cluster_nctarank(), crank = cluster_ctarank();

    const int64_t chunk = ceil_div64(ceil_div64(N, (int64_t)S * kGroupWarps), 32) * 32;
    const int64_t begin0 = ((int64_t)crank * kGroupWarps + warp) * chunk;
    const int64_t begin = begin0 < N ? begin0 : N;
    const int64_t end = begin + chunk < N ? begin + chunk : N;

    if (S > 1) cluster_arrive_relaxed();   // "I am running"; waited for before the first write to a peer
    for (int c = lane; c < C; c += 32) hist[warp][c] = 0;
    __syncwarp();
    ptx::grid_dependency_sync();   // r is the router's output

    // the first kGroupCached steps of the warp's tokens stay in registers for both passes (all loads in flight at once)
    int vreg[kGroupCached];
#pragma unroll
    for (int j = 0; j < kGroupCached; ++j) {
        const int64_t i = begin + j * 32 + lane;
        vreg[j] = i < end ? __ldg(r + i) : -1;
    }
    auto route_of = [&](int64_t i0) {
        const int64_t j = (i0 - begin) >> 5;
        int v = -1;
        if (j < kGroupCached) {
#pragma unroll
            for (int jj = 0; jj < kGroupCached; ++jj)
                if (jj == j) v = vreg[jj];
        } else {
            const int64_t i = i0 + lane;
            v = i < end ? __ldg(r + i) : -1;
        }
        return v;
    };

    bool bad = false;
    for (int64_t i0 = begin; i0 < end; i0 += 32) {
        const int v = route_of(i0);
        const bool routed = v >= 0 && v < C;
        bad |= (v < -1) || (v >= C);
        const unsigned peers = peers_of(v, routed, C);
        if (routed && lane == __ffs(peers) - 1) hist[warp][v] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();

    // exclusive prefix over this CTA's warps, per adapter; the totals are the CTA's histogram
    for (int c = threadIdx.x; c < C; c += kGroupThreads) {
        int run = 0;
#pragma unroll 8
        for (int w = 0; w < kGroupWarps; ++w) {
            const int t = hist[w][c];
            hist[w][c] = run;
            run += t;
        }
        if (S == 1) tot_all[0][c] = run;
        else tot_all[crank][c] = run;      // published to the peers below
    }
    if (S > 1) {
        // push my histogram into every peer's table; one cluster barrier makes all tables complete and visible.
        // Nothing is read from a peer afterwards, so the CTAs retire independently.
        __syncthreads();
        cluster_wait();                    // every peer is running
        for (int c = threadIdx.x; c < C; c += kGroupThreads) {
            const int mine = tot_all[crank][c];
            for (uint32_t q = 0; q < S; ++q)
                if (q != crank)
                    asm volatile("st.shared::cluster.s32 [%0], %1;" ::"r"(map_to_cta(smem_u32(&tot_all[crank][c]), q)), "r"(mine) : "memory");
        }
        cluster_sync_all();
    } else {
        __syncthreads();
    }

    // global histogram and the part that precedes this CTA
    for (int c = threadIdx.x; c < C; c += kGroupThreads) {
        int all = 0, low = 0;
        for (uint32_t q = 0; q < S; ++q) {
            const int t = tot_all[q][c];
            all += t;
            if (q < crank) low += t;
        }
        lower[c] = low;
        seg[c + 1] = all;      // shifted by one: turned into the prefix below
        if (crank == 0) counts[c] = all;
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
    if (crank == 0)
        for (int c = threadIdx.x; c <= C; c += kGroupThreads) offsets[c] = seg[c];

    // stable scatter
    for (int64_t i0 = begin; i0 < end; i0 += 32) {
        const int64_t i = i0 + lane;
        const int v = route_of(i0);
        const bool routed = v >= 0 && v < C;
        const unsigned peers = peers_of(v, routed, C);
        if (routed) {
            const int pos = seg[v] + lower[v] + hist[warp][v] + __popc(peers & lt_mask);
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
    // one CTA per ~1024 tokens (one 32-token step per warp), at most 8 CTAs
    int split = 1;
    while (split < kGroupMaxCluster && (int64_t)split * 1024 < N) split *= 2;
    if (const int64_t forced = tune(kTuneGroupSplit)) split = (int)std::max<int64_t>(1, std::min<int64_t>(forced, kGroupMaxCluster));
    return cuda_ok(launch_kernel(group_cluster_kernel, dim3((unsigned)split), dim3(kGroupThreads), 0, s, (unsigned)split, false,
                                  r, N, C, counts, offsets, perm, dev_status));
}

}  // namespace molora
