// Section 3.3 steps 1-3 (histogram, exclusive scan, stable permutation) done by ONE CTA in its own shared memory, for
// kernels that start from the routing decisions r instead of offsets / perm: every CTA of such a kernel runs this
// before its first copy request, which replaces the table load and saves the grouping launch.  At most MAXN tokens.
// Results: offs_s[0..C], perm_s[0..offs_s[C]); with write_out the CTAs also write counts, offsets and perm to global
// memory (CTA 0 the two small arrays, every CTA a slice of perm), bit-equal to what molora_group writes.
//   scratch   shared memory that is idle at this point: max(kGroupInCtaTableMaxC * NT * 4 + 4 * kGroupInCtaTableMaxC,
//             NT / 32 * MOLORA_MAX_ADAPTERS * 4) bytes
//   tstart_s  MOLORA_MAX_ADAPTERS ints of temporary storage (the caller's tile prefix, filled afterwards)
// Ends with a block-wide barrier.  All NT threads of the CTA must call it.
#pragma once
#include "common.cuh"

namespace molora {

constexpr int kGroupInCtaTableMaxC = 32;       // adapters handled by the per-thread count table (ballots / match above)

template <int NT, int MAXN>
__device__ __forceinline__ void group_in_cta(const int32_t* __restrict__ r, int N_, int C_, int32_t* offs_s, int32_t* tstart_s,
                                             int32_t* perm_s, unsigned char* scratch, bool write_out, int32_t* counts_out,
                                             int32_t* offsets_out, int32_t* perm_out, uint32_t* dev_status)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
        constexpr int NW = NT / 32;
      if (C_ <= kGroupInCtaTableMaxC) {
        // Up to 32 adapters: every thread owns a contiguous run of tokens and counts it into its own column of a
        // [adapter][thread] table in shared memory (consecutive threads hit consecutive banks); a warp
        // per adapter turns the table into exclusive prefixes over the threads, and every thread then writes its run
        // out in token order -- stable by construction, no atomics.
        constexpr int TPT = (MAXN + NT - 1) / NT;      // tokens per thread
        constexpr int LPT = NT / 32;                                   // table entries per lane in the scan
        int* cnt_s = reinterpret_cast<int*>(scratch);                              // [C][NT]
        int* tot_s = cnt_s + kGroupInCtaTableMaxC * NT;                    // [C] adapter totals
        const int C = C_, N = N_;
        const int per = (N + NT - 1) / NT;
        const int b0 = min(tid * per, N), e0 = min(b0 + per, N);
        int v[TPT];
        bool bad = false;
#pragma unroll
        for (int j = 0; j < TPT; ++j) {
            const int raw = b0 + j < e0 ? __ldg(r + b0 + j) : -1;
            bad |= (raw < -1) || (raw >= C);
            v[j] = (raw >= 0 && raw < C) ? raw : -1;
        }
        for (int c = 0; c < C; ++c) cnt_s[c * NT + tid] = 0;
#pragma unroll
        for (int j = 0; j < TPT; ++j)
            if (v[j] >= 0) cnt_s[v[j] * NT + tid] += 1;
        __syncthreads();
        for (int c = warp; c < C; c += NW) {           // exclusive prefix over the threads, lane = LPT consecutive threads
            int* row = cnt_s + c * NT + lane * LPT;
            int loc[LPT], sum = 0;
#pragma unroll
            for (int k = 0; k < LPT; ++k) {
                loc[k] = row[k];
                sum += loc[k];
            }
            int incl = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            int run = incl - sum;
#pragma unroll
            for (int k = 0; k < LPT; ++k) {
                row[k] = run;
                run += loc[k];
            }
            if (lane == 31) tot_s[c] = incl;
        }
        __syncthreads();
        if (warp == 0) {                               // offsets: exclusive prefix of the totals (C <= 32: one per lane)
            const int mine = lane < C ? tot_s[lane] : 0;
            int incl = mine;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            if (lane < C) offs_s[lane] = incl - mine;
            if (lane == C - 1) offs_s[C] = incl;
            if ((write_out && blockIdx.x == 0) && lane < C) counts_out[lane] = mine;
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < TPT; ++j)
            if (v[j] >= 0) {
                int* slot = cnt_s + v[j] * NT + tid;
                const int k = *slot;
                *slot = k + 1;
                perm_s[offs_s[v[j]] + k] = b0 + j;
            }
        if ((write_out && blockIdx.x == 0) && dev_status != nullptr && __any_sync(0xFFFFFFFFu, bad) && lane == 0)
            atomicOr(dev_status, MOLORA_DEV_BAD_ROUTE);
        __syncthreads();
        if ((write_out && blockIdx.x == 0))
            for (int c = tid; c <= C; c += NT) offsets_out[c] = offs_s[c];
      } else {
        constexpr int STEPS = (MAXN + NW * 32 - 1) / (NW * 32);      // 32-token steps of a warp
        int(*hist)[MOLORA_MAX_ADAPTERS] = reinterpret_cast<int(*)[MOLORA_MAX_ADAPTERS]>(scratch);   // [warp][adapter]
        const int C = C_, N = N_;
        const unsigned lt_mask = (1u << lane) - 1u;
        const int chunk = ((N + NW - 1) / NW + 31) / 32 * 32;                // tokens of a warp: ascending token order
        const int begin = min(warp * chunk, N), end = min(begin + chunk, N);
        int vreg[STEPS];
#pragma unroll
        for (int j = 0; j < STEPS; ++j) {
            const int i = begin + j * 32 + lane;
            vreg[j] = i < end ? __ldg(r + i) : -1;
        }
        for (int c = lane; c < C; c += 32) hist[warp][c] = 0;
        __syncwarp();
        bool bad = false;
#pragma unroll
        for (int j = 0; j < STEPS; ++j) {
            if (begin + j * 32 < end) {
                const int v = vreg[j];
                const bool routed = v >= 0 && v < C;
                bad |= (v < -1) || (v >= C);
                const unsigned peers = peers_of(v, routed, C);
                if (routed && lane == __ffs(peers) - 1) hist[warp][v] += __popc(peers);
                __syncwarp();
            }
        }
        __syncthreads();
        // exclusive prefix over the warps, per adapter; the totals are the histogram
        for (int c = tid; c < C; c += NT) {
            int run = 0;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const int t = hist[w][c];
                hist[w][c] = run;
                run += t;
            }
            tstart_s[c] = run;                 // counts, until the tile prefix replaces them below
        }
        __syncthreads();
        if (warp == 0) {                       // exclusive prefix over adapters, eight consecutive adapters per lane
            int local[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = lane * 8 + j;
                local[j] = c < C ? tstart_s[c] : 0;
                sum += local[j];
            }
            if ((write_out && blockIdx.x == 0)) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (lane * 8 + j < C) counts_out[lane * 8 + j] = local[j];
            }
            int incl = sum;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
                if (lane >= off) incl += up;
            }
            int run = incl - sum;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int c = lane * 8 + j;
                if (c <= C) offs_s[c] = run;
                run += local[j];
            }
            if (lane == 31 && C == MOLORA_MAX_ADAPTERS) offs_s[MOLORA_MAX_ADAPTERS] = run;
        }
        __syncthreads();
        // stable scatter into the CTA's copy of perm
#pragma unroll
        for (int j = 0; j < STEPS; ++j) {
            if (begin + j * 32 < end) {
                const int v = vreg[j];
                const bool routed = v >= 0 && v < C;
                const unsigned peers = peers_of(v, routed, C);
                if (routed) perm_s[offs_s[v] + hist[warp][v] + __popc(peers & lt_mask)] = begin + j * 32 + lane;
                __syncwarp();
                if (routed && lane == __ffs(peers) - 1) hist[warp][v] += __popc(peers);
                __syncwarp();
            }
        }
        if ((write_out && blockIdx.x == 0)) {
            for (int c = tid; c <= C; c += NT) offsets_out[c] = offs_s[c];
            if (dev_status != nullptr && __any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(dev_status, MOLORA_DEV_BAD_ROUTE);
        }
        __syncthreads();
      }
        if (write_out) {   // my slice of perm
            const int C = C_;
            const int total = offs_s[C];
            const int per = (total + (int)gridDim.x - 1) / (int)gridDim.x;
            const int lo = (int)blockIdx.x * per, hi = min(lo + per, total);
            for (int i = lo + tid; i < hi; i += NT) perm_out[i] = perm_s[i];
        }
}

}  // namespace molora
