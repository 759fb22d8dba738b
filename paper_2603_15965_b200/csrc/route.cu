// Routers: vocabulary-range routing (Definition 3.1) and the linear gate with top-1 argmax (Eq. 8, k = 1).
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"
#include "warp_reduce.cuh"

namespace molora {

// ------------------------------------------------------------------------------------------------
// Vocabulary routing: r = (number of interior/upper boundaries b_1..b_M that are <= v) when
// b_0 <= v < b_M, else -1.  For non-decreasing breaks this is the unique m with b_m <= v < b_{m+1}
// (an empty range b_m == b_{m+1} can hold no id and is skipped by the count).  M-1 integer compares
// per token, as the paper notes for Theorem 3.4; boundaries live in shared memory.
// ------------------------------------------------------------------------------------------------
// With `slot_of` non-null as well, adapter[i] is an adapter id of a catalog and slot_of[id] the hot-set slot that holds
// it (Definition 5.1), -1 if it is not resident: the target is slot * M + m.
// With `adapter` non-null the kernel is the compositional gate of Algorithm 1 (Definition 3.2): the modality m found
// from the id is combined with the token's adapter index a (request metadata) into the composite target a * M + m.
__global__ void __launch_bounds__(256) route_vocab_kernel(const int32_t* __restrict__ ids, int64_t N,
                                                          const int32_t* __restrict__ breaks, int M,
                                                          const int32_t* __restrict__ adapter, int n_adapters,
                                                          const int32_t* slot_of, int n_catalog,
                                                          int32_t* __restrict__ r_out, uint32_t* dev_status)
{
    __shared__ int32_t b[MOLORA_MAX_ADAPTERS + 1];
    ptx::grid_dependency_sync();
    for (int i = threadIdx.x; i <= M; i += blockDim.x) b[i] = __ldg(breaks + i);
    __syncthreads();
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool any_bad = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < N; i += stride) {
        const int32_t v = __ldg(ids + i);
        int32_t m;
        if (M <= 8) {
            m = 0;
#pragma unroll 8
            for (int j = 1; j < 8; ++j) m += (j < M && b[j] <= v) ? 1 : 0;
        } else {  // upper_bound(b_1..b_{M-1}, v) by bisection
            int lo = 1, hi = M;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (b[mid] <= v) lo = mid + 1; else hi = mid;
            }
            m = lo - 1;
        }
        bool inside = (v >= b[0]) && (v < b[M]);
        if (adapter != nullptr) {
            int32_t a = __ldg(adapter + i);
            if (slot_of != nullptr)                // hot-set: adapter id -> slot through the slot table's inverse (may be
                a = (a >= 0 && a < n_catalog) ? __ldcg(slot_of + a) : -1;      // rewritten by the maintenance stream)
            inside = inside && a >= 0 && a < n_adapters;
            m += a * M;
        }
        r_out[i] = inside ? m : -1;
        any_bad |= !inside;
    }
    if (dev_status != nullptr && __any_sync(0xFFFFFFFFu, any_bad) && lane_id() == 0)
        atomicOr(dev_status, MOLORA_DEV_ID_OUT_OF_RANGE);
}

molora_status_t launch_route_vocab(const int32_t* ids, int64_t N, const int32_t* breaks, int32_t M,
                                   const int32_t* adapter, int32_t n_adapters, int32_t* r_out, uint32_t* dev_status,
                                   cudaStream_t s, const int32_t* slot_of, int32_t n_catalog)
{
    if (N == 0) return MOLORA_OK;
    const int threads = 256;
    const int64_t want = ceil_div64(N, threads);
    const int blocks = (int)(want < 148 * 8 ? want : 148 * 8);
    return cuda_ok(launch_kernel(route_vocab_kernel, dim3(blocks), dim3(threads), 0, s, 1, false, ids, N, breaks, M, adapter,
                                  n_adapters, slot_of, n_catalog, r_out, dev_status));
}

// ------------------------------------------------------------------------------------------------
// Linear gate.  One warp owns TOK consecutive tokens; its 32 lanes split the hidden dimension in
// 16-byte vectors (lane L reads elements [L*VEC, L*VEC+VEC) of every KC = 32*VEC wide chunk), so x is
// streamed exactly once with fully coalesced 128-bit loads.  The matching KC x C slice of G is staged
// in shared memory once per CTA (8 warps share it) and read as float4 with a 4-float skew per lane,
// which makes the quarter-warp phases of LDS.128 bank-conflict free.  Each lane keeps TOK x CP fp32
// partial logits; one butterfly reduce-scatter per warp finishes them.
// ------------------------------------------------------------------------------------------------
template <typename T, int CP, int TOK>
__global__ void __launch_bounds__(256) route_gate_kernel(const T* __restrict__ x, int64_t N, int d, int64_t ldx,
                                                         const float* __restrict__ G, const float* __restrict__ bias,
                                                         int C, int32_t* __restrict__ r_out,
                                                         float* __restrict__ logits_out)
{
    constexpr int VEC = VecTraits<T>::kElems;
    constexpr int KC = 32 * VEC;                 // hidden elements per chunk
    constexpr int LANE_STRIDE = VEC * CP + 4;    // floats between the G rows of consecutive lanes (skewed)
    constexpr int WARPS = 8;
    __shared__ __align__(16) float Gs[32 * LANE_STRIDE];
    __shared__ float zs[WARPS][TOK][CP];

    const int warp = threadIdx.x >> 5, lane = lane_id();
    ptx::grid_dependency_sync();
    const int64_t tok0 = ((int64_t)blockIdx.x * WARPS + warp) * TOK;

    float acc[TOK][CP];
#pragma unroll
    for (int t = 0; t < TOK; ++t)
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[t][c] = 0.f;

    const T* xrow[TOK];
#pragma unroll
    for (int t = 0; t < TOK; ++t) {
        const int64_t i = tok0 + t < N ? tok0 + t : N - 1;   // clamp: tail tokens recompute the last row, never stored
        xrow[t] = x + i * ldx;
    }

    for (int k0 = 0; k0 < d; k0 += KC) {
        // stage G[k0 .. k0+KC) x [0, C) into the skewed layout, zero-filling c >= C and k >= d
        for (int e = threadIdx.x; e < KC * CP; e += blockDim.x) {
            const int kk = e / CP, c = e - kk * CP;
            const int k = k0 + kk;
            const float g = (k < d && c < C) ? __ldg(G + (int64_t)k * C + c) : 0.f;
            Gs[(kk / VEC) * LANE_STRIDE + (kk % VEC) * CP + c] = g;
        }
        __syncthreads();
        const int k = k0 + lane * VEC;
        if (k < d) {   // d is a multiple of VEC, so a vector is either fully inside or fully outside
            float xv[TOK][VEC];
#pragma unroll
            for (int t = 0; t < TOK; ++t) {
                const uint4 v = ldg128_stream(xrow[t] + k);
                unpack<T>(v, xv[t]);
            }
            const float* g = Gs + lane * LANE_STRIDE;
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
#pragma unroll
                for (int c4 = 0; c4 < CP; c4 += 4) {
                    const float4 gv = *reinterpret_cast<const float4*>(g + j * CP + c4);
#pragma unroll
                    for (int t = 0; t < TOK; ++t) {
                        acc[t][c4 + 0] = fmaf(xv[t][j], gv.x, acc[t][c4 + 0]);
                        acc[t][c4 + 1] = fmaf(xv[t][j], gv.y, acc[t][c4 + 1]);
                        acc[t][c4 + 2] = fmaf(xv[t][j], gv.z, acc[t][c4 + 2]);
                        acc[t][c4 + 3] = fmaf(xv[t][j], gv.w, acc[t][c4 + 3]);
                    }
                }
            }
        }
        __syncthreads();
    }

    // finish the logits: reduce-scatter over the warp, then park them in shared memory
    constexpr int NV = TOK * CP;
    float* flat = &acc[0][0];
    warp_reduce_scatter<NV>(flat, lane);
    constexpr int PER_LANE = NV >= 32 ? NV / 32 : 1;
    constexpr int REPLICAS = NV >= 32 ? 1 : 32 / NV;   // lanes that end up holding the same sum
    const int base = reduce_scatter_base<NV>(lane);
    if (lane % REPLICAS == 0) {
#pragma unroll
        for (int j = 0; j < PER_LANE; ++j) (&zs[warp][0][0])[base + j] = flat[j];
    }
    __syncwarp();
    if (lane < TOK && tok0 + lane < N) {
        const int64_t i = tok0 + lane;
        float best = 0.f;
        int arg = 0;
        for (int c = 0; c < C; ++c) {
            float z = zs[warp][lane][c];
            if (bias != nullptr) z += __ldg(bias + c);
            if (logits_out != nullptr) logits_out[i * C + c] = z;
            if (c == 0 || z > best) { best = z; arg = c; }   // strict '>' keeps the lowest index on ties
        }
        r_out[i] = arg;
    }
}

// ------------------------------------------------------------------------------------------------
// Linear gate, few adapters (C <= 8) and d * CP * 4 bytes of G small enough to stay resident in shared
// memory: no per-chunk staging and no block-wide synchronisation inside the token loop.  A CTA of four
// warps copies G once (skewed per lane as above); then each warp streams its tokens two at a time with all
// of their 16-byte loads issued before the first FMA, which keeps ~8 KB per warp in flight.
// ------------------------------------------------------------------------------------------------
template <typename T, int CP>
__global__ void __launch_bounds__(128) route_gate_resident_kernel(const T* __restrict__ x, int64_t N, int d, int64_t ldx,
                                                                  const float* __restrict__ G,
                                                                  const float* __restrict__ bias, int C,
                                                                  int32_t* __restrict__ r_out,
                                                                  float* __restrict__ logits_out, int tokens_per_warp)
{
    constexpr int VEC = VecTraits<T>::kElems;
    constexpr int KC = 32 * VEC;
    constexpr int LANE_STRIDE = VEC * CP + 4;
    constexpr int BATCH = 8;                       // 16-byte vectors per token kept in flight per lane
    extern __shared__ __align__(16) float Gres[];  // [chunks][32 lanes][LANE_STRIDE]
    const int chunks = (d + KC - 1) / KC;
    ptx::grid_dependency_sync();
    if (C == CP && (d % KC) == 0) {
        // G rows are CP floats = whole 16-byte vectors: copy them as they are (coalesced float4 loads)
        constexpr int V = CP / 4;
        // (asynchronous 16-byte copies: all of a thread's requests are in flight at once)
        for (int e = threadIdx.x; e < d * V; e += blockDim.x) {
            const int k = e / V, v = e - k * V;
            const int ch = k / KC, kk = k - ch * KC;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(
                &Gres[(ch * 32 + kk / VEC) * LANE_STRIDE + (kk % VEC) * CP + v * 4]);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(reinterpret_cast<const float4*>(G) + e)
                         : "memory");
        }
        asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    } else {
        for (int e = threadIdx.x; e < chunks * KC * CP; e += blockDim.x) {
            const int k = e / CP, c = e - k * CP;
            const float g = (k < d && c < C) ? __ldg(G + (int64_t)k * C + c) : 0.f;
            const int ch = k / KC, kk = k - ch * KC;
            Gres[(ch * 32 + kk / VEC) * LANE_STRIDE + (kk % VEC) * CP + c] = g;
        }
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t wtok0 = ((int64_t)blockIdx.x * 4 + warp) * tokens_per_warp;
    for (int t0 = 0; t0 < tokens_per_warp; t0 += 2) {
        const int64_t i0 = wtok0 + t0;
        if (i0 >= N) break;
        const int64_t i1 = i0 + 1 < N && t0 + 1 < tokens_per_warp ? i0 + 1 : i0;
        const T* x0 = x + i0 * ldx + lane * VEC;
        const T* x1 = x + i1 * ldx + lane * VEC;
        float acc[2][CP];
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[0][c] = acc[1][c] = 0.f;
        for (int cb = 0; cb < chunks; cb += BATCH) {
            uint4 v0[BATCH], v1[BATCH];
#pragma unroll
            for (int b = 0; b < BATCH; ++b) {
                const int k = (cb + b) * KC + lane * VEC;
                if (k < d) {
                    v0[b] = ldg128_stream(x0 + (cb + b) * KC);
                    v1[b] = ldg128_stream(x1 + (cb + b) * KC);
                } else {
                    v0[b] = make_uint4(0, 0, 0, 0);
                    v1[b] = make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int b = 0; b < BATCH; ++b) {
                if (cb + b < chunks) {
                    float f0[VEC], f1[VEC];
                    unpack<T>(v0[b], f0);
                    unpack<T>(v1[b], f1);
                    const float* g = Gres + ((cb + b) * 32 + lane) * LANE_STRIDE;
#pragma unroll
                    for (int j = 0; j < VEC; ++j) {
#pragma unroll
                        for (int c4 = 0; c4 < CP; c4 += 4) {
                            const float4 gv = *reinterpret_cast<const float4*>(g + j * CP + c4);
                            acc[0][c4 + 0] = fmaf(f0[j], gv.x, acc[0][c4 + 0]);
                            acc[0][c4 + 1] = fmaf(f0[j], gv.y, acc[0][c4 + 1]);
                            acc[0][c4 + 2] = fmaf(f0[j], gv.z, acc[0][c4 + 2]);
                            acc[0][c4 + 3] = fmaf(f0[j], gv.w, acc[0][c4 + 3]);
                            acc[1][c4 + 0] = fmaf(f1[j], gv.x, acc[1][c4 + 0]);
                            acc[1][c4 + 1] = fmaf(f1[j], gv.y, acc[1][c4 + 1]);
                            acc[1][c4 + 2] = fmaf(f1[j], gv.z, acc[1][c4 + 2]);
                            acc[1][c4 + 3] = fmaf(f1[j], gv.w, acc[1][c4 + 3]);
                        }
                    }
                }
            }
        }
        // finish both tokens' logits: plain butterfly sums (2 * CP values, small next to the d / 32 FMAs per lane)
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                float v = acc[t][c];
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
                acc[t][c] = v;
            }
        if (lane < 2) {
            const int64_t i = lane == 0 ? i0 : i1;
            if (lane == 0 || i1 != i0) {
                float best = 0.f;
                int arg = 0;
#pragma unroll
                for (int c = 0; c < CP; ++c) {
                    if (c < C) {
                        float z = lane == 0 ? acc[0][c] : acc[1][c];
                        if (bias != nullptr) z += __ldg(bias + c);
                        if (logits_out != nullptr) logits_out[i * C + c] = z;
                        if (c == 0 || z > best) { best = z; arg = c; }
                    }
                }
                r_out[i] = arg;
            }
        }
    }
}

// Small calls (at most four tokens per warp, rows of at most eight 16-byte vectors per lane): latency decides, so
// a warp requests ALL of its activations first (up to 16 KB in flight per warp), while the CTA's copy of G is still
// on its way into shared memory, and only then starts the FMAs.  Same layout of G and the same summation order per
// token as route_gate_resident_kernel.
template <typename T, int CP, int TPW>
__global__ void __launch_bounds__(128) route_gate_resident_burst_kernel(const T* __restrict__ x, int64_t N, int d,
                                                                        int64_t ldx, const float* __restrict__ G,
                                                                        const float* __restrict__ bias, int C,
                                                                        int32_t* __restrict__ r_out,
                                                                        float* __restrict__ logits_out)
{
    constexpr int VEC = VecTraits<T>::kElems;
    constexpr int KC = 32 * VEC;
    constexpr int LANE_STRIDE = VEC * CP + 4;
    constexpr int MAXCH = 8;                       // chunks per row (the launcher guarantees d <= MAXCH * KC)
    extern __shared__ __align__(16) float Gres[];  // [chunks][32 lanes][LANE_STRIDE]
    const int chunks = (d + KC - 1) / KC;
    const int warp = threadIdx.x >> 5, lane = lane_id();
    ptx::grid_dependency_sync();

    // ---- all activations of my tokens
    const int64_t wtok0 = ((int64_t)blockIdx.x * 4 + warp) * TPW;
    uint4 v[TPW][MAXCH];
#pragma unroll
    for (int t = 0; t < TPW; ++t) {
        const int64_t i = wtok0 + t < N ? wtok0 + t : N - 1;          // tail tokens recompute the last one
        const T* xi = x + i * ldx + lane * VEC;
#pragma unroll
        for (int b = 0; b < MAXCH; ++b)
            v[t][b] = (b * KC + lane * VEC < d) ? ldg128_stream(xi + b * KC) : make_uint4(0, 0, 0, 0);
    }
    // ---- G into shared memory
    if (C == CP && (d % KC) == 0) {
        constexpr int V = CP / 4;
        for (int e = threadIdx.x; e < d * V; e += blockDim.x) {
            const int k = e / V, vv = e - k * V;
            const int ch = k / KC, kk = k - ch * KC;
            const uint32_t dst = (uint32_t)__cvta_generic_to_shared(
                &Gres[(ch * 32 + kk / VEC) * LANE_STRIDE + (kk % VEC) * CP + vv * 4]);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(reinterpret_cast<const float4*>(G) + e)
                         : "memory");
        }
        asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
    } else {
        for (int e = threadIdx.x; e < chunks * KC * CP; e += blockDim.x) {
            const int k = e / CP, c = e - k * CP;
            const float g = (k < d && c < C) ? __ldg(G + (int64_t)k * C + c) : 0.f;
            const int ch = k / KC, kk = k - ch * KC;
            Gres[(ch * 32 + kk / VEC) * LANE_STRIDE + (kk % VEC) * CP + c] = g;
        }
    }
    __syncthreads();
    if (wtok0 >= N) return;

    float acc[TPW][CP];
#pragma unroll
    for (int t = 0; t < TPW; ++t)
#pragma unroll
        for (int c = 0; c < CP; ++c) acc[t][c] = 0.f;
#pragma unroll
    for (int b = 0; b < MAXCH; ++b) {
        if (b < chunks) {
            float f[TPW][VEC];
#pragma unroll
            for (int t = 0; t < TPW; ++t) unpack<T>(v[t][b], f[t]);
            const float* g = Gres + (b * 32 + lane) * LANE_STRIDE;
#pragma unroll
            for (int j = 0; j < VEC; ++j) {
#pragma unroll
                for (int c4 = 0; c4 < CP; c4 += 4) {
                    const float4 gv = *reinterpret_cast<const float4*>(g + j * CP + c4);
#pragma unroll
                    for (int t = 0; t < TPW; ++t) {
                        acc[t][c4 + 0] = fmaf(f[t][j], gv.x, acc[t][c4 + 0]);
                        acc[t][c4 + 1] = fmaf(f[t][j], gv.y, acc[t][c4 + 1]);
                        acc[t][c4 + 2] = fmaf(f[t][j], gv.z, acc[t][c4 + 2]);
                        acc[t][c4 + 3] = fmaf(f[t][j], gv.w, acc[t][c4 + 3]);
                    }
                }
            }
        }
    }
    // finish the logits: plain butterfly sums
#pragma unroll
    for (int t = 0; t < TPW; ++t)
#pragma unroll
        for (int c = 0; c < CP; ++c) {
            float z = acc[t][c];
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) z += __shfl_xor_sync(0xFFFFFFFFu, z, off);
            acc[t][c] = z;
        }
    if (lane < TPW && wtok0 + lane < N) {
        const int64_t i = wtok0 + lane;
        float best = 0.f;
        int arg = 0;
#pragma unroll
        for (int c = 0; c < CP; ++c) {
            if (c < C) {
                float z = 0.f;
#pragma unroll
                for (int t = 0; t < TPW; ++t)
                    if (t == lane) z = acc[t][c];
                if (bias != nullptr) z += __ldg(bias + c);
                if (logits_out != nullptr) logits_out[i * C + c] = z;
                if (c == 0 || z > best) { best = z; arg = c; }
            }
        }
        r_out[i] = arg;
    }
}

template <typename T, int CP>
static molora_status_t gate_resident_launch(const void* x, int64_t N, int d, int64_t ldx, const float* G,
                                            const float* bias, int C, int32_t* r_out, float* logits_out,
                                            cudaStream_t s, bool& handled)
{
    constexpr int VEC = VecTraits<T>::kElems;
    const int chunks = (d + 32 * VEC - 1) / (32 * VEC);
    const size_t smem = (size_t)chunks * 32 * (VEC * CP + 4) * sizeof(float);
    handled = smem <= 96 * 1024;
    if (!handled) return MOLORA_OK;
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(route_gate_resident_kernel<T, CP>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 96 * 1024) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        configured = true;
    }
    // tokens per warp: 8 when that still gives at least ~one CTA per SM, otherwise fewer (small calls)
    int tpw = 8;
    while (tpw > 2 && ceil_div64(N, 4 * tpw) < 148) tpw /= 2;
    const int64_t blocks = ceil_div64(N, 4 * tpw);
    if (tpw <= 4 && chunks <= 8) {   // small call: the burst variant (every load of a warp in flight at once)
        static bool configured_burst_dev[kMaxDevices] = {};
        bool& configured_burst = configured_burst_dev[device_slot()];
        if (!configured_burst) {
            if (cudaFuncSetAttribute(route_gate_resident_burst_kernel<T, CP, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     96 * 1024) != cudaSuccess ||
                cudaFuncSetAttribute(route_gate_resident_burst_kernel<T, CP, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     96 * 1024) != cudaSuccess)
                return MOLORA_ERR_CUDA;
            configured_burst = true;
        }
        if (tpw == 4)
            return cuda_ok(launch_kernel(route_gate_resident_burst_kernel<T, CP, 4>, dim3((unsigned)blocks), dim3(128), smem,
                                         s, 1, false, static_cast<const T*>(x), N, d, ldx, G, bias, C, r_out, logits_out));
        return cuda_ok(launch_kernel(route_gate_resident_burst_kernel<T, CP, 2>, dim3((unsigned)blocks), dim3(128), smem, s,
                                     1, false, static_cast<const T*>(x), N, d, ldx, G, bias, C, r_out, logits_out));
    }
    return cuda_ok(launch_kernel(route_gate_resident_kernel<T, CP>, dim3((unsigned)blocks), dim3(128), smem, s, 1, false,
                                  static_cast<const T*>(x), N, d, ldx, G, bias, C, r_out, logits_out, tpw));
}

template <typename T, int CP, int TOK>
static molora_status_t gate_launch(const void* x, int64_t N, int d, int64_t ldx, const float* G, const float* bias,
                                   int C, int32_t* r_out, float* logits_out, cudaStream_t s)
{
    const int64_t blocks = ceil_div64(N, 8 * TOK);
    return cuda_ok(launch_kernel(route_gate_kernel<T, CP, TOK>, dim3((unsigned)blocks), dim3(256), 0, s, 1, false,
                                  static_cast<const T*>(x), N, d, ldx, G, bias, C, r_out, logits_out));
}

template <typename T>
static molora_status_t gate_dispatch(const void* x, int64_t N, int d, int64_t ldx, const float* G, const float* bias,
                                     int C, int32_t* r_out, float* logits_out, cudaStream_t s)
{
    if (C <= 8) {   // few adapters: G stays resident in shared memory when it fits
        bool handled = false;
        const molora_status_t st =
            C <= 4 ? gate_resident_launch<T, 4>(x, N, d, ldx, G, bias, C, r_out, logits_out, s, handled)
                   : gate_resident_launch<T, 8>(x, N, d, ldx, G, bias, C, r_out, logits_out, s, handled);
        if (handled || st != MOLORA_OK) return st;
    }
    if (C <= 4) return gate_launch<T, 4, 4>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);
    if (C <= 8) return gate_launch<T, 8, 4>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);
    if (C <= 16) return gate_launch<T, 16, 4>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);
    return gate_launch<T, 32, 2>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);   // C <= 32 checked by the caller
}

// ------------------------------------------------------------------------------------------------
// Top-k weighted routing (Eq. 8): per token the k largest logits (equal logits: lowest index first) and the softmax
// over the kept ones.  One thread per token, C <= 32 logits in registers; k passes of a masked argmax.
__global__ void __launch_bounds__(256) topk_softmax_kernel(const float* __restrict__ logits, int64_t N, int C, int k,
                                                           int32_t* __restrict__ idx_out, float* __restrict__ w_out)
{
    ptx::grid_dependency_sync();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    float z[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) z[c] = c < C ? __ldg(logits + i * C + c) : 0.f;
    uint32_t taken = 0;
    float zmax = 0.f, den = 0.f;
    float kept[32];
    for (int j = 0; j < k; ++j) {
        int best = -1;
        float bz = 0.f;
#pragma unroll
        for (int c = 0; c < 32; ++c) {
            if (c < C && !((taken >> c) & 1u) && (best < 0 || z[c] > bz)) {
                best = c;
                bz = z[c];
            }
        }
        taken |= 1u << best;
        idx_out[(int64_t)j * N + i] = best;
        if (j == 0) zmax = bz;
        const float e = expf(bz - zmax);
#pragma unroll
        for (int q = 0; q < 32; ++q)
            if (q == j) kept[q] = e;
        den += e;
    }
    for (int j = 0; j < k; ++j) {
        float e = 0.f;
#pragma unroll
        for (int q = 0; q < 32; ++q)
            if (q == j) e = kept[q];
        w_out[(int64_t)j * N + i] = e / den;
    }
}

molora_status_t launch_topk_softmax(const float* logits, int64_t N, int32_t C, int32_t k, int32_t* idx_out, float* w_out,
                                    cudaStream_t s)
{
    if (N == 0) return MOLORA_OK;
    return cuda_ok(launch_kernel(topk_softmax_kernel, dim3((unsigned)ceil_div64(N, 256)), dim3(256), 0, s, 1, false, logits, N,
                                 (int)C, (int)k, idx_out, w_out));
}

// Top-k routing in one pass: the k adapters of a token, sorted by index, name a SET (a multiset: a caller may repeat an
// adapter); sets are numbered densely, rank = sum_j binom(a_j + j, j + 1) over the sorted adapters, and the weights are
// stored in the same order.  Tokens with an adapter outside [0, C) are left unrouted.  k <= 4.  The first block also
// writes the table set -> adapters (4 bytes per set) that the apply kernels read.
__global__ void __launch_bounds__(256) topk_sets_kernel(const int32_t* __restrict__ idx, const float* __restrict__ w, int64_t N,
                                                        int C, int k, int32_t* __restrict__ set_out, float* __restrict__ w_out,
                                                        uint8_t* __restrict__ table_out)
{
    ptx::grid_dependency_sync();
    if (blockIdx.x == 0) {
        const int n_sets = (int)topk_set_count(C, k);
        for (int t = threadIdx.x; t < n_sets; t += blockDim.x) {
            int rest = t;
            uint8_t a[4] = {0, 0, 0, 0};
            for (int j = k - 1; j >= 0; --j) {                      // largest b with binom(b, j + 1) <= rest; a_j = b - j
                int b = j;
                while (binom_small(b + 1, j + 1) <= rest) ++b;
                rest -= (int)binom_small(b, j + 1);
                a[j] = (uint8_t)(b - j);
            }
            for (int j = 0; j < 4; ++j) table_out[t * 4 + j] = a[j];
        }
    }
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= N) return;
    int a[4];
    float f[4];
    bool ok = true;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        a[j] = j < k ? __ldg(idx + (int64_t)j * N + i) : 0x7FFFFFFF;
        f[j] = j < k ? __ldg(w + (int64_t)j * N + i) : 0.f;
        ok = ok && (j >= k || (a[j] >= 0 && a[j] < C));
    }
#pragma unroll
    for (int p = 0; p < 3; ++p)                     // three rounds of a bubble sort over four entries
#pragma unroll
        for (int j = 0; j < 3 - p; ++j)
            if (a[j] > a[j + 1]) {
                const int ta = a[j]; a[j] = a[j + 1]; a[j + 1] = ta;
                const float tf = f[j]; f[j] = f[j + 1]; f[j + 1] = tf;
            }
    int set = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (j < k) {
            if (ok) set += (int)binom_small(a[j] + j, j + 1);
            w_out[(int64_t)j * N + i] = f[j];
        }
    set_out[i] = ok ? set : -1;
}

molora_status_t launch_topk_sets(const int32_t* idx, const float* w, int64_t N, int32_t C, int32_t k, int32_t* set_out,
                                 float* w_out, uint8_t* table_out, cudaStream_t s)
{
    if (N == 0) return MOLORA_OK;
    return cuda_ok(launch_kernel(topk_sets_kernel, dim3((unsigned)ceil_div64(N, 256)), dim3(256), 0, s, 1, false, idx, w, N, (int)C,
                                 (int)k, set_out, w_out, table_out));
}

size_t route_gate_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C)
{
    if (xdt != MOLORA_BF16) return 0;
    const size_t a = route_gate_mma_workspace_bytes(d, C), b = route_gate_umma_workspace_bytes(d, C);
    return a > b ? a : b;      // which kernel runs depends on N, which this query does not know
}

size_t route_gate_prepared_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C)
{
    if (xdt != MOLORA_BF16 || C <= 4) return 0;
    return (route_gate_umma_workspace_bytes(d, C) + 255) / 256 * 256 + route_gate_mma_workspace_bytes(d, C);
}

molora_status_t launch_route_gate(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* G,
                                  const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                  uint32_t* dev_status, cudaStream_t s, int image)
{
    // prepared form: the workspace holds the tcgen05 gate's image (if that kernel can take this d and C) and behind it
    // the mma.sync gate's; otherwise one image at the start of the workspace, whichever kernel runs
    const bool two = image != kImageBuildAndUse;
    char* ws_mma = static_cast<char*>(ws) + (two ? (route_gate_umma_workspace_bytes(d, C) + 255) / 256 * 256 : 0);
    if (image == kImageBuildOnly) {
        if (xdt != MOLORA_BF16 || C <= 4) return MOLORA_OK;       // the CUDA-core gates read G as it is
        if (gate_umma_eligible(1 << 20, d, C)) {
            const molora_status_t st = launch_route_gate_umma(nullptr, 0, d, 0, G, nullptr, C, nullptr, nullptr, ws, nullptr, s, image);
            if (st != MOLORA_OK) return st;
        }
        return launch_route_gate_mma(nullptr, 0, d, 0, G, nullptr, C, nullptr, nullptr, ws_mma, s, image);
    }
    if (N == 0) return MOLORA_OK;
    if (xdt == MOLORA_BF16 && gate_umma_eligible(N, d, C))       // the only gate kernel with device-side waits
        return launch_route_gate_umma(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, dev_status, s, image);
    if (xdt == MOLORA_BF16 && C > 4)
        return launch_route_gate_mma(x, N, d, ldx, G, bias, C, r_out, logits_out, ws_mma, s, image);
    if (xdt == MOLORA_BF16) return gate_dispatch<__nv_bfloat16>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);
    return gate_dispatch<float>(x, N, d, ldx, G, bias, C, r_out, logits_out, s);
}

}  // namespace molora
