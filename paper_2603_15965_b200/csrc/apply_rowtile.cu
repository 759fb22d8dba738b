// Grouped LoRA shrink -> expand on CUDA cores (Eq. 2 evaluated segment by segment, Figure 2 right).
//
// This is the path for small segments (decode-sized batches) and for fp32 storage.  One CTA owns a
// tile of TM = 128 / rank consecutive positions of one segment (all rows of a tile share adapter c):
//
//   shrink  t[m][n] = sum_k x[row_m][k] * A_c[k][n]
//           the 256 threads split d_in in 16-byte vectors; thread-local partial sums for the whole
//           TM x rank tile (128 fp32 registers) are finished by one butterfly reduce-scatter per warp
//           and a cross-warp add through shared memory.  x is streamed once with 128-bit loads;
//           A_c rows (rank elements, contiguous) come through L1/L2.
//   expand  y[row_m][o] += scale * sum_n t[m][n] * B_c[n][o]
//           the threads split d_out in 16-byte vectors; t is broadcast from shared memory, B_c rows
//           are read with coalesced 128-bit loads, y is read, updated in fp32 and stored once (one
//           rounding to the storage type) at the token's original row.
//
// The intermediate t never leaves the chip.  Tiles are located on the device from `offsets`
// (no host read of the histogram), so the grid is sized for the worst case and surplus CTAs exit.
#include "common.cuh"
#include "sm100_ptx.cuh"
#include "warp_reduce.cuh"

namespace molora {

struct ApplyBatchParams {
    molora_proj_desc_t p[MOLORA_MAX_PROJECTIONS];
    const int32_t* offsets;
    const int32_t* perm;
    int32_t P;
    int32_t C;
    int32_t max_rows;     // segments with at least this many rows belong to the tensor-core kernel
};

constexpr int kRowTileThreads = 256;

template <typename T, int R>
__global__ void __launch_bounds__(kRowTileThreads, 1) apply_rowtile_kernel(const __grid_constant__ ApplyBatchParams prm)
{
    constexpr int VEC = VecTraits<T>::kElems;
    constexpr int TM = 128 / R;              // rows per tile: TM * R = 128 partial sums per thread
    constexpr int WARPS = kRowTileThreads / 32;
    constexpr int RV = R / VEC;              // 16-byte vectors per row of A_c

    const molora_proj_desc_t& pd = prm.p[blockIdx.y];
    if (pd.rank != R) return;                // a launch of this instantiation serves the projections of rank R

    ptx::grid_dependency_sync();             // offsets and perm come from the grouping kernel
    int seg, row0, rows;
    if (!find_tile(prm.offsets, prm.C, TM, blockIdx.x, 1, prm.max_rows, seg, row0, rows)) return;

    __shared__ __align__(16) float partial[WARPS][128];
    __shared__ __align__(16) float t_s[128];   // [TM][R]
    __shared__ int32_t row_s[TM];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid < TM) row_s[tid] = __ldg(prm.perm + row0 + (tid < rows ? tid : rows - 1));   // pad with the last row
    __syncthreads();

    const int d_in = pd.d_in, d_out = pd.d_out;
    const T* __restrict__ x = static_cast<const T*>(pd.x);
    T* __restrict__ y = static_cast<T*>(pd.y);
    const T* __restrict__ Ac = static_cast<const T*>(pd.A) + (int64_t)seg * d_in * R;
    const T* __restrict__ Bc = static_cast<const T*>(pd.B) + (int64_t)seg * R * d_out;

    // ---------------- shrink ----------------
    float acc[TM * R];
#pragma unroll
    for (int i = 0; i < TM * R; ++i) acc[i] = 0.f;

    for (int k0 = tid * VEC; k0 < d_in; k0 += kRowTileThreads * VEC) {
        uint4 xp[TM];
#pragma unroll
        for (int m = 0; m < TM; ++m) xp[m] = ldg128_stream(x + (int64_t)row_s[m] * pd.ldx + k0);
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            float af[R];
#pragma unroll
            for (int v = 0; v < RV; ++v) unpack<T>(ldg128(Ac + (int64_t)(k0 + j) * R + v * VEC), af + v * VEC);
#pragma unroll
            for (int m = 0; m < TM; ++m) {
                float xv[VEC];
                unpack<T>(xp[m], xv);
#pragma unroll
                for (int n = 0; n < R; ++n) acc[m * R + n] = fmaf(xv[j], af[n], acc[m * R + n]);
            }
        }
    }

    warp_reduce_scatter<128>(acc, lane);
    {
        const int base = reduce_scatter_base<128>(lane);
        *reinterpret_cast<float4*>(&partial[warp][base]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    }
    __syncthreads();
    if (tid < 128) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < WARPS; ++w) s += partial[w][tid];
        // fold the LoRA scale (and the token's routing weight, if given) into t once: t_s is [TM][R], row m = tid / R
        const float rs = pd.row_scale != nullptr ? __ldg(pd.row_scale + row_s[tid / R]) : 1.f;
        t_s[tid] = s * pd.scale * rs;
    }
    __syncthreads();

    // ---------------- expand ----------------
    for (int o0 = tid * VEC; o0 < d_out; o0 += kRowTileThreads * VEC) {
        uint4 yp[TM];
#pragma unroll
        for (int m = 0; m < TM; ++m) yp[m] = ld128_rw_stream(y + (int64_t)row_s[m] * pd.ldy + o0);
        float out[TM][VEC];
#pragma unroll
        for (int m = 0; m < TM; ++m)
#pragma unroll
            for (int j = 0; j < VEC; ++j) out[m][j] = 0.f;
#pragma unroll
        for (int n4 = 0; n4 < R; n4 += 4) {
            float bf[4][VEC];
#pragma unroll
            for (int q = 0; q < 4; ++q) unpack<T>(ldg128(Bc + (int64_t)(n4 + q) * d_out + o0), bf[q]);
#pragma unroll
            for (int m = 0; m < TM; ++m) {
                const float4 tv = *reinterpret_cast<const float4*>(&t_s[m * R + n4]);
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    out[m][j] = fmaf(tv.x, bf[0][j], out[m][j]);
                    out[m][j] = fmaf(tv.y, bf[1][j], out[m][j]);
                    out[m][j] = fmaf(tv.z, bf[2][j], out[m][j]);
                    out[m][j] = fmaf(tv.w, bf[3][j], out[m][j]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < TM; ++m) {
            if (m < rows) {
                float yv[VEC];
                unpack<T>(yp[m], yv);
#pragma unroll
                for (int j = 0; j < VEC; ++j) yv[j] += out[m][j];
                stg128(y + (int64_t)row_s[m] * pd.ldy + o0, pack<T>(yv));
            }
        }
    }
}

template <typename T, int R>
static cudaError_t rowtile_launch(const ApplyBatchParams& prm, int64_t N, cudaStream_t s)
{
    constexpr int TM = 128 / R;
    // every segment adds at most one partial tile; with a row cap only min(N, C * cap) rows can come here
    const int64_t cap_rows = prm.max_rows == INT32_MAX ? N : (N < (int64_t)prm.C * prm.max_rows ? N : (int64_t)prm.C * prm.max_rows);
    const int64_t tiles = ceil_div64(cap_rows, TM) + prm.C;
    dim3 grid((unsigned)tiles, (unsigned)prm.P);
    return launch_kernel(apply_rowtile_kernel<T, R>, grid, dim3(kRowTileThreads), 0, s, 1, false, prm);
}

template <typename T>
static cudaError_t rowtile_dispatch(const ApplyBatchParams& prm, int64_t N, cudaStream_t s)
{
    bool has[4] = {false, false, false, false};
    for (int i = 0; i < prm.P; ++i) {
        const int r = prm.p[i].rank;
        has[r == 8 ? 0 : r == 16 ? 1 : r == 32 ? 2 : 3] = true;
    }
    cudaError_t e = cudaSuccess;
    if (has[0] && e == cudaSuccess) e = rowtile_launch<T, 8>(prm, N, s);
    if (has[1] && e == cudaSuccess) e = rowtile_launch<T, 16>(prm, N, s);
    if (has[2] && e == cudaSuccess) e = rowtile_launch<T, 32>(prm, N, s);
    if (has[3] && e == cudaSuccess) e = rowtile_launch<T, 64>(prm, N, s);
    return e;
}

molora_status_t launch_apply_rowtile(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N,
                                     int32_t C, const int32_t* offsets, const int32_t* perm, int32_t max_rows,
                                     cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    ApplyBatchParams prm;
    for (int i = 0; i < P; ++i) prm.p[i] = projs[i];
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) prm.p[i] = molora_proj_desc_t{};
    prm.offsets = offsets;
    prm.perm = perm;
    prm.P = P;
    prm.C = C;
    prm.max_rows = max_rows;
    return cuda_ok(dt == MOLORA_BF16 ? rowtile_dispatch<__nv_bfloat16>(prm, N, s) : rowtile_dispatch<float>(prm, N, s));
}

}  // namespace molora
