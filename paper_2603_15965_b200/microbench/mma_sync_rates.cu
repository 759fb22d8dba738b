// Micro-benchmark behind the small-tile apply kernels' design notes: latency of a dependent chain of
// mma.sync.m16n8k16 (bf16 in, fp32 accumulate), its throughput per warp and per SM, and the dependent latency of
// ldmatrix.x4, on one B200.  Not part of the library.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o mma_sync_rates mma_sync_rates.cu && ./mma_sync_rates
#include <cstdio>
#include <cuda_runtime.h>
#include <stdint.h>
__device__ __forceinline__ void mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <int ILP>
__global__ void k(float* out, long long* cyc, int iters)
{
    uint32_t a[4] = {threadIdx.x, 2, 3, 4};
    float c[ILP][4];
    for (int i = 0; i < ILP; ++i) for (int j = 0; j < 4; ++j) c[i][j] = 0.f;
    __syncthreads();
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < ILP; ++i) mma(c[i], a, 5 + i, 7);
    }
    long long t1 = clock64();
    float s = 0; for (int i = 0; i < ILP; ++i) for (int j = 0; j < 4; ++j) s += c[i][j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
    if (threadIdx.x == 0) cyc[blockIdx.x] = t1 - t0;
}
__global__ void ldsm_lat(float* out, long long* cyc, int iters)
{
    __shared__ __align__(16) unsigned char sm[8192];
    for (int i = threadIdx.x; i < 2048; i += blockDim.x) ((uint32_t*)sm)[i] = (i * 16) % 4096;
    __syncthreads();
    uint32_t addr = (uint32_t)__cvta_generic_to_shared(sm) + (threadIdx.x & 31) * 16;
    uint32_t base = (uint32_t)__cvta_generic_to_shared(sm);
    uint32_t r[4] = {0, 0, 0, 0};
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
        addr = base + ((r[0] + (threadIdx.x & 31) * 16) & 4095);
    }
    long long t1 = clock64();
    out[threadIdx.x] = r[0] + r[1];
    if (threadIdx.x == 0) cyc[0] = t1 - t0;
}
int main()
{
    float* out; long long* cyc; cudaMalloc(&out, 1 << 20); cudaMalloc(&cyc, 4096);
    long long h[148];
    const int iters = 2000;
    auto run = [&](auto kern, int ilp, int warps, int blocks) {
        kern<<<blocks, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize();
        kern<<<blocks, warps * 32>>>(out, cyc, iters); cudaDeviceSynchronize();
        cudaMemcpy(h, cyc, sizeof(long long) * blocks, cudaMemcpyDeviceToHost);
        double cy = (double)h[0] / iters;
        printf("ILP %d warps %2d blocks %3d: %.1f cycles per round of %d MMAs per warp -> %.2f cycles per MMA per warp, %.3f MMA/cycle/SM\n", ilp, warps, blocks, cy, ilp, cy / ilp, ilp * warps / cy);
    };
    run(k<1>, 1, 1, 1); run(k<2>, 2, 1, 1); run(k<4>, 4, 1, 1); run(k<8>, 8, 1, 1); run(k<16>, 16, 1, 1);
    run(k<1>, 1, 4, 1); run(k<1>, 1, 8, 1); run(k<1>, 1, 16, 1); run(k<4>, 4, 8, 1); run(k<8>, 8, 8, 1); run(k<4>, 4, 16, 1); run(k<8>, 8, 16, 148);
    ldsm_lat<<<1, 32>>>(out, cyc, iters); cudaDeviceSynchronize();
    cudaMemcpy(h, cyc, sizeof(long long), cudaMemcpyDeviceToHost);
    printf("ldmatrix.x4 dependent latency: %.1f cycles\n", (double)h[0] / iters);
    printf("%s\n", cudaGetErrorString(cudaGetLastError()));
    return 0;
}
