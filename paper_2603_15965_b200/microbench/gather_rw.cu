// Micro-benchmark (stand-alone, not part of the library): what DRAM delivers for the apply's access pattern -- gathered row
// pieces of two arrays read and one written back (2 reads : 1 write, like x and y in, y out), rows of 8 KB in random order,
// PIECE contiguous bytes per row and step, plain 16-byte loads and stores with ample parallelism.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o gather_rw gather_rw.cu && ./gather_rw
#include <cstdio>
#include <vector>
#include <algorithm>
#include <random>
#include <cuda_runtime.h>
template <int PIECE>
__global__ void __launch_bounds__(512, 2) rw(const uint4* __restrict__ x, uint4* __restrict__ y, const int* __restrict__ perm, int tiles, int row_u4)
{
    constexpr int TPR = PIECE / 16, ROWS_PER_PASS = 512 / TPR, PASSES = 128 / ROWS_PER_PASS;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        int rows[PASSES];
#pragma unroll
        for (int p = 0; p < PASSES; ++p) rows[p] = perm[tile * 128 + p * ROWS_PER_PASS + threadIdx.x / TPR];
        for (int c = 0; c < row_u4 / TPR; ++c) {
            uint4 a[PASSES], b[PASSES];
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const size_t o = (size_t)rows[p] * row_u4 + c * TPR + threadIdx.x % TPR;
                a[p] = __ldcs(x + o);
                b[p] = __ldcs(y + o);
            }
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const size_t o = (size_t)rows[p] * row_u4 + c * TPR + threadIdx.x % TPR;
                uint4 v = make_uint4(a[p].x + b[p].x, a[p].y + b[p].y, a[p].z + b[p].z, a[p].w + b[p].w);
                __stcs(y + o, v);
            }
        }
    }
}
template <int PIECE>
float run(const uint4* x, uint4* y, const int* perm, int tiles, int row_u4)
{
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    rw<PIECE><<<296, 512>>>(x, y, perm, tiles, row_u4);
    cudaEventRecord(e0);
    rw<PIECE><<<296, 512>>>(x, y, perm, tiles, row_u4);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1); return ms;
}
int main()
{
    const int N = 32768, row_bytes = 8192, row_u4 = row_bytes / 16;
    uint4 *x, *y; cudaMalloc(&x, (size_t)N * row_bytes); cudaMalloc(&y, (size_t)N * row_bytes);
    cudaMemset(x, 1, (size_t)N * row_bytes); cudaMemset(y, 2, (size_t)N * row_bytes);
    std::vector<int> perm(N); for (int i = 0; i < N; ++i) perm[i] = i;
    std::mt19937 g(1); std::shuffle(perm.begin(), perm.end(), g);
    int* dperm; cudaMalloc(&dperm, N * 4); cudaMemcpy(dperm, perm.data(), N * 4, cudaMemcpyHostToDevice);
    const double bytes = 3.0 * (double)N * row_bytes;
    float ms;
    ms = run<128>(x, y, dperm, N / 128, row_u4);  printf("piece  128 B: %.3f ms  %.0f GB/s (2 reads + 1 write)\n", ms, bytes / ms / 1e6);
    ms = run<256>(x, y, dperm, N / 128, row_u4);  printf("piece  256 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    printf("%s\n", cudaGetErrorString(cudaGetLastError()));
    return 0;
}
