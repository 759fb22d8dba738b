// Micro-benchmark (stand-alone, not part of the library): gather bandwidth from DRAM as a function of the contiguous
// piece read per row.  65 536 rows of 8 KB (4096 bf16, 512 MB), row order random; a CTA walks tiles of 128 rows and reads
// PIECE bytes of each row per step with plain 16-byte loads.  Question: do the 128-byte row pieces of a 64-column chunk
// under-use DRAM pages?
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o gather_piece gather_piece.cu && ./gather_piece
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <algorithm>
#include <random>
#include <cuda_runtime.h>
template <int PIECE>
__global__ void __launch_bounds__(512, 2) gather(const uint4* __restrict__ x, const int* __restrict__ perm, int tiles, int row_u4, unsigned* sink)
{
    // thread t: lanes of PIECE/16 consecutive threads cover one row piece; 512 threads cover 512*16/PIECE rows per pass
    constexpr int TPR = PIECE / 16;              // threads per row piece
    constexpr int ROWS_PER_PASS = 512 / TPR;
    constexpr int PASSES = 128 / ROWS_PER_PASS > 0 ? 128 / ROWS_PER_PASS : 1;
    unsigned acc = 0;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        int rows[PASSES];
#pragma unroll
        for (int p = 0; p < PASSES; ++p) rows[p] = perm[tile * 128 + (p * ROWS_PER_PASS + threadIdx.x / TPR) % 128];
        for (int c = 0; c < row_u4 / TPR; c += 2) {
            uint4 v[PASSES * 2];
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                v[2 * p] = __ldcs(x + (size_t)rows[p] * row_u4 + c * TPR + threadIdx.x % TPR);
                v[2 * p + 1] = __ldcs(x + (size_t)rows[p] * row_u4 + (c + 1) * TPR + threadIdx.x % TPR);
            }
#pragma unroll
            for (int p = 0; p < PASSES * 2; ++p) acc ^= v[p].x ^ v[p].w;
        }
    }
    if (acc == 0x12345678u) *sink = acc;
}
template <int PIECE>
float run(const uint4* x, const int* perm, int tiles, int row_u4, unsigned* sink)
{
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    gather<PIECE><<<296, 512>>>(x, perm, tiles, row_u4, sink);
    cudaEventRecord(e0);
    gather<PIECE><<<296, 512>>>(x, perm, tiles, row_u4, sink);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1); return ms;
}
int main()
{
    const int N = 65536, row_bytes = 8192, row_u4 = row_bytes / 16;
    uint4* x; cudaMalloc(&x, (size_t)N * row_bytes); cudaMemset(x, 1, (size_t)N * row_bytes);
    std::vector<int> perm(N); for (int i = 0; i < N; ++i) perm[i] = i;
    std::mt19937 g(1); std::shuffle(perm.begin(), perm.end(), g);
    int* dperm; cudaMalloc(&dperm, N * 4); cudaMemcpy(dperm, perm.data(), N * 4, cudaMemcpyHostToDevice);
    unsigned* sink; cudaMalloc(&sink, 4);
    const double bytes = (double)N * row_bytes;
    float ms;
    ms = run<64>(x, dperm, N / 128, row_u4, sink);   printf("piece   64 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    ms = run<128>(x, dperm, N / 128, row_u4, sink);  printf("piece  128 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    ms = run<256>(x, dperm, N / 128, row_u4, sink);  printf("piece  256 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    ms = run<512>(x, dperm, N / 128, row_u4, sink);  printf("piece  512 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    ms = run<1024>(x, dperm, N / 128, row_u4, sink); printf("piece 1024 B: %.3f ms  %.0f GB/s\n", ms, bytes / ms / 1e6);
    printf("%s\n", cudaGetErrorString(cudaGetLastError()));
    return 0;
}
