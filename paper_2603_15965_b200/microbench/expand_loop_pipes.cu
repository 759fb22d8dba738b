// Micro-benchmark behind the small-tile apply kernels' design notes: the expand inner loop (y += t B_c on a staged
// 16-row x 1024-column chunk, rank 16, bf16 hi + lo split of t) on data that already sits in shared memory, for
// 4 / 8 / 16 warps and one or two 32-column groups per step, and a variant that moves y with ldmatrix / stmatrix.
// It shows what bounds a chunk once its bytes have arrived: cycles per chunk ~ shared-memory wavefronts (768) + tensor
// pipe (256 MMAs x 2 cycles), i.e. the two pipes do not overlap with so few warps.  Not part of the library.
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -o expand_loop_pipes expand_loop_pipes.cu && ./expand_loop_pipes
#include <cstdio>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
__device__ __forceinline__ void mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void stsm(uint32_t addr, const uint32_t (&r)[4])
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}
__device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pk(float a, float b) { __nv_bfloat162 v = __floats2bfloat162_rn(a, b); return *reinterpret_cast<uint32_t*>(&v); }
constexpr int R = 16, KB = 1, ROWS = 16, TP = R * 2 + 16, DATA = 66048;
template <int VARIANT, int PARTS = 7, int NW = 8>
__global__ void __launch_bounds__(NW * 32, 1) k(long long* cyc, int nc, int iters, float* sink)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < (DATA + 2048) / 4; i += NW * 32) ((uint32_t*)dsm)[i] = 0x3c003c00u + i % 7;
    __syncthreads();
    const uint32_t sb = (uint32_t)__cvta_generic_to_shared(dsm);
    unsigned char* sp = dsm;
    const uint32_t pitch = nc * 2 + 16;
    const int g4 = lane >> 2, q = lane & 3, mi = lane >> 3;
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        const uint32_t tb = sb + DATA;
        uint32_t thi[KB][4], tlo[KB][4];
        for (int kb = 0; kb < KB; ++kb) {
            ldsm(thi[kb], tb + (lane & 15) * TP + (kb * 16 + (lane >> 4) * 8) * 2);
            ldsm(tlo[kb], tb + (ROWS + (lane & 15)) * TP + (kb * 16 + (lane >> 4) * 8) * 2);
        }
        constexpr int GI = VARIANT == 2 ? 4 : VARIANT == 3 ? 1 : 2;
        const int ngroups = nc / 32;
        unsigned char* yp = sp + g4 * pitch + q * 4;
        const uint32_t ba = sb + (ROWS + (mi & 1) * 8 + (lane & 7)) * pitch + (mi >> 1) * 16;
        for (int grp0 = warp; grp0 < ngroups; grp0 += GI * NW) {
            uint32_t yv[GI][2][4] = {}, bf[GI][KB][2][4] = {};
            float d[GI][4][4];
#pragma unroll
            for (int gi = 0; gi < GI; ++gi) {
                const int grp = grp0 + gi * NW;
                if ((PARTS & 1) && (VARIANT == 1 || grp < ngroups)) {
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int p2 = 0; p2 < 2; ++p2) ldsm_t(bf[gi][kb][p2], ba + kb * 16 * pitch + (grp * 32 + p2 * 16) * 2);
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) yv[gi][h][nt] = *reinterpret_cast<const uint32_t*>(yp + h * 8 * pitch + (grp * 32 + nt * 8) * 2);
                }
            }
#pragma unroll
            for (int gi = 0; gi < GI; ++gi) {
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) d[gi][nt][i] = 0.f;
                const int grp = grp0 + gi * NW;
                if ((PARTS & 2) && (VARIANT == 1 || grp < ngroups)) {
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int p2 = 0; p2 < 2; ++p2) {
                            mma(d[gi][2 * p2], thi[kb], bf[gi][kb][p2][0], bf[gi][kb][p2][1]);
                            mma(d[gi][2 * p2 + 1], thi[kb], bf[gi][kb][p2][2], bf[gi][kb][p2][3]);
                        }
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int p2 = 0; p2 < 2; ++p2) {
                            mma(d[gi][2 * p2], tlo[kb], bf[gi][kb][p2][0], bf[gi][kb][p2][1]);
                            mma(d[gi][2 * p2 + 1], tlo[kb], bf[gi][kb][p2][2], bf[gi][kb][p2][3]);
                        }
                }
            }
#pragma unroll
            for (int gi = 0; gi < GI; ++gi) {
                const int grp = grp0 + gi * NW;
                if ((PARTS & 4) && (VARIANT == 1 || grp < ngroups)) {
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) {
                            const uint32_t v = yv[gi][h][nt];
                            *reinterpret_cast<uint32_t*>(yp + h * 8 * pitch + (grp * 32 + nt * 8) * 2) = pk(lo(v) + d[gi][nt][2 * h], hi(v) + d[gi][nt][2 * h + 1]);
                        }
                }
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(NW * 32) : "memory");
    }
    long long t1 = clock64();
    if (tid == 0) cyc[0] = t1 - t0;
    if (sink) { float a = 0; for (int i = tid; i < DATA / 4; i += NW * 32) a += (float)(((uint32_t*)dsm)[i] & 0xffff); sink[tid] = a; }
}

// variant 3: y through ldmatrix / stmatrix (accumulator layout), one 32-column group per step, loads of the next step
// issued before the MMAs of this one
__global__ void __launch_bounds__(256, 1) k3(long long* cyc, int nc, int iters, float* sink)
{
    extern __shared__ __align__(128) unsigned char dsm[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i < (DATA + 2048) / 4; i += 256) ((uint32_t*)dsm)[i] = 0x3c003c00u + i % 7;
    __syncthreads();
    const uint32_t sb = (uint32_t)__cvta_generic_to_shared(dsm);
    const uint32_t pitch = nc * 2 + 16;
    const int mi = lane >> 3;
    long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        const uint32_t tb = sb + DATA;
        uint32_t thi[4], tlo[4];
        ldsm(thi, tb + (lane & 15) * TP + ((lane >> 4) * 8) * 2);
        ldsm(tlo, tb + (ROWS + (lane & 15)) * TP + ((lane >> 4) * 8) * 2);
        const int ngroups = nc / 32;
        const uint32_t ya = sb + ((lane & 7) + 8 * (mi & 1)) * pitch + (mi >> 1) * 16;       // y: rows via matrices 0/1, cols via 2/3
        const uint32_t ba = sb + (ROWS + (mi & 1) * 8 + (lane & 7)) * pitch + (mi >> 1) * 16;
        uint32_t y[2][2][4], bf[2][2][4];
        int grp = warp;
        if (grp < ngroups) {
#pragma unroll
            for (int p2 = 0; p2 < 2; ++p2) { ldsm_t(bf[0][p2], ba + (grp * 32 + p2 * 16) * 2); ldsm(y[0][p2], ya + (grp * 32 + p2 * 16) * 2); }
        }
        int cur = 0;
        for (; grp < ngroups; grp += 8, cur ^= 1) {
            const int nxt = grp + 8;
            if (nxt < ngroups) {
#pragma unroll
                for (int p2 = 0; p2 < 2; ++p2) {
                    if (cur == 0) { ldsm_t(bf[1][p2], ba + (nxt * 32 + p2 * 16) * 2); ldsm(y[1][p2], ya + (nxt * 32 + p2 * 16) * 2); }
                    else { ldsm_t(bf[0][p2], ba + (nxt * 32 + p2 * 16) * 2); ldsm(y[0][p2], ya + (nxt * 32 + p2 * 16) * 2); }
                }
            }
            float d[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) d[nt][i] = 0.f;
#pragma unroll
            for (int p2 = 0; p2 < 2; ++p2) {
                const uint32_t (&b)[4] = cur == 0 ? bf[0][p2] : bf[1][p2];
                mma(d[2 * p2], thi, b[0], b[1]);
                mma(d[2 * p2 + 1], thi, b[2], b[3]);
            }
#pragma unroll
            for (int p2 = 0; p2 < 2; ++p2) {
                const uint32_t (&b)[4] = cur == 0 ? bf[0][p2] : bf[1][p2];
                mma(d[2 * p2], tlo, b[0], b[1]);
                mma(d[2 * p2 + 1], tlo, b[2], b[3]);
            }
#pragma unroll
            for (int p2 = 0; p2 < 2; ++p2) {
                const uint32_t (&yv)[4] = cur == 0 ? y[0][p2] : y[1][p2];
                uint32_t o[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {     // register j: n8 tile 2*p2 + (j >> 1), rows g4 + 8 * (j & 1)
                    const int nt = 2 * p2 + (j >> 1), h = j & 1;
                    o[j] = pk(lo(yv[j]) + d[nt][2 * h], hi(yv[j]) + d[nt][2 * h + 1]);
                }
                stsm(ya + (grp * 32 + p2 * 16) * 2, o);
            }
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");
    }
    long long t1 = clock64();
    if (tid == 0) cyc[0] = t1 - t0;
    if (sink) { float a = 0; for (int i = tid; i < DATA / 4; i += 256) a += (float)(((uint32_t*)dsm)[i] & 0xffff); sink[tid] = a; }
}
int main()
{
    long long* cyc; cudaMalloc(&cyc, 64); long long h;
    const int smem = DATA + 2048;
    auto run = [&](auto kern, const char* name, int nc, int threads = 256) {
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        kern<<<1, threads, smem>>>(cyc, nc, 200, nullptr); cudaDeviceSynchronize();
        kern<<<1, threads, smem>>>(cyc, nc, 200, nullptr); cudaDeviceSynchronize();
        cudaMemcpy(&h, cyc, 8, cudaMemcpyDeviceToHost);
        printf("%s nc=%d: %.0f cycles per job (%s)\n", name, nc, (double)h / 200, cudaGetErrorString(cudaGetLastError()));
    };
    run(k<0, 1>, "loads only", 1024); run(k<0, 2>, "mma only", 1024); run(k<0, 4>, "epilogue only", 1024); run(k<0, 3>, "loads+mma", 1024); run(k<0, 5>, "loads+epilogue", 1024); run(k<0, 6>, "mma+epilogue", 1024);
    run(k<0>, "GI=2 guarded", 1024); run(k<0, 7, 16>, "GI=2, 16 warps", 1024, 512); run(k<3, 7, 16>, "GI=1, 16 warps", 1024, 512); run(k<3, 7, 8>, "GI=1, 8 warps", 1024, 256); run(k<3, 7, 4>, "GI=1, 4 warps", 1024, 128);
    run(k3, "ldsm/stsm pipelined", 1024); run(k3, "ldsm/stsm pipelined", 512);
    // same result?  (one iteration each from the same initial contents)
    float *s0, *s3; cudaMalloc(&s0, 1024); cudaMalloc(&s3, 1024); float h0[256], h3[256];
    k<0><<<1, 256, smem>>>(cyc, 1024, 1, s0); k3<<<1, 256, smem>>>(cyc, 1024, 1, s3); cudaDeviceSynchronize();
    cudaMemcpy(h0, s0, 1024, cudaMemcpyDeviceToHost); cudaMemcpy(h3, s3, 1024, cudaMemcpyDeviceToHost);
    int same = 1; for (int i = 0; i < 256; ++i) same &= h0[i] == h3[i];
    printf("checksums equal: %d (%f %f)\n", same, h0[0], h3[0]);
    return 0;
}
