// Linear gate with top-1 argmax (Eq. 8, k = 1) for bf16 activations: z = x G on the warp-level tensor cores.
//
// The gate is a [N, d] x [d, C] product with a tiny C, so its cost is streaming x once (N*d*2 bytes); on CUDA
// cores the N*d*C fp32 FMAs would cost more than that stream for C = 16 (Theorem 3.4's O(E*d) routing cost).
// G stays fp32 in the interface.  Inside the kernel every G value is split into three bf16 terms
// hi + mid + lo (24 mantissa bits in total), each bf16 x bf16 product is exact in fp32, and the three
// mma.sync.m16n8k16 products accumulate into one fp32 fragment -- the same accuracy class as an fp32 FMA chain.
//
// Layout.  One warp owns 16 tokens.  A thread (g = lane / 4, q = lane % 4) feeds rows g and g + 8 of the A
// fragment straight from global memory with 16-byte loads: the 8 contiguous elements at k = 32 b + 8 q serve two
// k-steps (4 each), i.e. the k order inside a 32-block is permuted -- harmless for a dot product as long as
// the B fragments use the same permutation.  The split G chunk lives in shared memory as [term][c][k'], with
// k' already in that permuted order, so a B fragment pair (b0, b1) is one 64-bit load.  The split is done
// once per call by a small preparation kernel that writes the exact shared-memory image of every k chunk into
// the caller's workspace; the gate CTAs then only copy images (cp.async, double buffered).
#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace molora {

constexpr int kGateRowPad = 16;              // bf16 elements of padding per (term, c) row: conflict-free B loads

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// position of memory k (offset inside a chunk) in the permuted order the fragments use
__device__ __forceinline__ int gate_kperm(int k)
{
    const int blk = k >> 5, r = k & 31;
    const int q = r >> 3, s = (r >> 2) & 1, e = r & 3;
    return blk * 32 + s * 16 + q * 4 + e;
}

template <int NT, int KC>
struct GateImage {                                  // one k chunk of split G as it sits in shared memory
    static constexpr int CP = NT * 8;
    static constexpr int ROW = KC + kGateRowPad;    // bf16 elements per (term, c) row
    static constexpr int kElems = 3 * CP * ROW;
    static constexpr int kBytes = kElems * 2;
};

// Preparation: fp32 G [d, C] -> chunk images [chunks][3 terms][CP][ROW] in bf16 (zero padded).
template <int NT, int KC>
__global__ void __launch_bounds__(256) gate_split_kernel(const float* __restrict__ G, int d, int C,
                                                         __nv_bfloat16* __restrict__ img)
{
    using Img = GateImage<NT, KC>;
    const int chunks = (d + KC - 1) / KC;
    const int64_t total = (int64_t)chunks * KC * Img::CP;
    ptx::grid_dependency_sync();     // an earlier gate call may still be reading the images this kernel rewrites
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(e % Img::CP);
        const int64_t k = e / Img::CP;
        const float v = (k < d && c < C) ? __ldg(G + k * C + c) : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        const float r1 = v - __bfloat162float(hi);
        const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
        const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
        const int ch = (int)(k / KC), kp = gate_kperm((int)(k % KC));
        __nv_bfloat16* base = img + (int64_t)ch * Img::kElems + c * Img::ROW + kp;
        base[0] = hi;
        base[Img::CP * Img::ROW] = mid;
        base[2 * Img::CP * Img::ROW] = lo;
    }
}

template <int NT, int WARPS, int KC>   // NT n-tiles of 8 adapters (C <= 8 NT); WARPS x 16 tokens per CTA; KC k per chunk
__global__ void __launch_bounds__(WARPS * 32) route_gate_mma_kernel(const __nv_bfloat16* __restrict__ x, int64_t N,
                                                                    int d, int64_t ldx,
                                                                    const __nv_bfloat16* __restrict__ img,
                                                                    const float* __restrict__ bias, int C,
                                                                    int32_t* __restrict__ r_out,
                                                                    float* __restrict__ logits_out)
{
    using Img = GateImage<NT, KC>;
    constexpr int CP = Img::CP, ROW = Img::ROW;
    constexpr int THREADS = WARPS * 32;
    constexpr int NB = KC / 32;                                      // 32-wide k blocks per chunk
    constexpr int IB = 3;                                            // weight-image buffers (two requests ahead)
    __shared__ __align__(16) __nv_bfloat16 Gs[IB][3][CP][ROW];        // [buffer][term][c][k']

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    ptx::grid_dependency_sync();     // the weight images come from gate_split_kernel
    const int g = lane >> 2, q = lane & 3;
    const int64_t tok0 = ((int64_t)blockIdx.x * WARPS + warp) * 16;
    const int64_t rowA = tok0 + g < N ? tok0 + g : N - 1;             // tail rows recompute the last token
    const int64_t rowB = tok0 + g + 8 < N ? tok0 + g + 8 : N - 1;
    const __nv_bfloat16* xa = x + rowA * ldx + q * 8;
    const __nv_bfloat16* xb = x + rowB * ldx + q * 8;

    // one accumulator fragment per (n-tile, term, k-step parity): independent MMA chains hide the MMA latency
    float acc3[NT][3][2][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int t = 0; t < 3; ++t)
#pragma unroll
            for (int s = 0; s < 2; ++s)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc3[n][t][s][i] = 0.f;

    const int chunks = (d + KC - 1) / KC;
    auto copy_image = [&](int buf, int ch) {
        const uint32_t dst = (uint32_t)__cvta_generic_to_shared(&Gs[buf][0][0][0]);
        const char* src = reinterpret_cast<const char*>(img + (int64_t)ch * Img::kElems);
        if (ch < chunks)
            for (int o = tid * 16; o < Img::kBytes; o += THREADS * 16)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + o), "l"(src + o) : "memory");
        asm volatile("cp.async.commit_group;" ::: "memory");         // an empty group keeps the group count uniform
    };

    // activations of one chunk: NB blocks of 32 k, two rows, 16 bytes each
    auto load_x = [&](uint4 (&va)[NB], uint4 (&vb)[NB], int k0) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const int k = k0 + b * 32 + q * 8;
            if (k < d) {
                va[b] = ldg128_stream(xa + k0 + b * 32);
                vb[b] = ldg128_stream(xb + k0 + b * 32);
            } else {
                va[b] = make_uint4(0, 0, 0, 0);
                vb[b] = make_uint4(0, 0, 0, 0);
            }
        }
    };

    // Software pipeline: the activations of kDepth - 1 chunks ahead and the next weight image are requested
    // before a chunk's math, so ~kDepth chunks (4 KB each per warp) are in flight.  The register ring is indexed
    // statically by unrolling the chunk loop kDepth times.
    constexpr int kDepth = 4;
    copy_image(0, 0);
    copy_image(1, 1);
    uint4 va[kDepth][NB], vb[kDepth][NB];
#pragma unroll
    for (int u = 0; u < kDepth - 1; ++u)
        if (u < chunks) load_x(va[u], vb[u], u * KC);
    for (int ch0 = 0; ch0 < chunks; ch0 += kDepth) {
#pragma unroll
        for (int u = 0; u < kDepth; ++u) {
            const int ch = ch0 + u;
            if (ch < chunks) {                                       // uniform over the CTA
                if (ch + kDepth - 1 < chunks)
                    load_x(va[(u + kDepth - 1) % kDepth], vb[(u + kDepth - 1) % kDepth], (ch + kDepth - 1) * KC);
                copy_image((ch + 2) % IB, ch + 2);                   // its buffer was released at the end of chunk ch - 1
                asm volatile("cp.async.wait_group 2;" ::: "memory");
                __syncthreads();                                     // image `ch` is complete for every thread
                const int buf = ch % IB;
#pragma unroll
                for (int b = 0; b < NB; ++b) {
#pragma unroll
                    for (int s = 0; s < 2; ++s) {
                        // A fragment of k-step (b, s): a0 = row g k-slots 2q,2q+1; a1 = row g+8; a2 = row g slots 2q+8,+9
                        uint32_t a[4];
                        a[0] = s ? va[u][b].z : va[u][b].x;
                        a[2] = s ? va[u][b].w : va[u][b].y;
                        a[1] = s ? vb[u][b].z : vb[u][b].x;
                        a[3] = s ? vb[u][b].w : vb[u][b].y;
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
#pragma unroll
                            for (int t = 0; t < 3; ++t) {
                                const uint2 bb =
                                    *reinterpret_cast<const uint2*>(&Gs[buf][t][n * 8 + g][b * 32 + s * 16 + q * 4]);
                                mma_bf16_16816(acc3[n][t][s], a, bb.x, bb.y);
                            }
                        }
                    }
                }
                __syncthreads();                                     // this buffer is refilled by the next iteration's request
            }
        }
    }

    // fold the partial fragments in a fixed order: ((lo + mid) + hi), even k-steps then odd
    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int i = 0; i < 4; ++i)
            acc[n][i] = ((acc3[n][2][0][i] + acc3[n][2][1][i]) + (acc3[n][1][0][i] + acc3[n][1][1][i])) +
                        (acc3[n][0][0][i] + acc3[n][0][1][i]);

    // fragment -> logits: acc[n][0..1] = (row g, c = 8n + 2q, +1), acc[n][2..3] = (row g + 8, same columns)
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int64_t i = tok0 + g + 8 * half;
        float best = 0.f;
        int arg = INT32_MAX;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int c = n * 8 + 2 * q + e;
                if (c < C) {
                    float z = acc[n][half * 2 + e];
                    if (bias != nullptr) z += __ldg(bias + c);
                    if (logits_out != nullptr && i < N) logits_out[i * C + c] = z;
                    if (arg == INT32_MAX || z > best) { best = z; arg = c; }   // ascending c: strict '>' keeps the lowest
                }
            }
        }
        // combine the four lanes of the quad; ties go to the lowest adapter index
#pragma unroll
        for (int off = 1; off <= 2; off <<= 1) {
            const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, off);
            const int oa = __shfl_xor_sync(0xFFFFFFFFu, arg, off);
            if (oa != INT32_MAX && (arg == INT32_MAX || ob > best || (ob == best && oa < arg))) { best = ob; arg = oa; }
        }
        if (q == 0 && i < N) r_out[i] = arg;
    }
}

template <int NT, int WARPS, int KC>
static molora_status_t gate_mma_launch(const void* x, int64_t N, int d, int64_t ldx, const float* G, const float* bias,
                                       int C, int32_t* r_out, float* logits_out, void* ws, cudaStream_t s, int image)
{
    __nv_bfloat16* img = static_cast<__nv_bfloat16*>(ws);
    const int chunks = (d + KC - 1) / KC;
    const int64_t elems = (int64_t)chunks * KC * NT * 8;
    if (image != kImageUseOnly) {
        if (cudaError_t e = launch_kernel(gate_split_kernel<NT, KC>,
                                          dim3((unsigned)std::min<int64_t>(ceil_div64(elems, 256), 148 * 4)), dim3(256), 0, s,
                                          1, false, G, d, C, img);
            e != cudaSuccess)
            return MOLORA_ERR_CUDA;
    }
    if (image == kImageBuildOnly) return MOLORA_OK;
    const int64_t blocks = ceil_div64(N, 16 * WARPS);
    return cuda_ok(launch_kernel(route_gate_mma_kernel<NT, WARPS, KC>, dim3((unsigned)blocks), dim3(WARPS * 32), 0, s, 1,
                                 image == kImageBuildAndUse,
                                  static_cast<const __nv_bfloat16*>(x), N, d, ldx, img, bias, C, r_out, logits_out));
}

size_t route_gate_mma_workspace_bytes(int32_t d, int32_t C)
{
    if (C <= 4) return 0;
    if (C <= 8) return (size_t)((d + 127) / 128) * GateImage<1, 128>::kBytes;
    if (C <= 16) return (size_t)((d + 127) / 128) * GateImage<2, 128>::kBytes;
    return (size_t)((d + 63) / 64) * GateImage<4, 64>::kBytes;
}

molora_status_t launch_route_gate_mma(const void* x, int64_t N, int32_t d, int64_t ldx, const float* G,
                                      const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                      cudaStream_t s, int image)
{
    if (N == 0 && image != kImageBuildOnly) return MOLORA_OK;
    if (C <= 8) return gate_mma_launch<1, 4, 128>(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, s, image);
    if (C <= 16) return gate_mma_launch<2, 4, 128>(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, s, image);
    return gate_mma_launch<4, 4, 64>(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, s, image);
}

}  // namespace molora

// ------------------------------------------------------------------------------------------------
// molora_route_gate_noalloc: the gate for callers that cannot hand the library a workspace.
//
// The split gate weights normally go to caller-provided scratch.  Here they go to a fixed array that is
// part of the library image: every GPU that loads the library holds these 2 MiB until the process exits.
// In host code the array's name is only a handle; the device address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and is what the kernels receive.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr size_t kNoAllocScratchBytes = 2u << 20;
static __device__ __align__(256) unsigned char g_gate_scratch[kNoAllocScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (looked up on the first call per device).
molora_status_t scratch_for_current_device(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MOLORA_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_gate_scratch) != cudaSuccess || p == nullptr) return MOLORA_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return MOLORA_OK;
}

}  // namespace

extern "C" molora_status_t molora_route_gate_noalloc(const void* x, molora_dtype_t xdt, int64_t N, int32_t d,
                                                     int64_t ldx, const float* G, const float* bias, int32_t C,
                                                     int32_t* r_out, float* logits_out, void* stream)
{
    if (d <= 0 || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (C > 32) return MOLORA_ERR_UNSUPPORTED;
    const size_t need = molora_route_gate_workspace_bytes(xdt, d, C);
    if (need > kNoAllocScratchBytes) return MOLORA_ERR_WORKSPACE;     // d * C too large for the built-in scratch
    void* scratch = nullptr;
    if (need > 0) {
        const molora_status_t st = scratch_for_current_device(&scratch);
        if (st != MOLORA_OK) return st;
    }
    return molora_route_gate(x, xdt, N, d, ldx, G, bias, C, r_out, logits_out, scratch, need > 0 ? kNoAllocScratchBytes : 0,
                             nullptr, stream);
}
