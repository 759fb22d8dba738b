// The paper's learned router (Eq. 9): g(x) = W2 GELU(W1 x + b1) + b2, hidden width H = 64 (or up to 128), followed by
// top-1 selection as in the linear gate (lowest index on ties).
//
// The first layer is a dense contraction [N, d] x [d, H] and runs on the 5th-generation tensor cores for bf16
// activations (d a multiple of 64): one CTA owns 128 consecutive tokens, x chunks [128, 64] arrive by 2-D TMA into the
// 128-byte-swizzled K-major layout, W1 (fp32 in the interface) is split by a preparation kernel into three bf16 terms
// hi + mid + lo per value and written as K-major operand images [3*HP rows (term, hidden unit)][64 k] per chunk, and
// tcgen05.mma (M = 128, N = 192, K = 16) accumulates the three terms in separate TMEM columns over all of d.  The
// products are exact in fp32 and the epilogue adds (lo + mid) + hi, so the pre-activations have the accuracy of an
// fp32 FMA chain.  The epilogue (one thread per token) walks the hidden units in slices of 16 TMEM columns: bias,
// exact GELU 0.5 t (1 + erf(t / sqrt 2)), and the second layer as FMAs against W2 held in shared memory; then the
// output bias and the argmax.  The hidden activations never leave the SM.
//
// Other inputs (fp32 activations, d not a multiple of 64, H not a multiple of 16) take a CUDA-core kernel: one warp
// per token, lanes split d, HP partial pre-activations per lane, butterfly sums, GELU and the second layer in lanes.
//
// Warp roles of the tensor-core kernel (192 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps
// 2-5 epilogue.  Waits are bounded as in the apply kernel.
#include <algorithm>

#include "common.cuh"
#include "gate_image.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"
#include "warp_reduce.cuh"

namespace molora {

using namespace ptx;

constexpr int kMlpThreads = 192;
constexpr int kMlpTileBytes = 128 * 128;          // x chunk: 128 tokens x 64 bf16
constexpr int kMlpMaxC = 32;

struct MlpParams {
    CUtensorMap tm_x, tm_w;
    const float* b1;
    const float* W2;
    const float* b2;
    int32_t* r_out;
    float* logits_out;
    uint32_t* dev_status;
    int64_t N;
    int32_t d, H, C;
};

struct MlpCtrl {
    uint64_t full[6], empty[6], done;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ float gelu_exact(float t) { return 0.5f * t * (1.f + erff(t * 0.70710678118654752f)); }

// HP: padded hidden width, 64 or 128
template <int HP>
__global__ void __launch_bounds__(kMlpThreads, 1) route_mlp_umma_kernel(const __grid_constant__ MlpParams prm)
{
    constexpr int NP = 3 * HP;                      // accumulator columns: three term blocks of HP hidden units
    constexpr int WBYTES = NP * 128;                // W1 image of one chunk
    constexpr int STAGE = kMlpTileBytes + WBYTES;
    constexpr int STAGES = HP == 64 ? 5 : 3;
    constexpr int NMMA = NP / 192;                  // MMAs of N = 192 per k step
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    MlpCtrl* ctrl = reinterpret_cast<MlpCtrl*>(smem_raw + (base + STAGES * STAGE - raw));
    float* w2s = reinterpret_cast<float*>(smem_raw + (base + STAGES * STAGE + 256 - raw));   // [HP][C], then b1[HP]
    float* b1s = w2s + HP * kMlpMaxC;
    volatile int* abort_flag = &ctrl->abort_flag;
    auto stage = [&](int s) { return base + (uint32_t)s * STAGE; };
    auto bar = [&](const uint64_t* b) { return smem_u32(b); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int chunks = prm.d / 64;
    const int64_t tok0 = (int64_t)blockIdx.x * 128;

    if (tid == 0) {
        prefetch_tensormap(&prm.tm_x);
        prefetch_tensormap(&prm.tm_w);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(&ctrl->full[s]), 1);
            mbar_init(bar(&ctrl->empty[s]), 1);
        }
        mbar_init(bar(&ctrl->done), 1);
        ctrl->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), 512);
        tmem_relinquish();
    }
    // second-layer weights and first-layer bias on chip (rows of hidden units that do not exist are zero)
    for (int e = tid; e < HP * prm.C; e += kMlpThreads) {
        const int j = e / prm.C, c = e - j * prm.C;
        w2s[j * kMlpMaxC + c] = j < prm.H ? __ldg(prm.W2 + (int64_t)j * prm.C + c) : 0.f;
    }
    for (int j = tid; j < HP; j += kMlpThreads) b1s[j] = (prm.b1 != nullptr && j < prm.H) ? __ldg(prm.b1 + j) : 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 1;
            bool images_ready = false;
            for (int kc = 0; kc < chunks; ++kc) {
                wait_bar(bar(&ctrl->empty[s]), ph, abort_flag, prm.dev_status);
                if (*abort_flag) break;
                const uint32_t fb = bar(&ctrl->full[s]);
                mbar_arrive_expect_tx(fb, (uint32_t)STAGE);
                tma_load_2d(stage(s), &prm.tm_x, kc * 64, (int)tok0, fb);          // rows past N are zero-filled
                if (!images_ready) {           // the preparation kernel (previous launch) has completed and flushed
                    grid_dependency_sync();
                    images_ready = true;
                }
#pragma unroll
                for (int h2 = 0; h2 < NMMA; ++h2)
                    tma_load_2d(stage(s) + kMlpTileBytes + h2 * 192 * 128, &prm.tm_w, 0, kc * NP + h2 * 192, fb);
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(128, 192, 0, 0);              // both operands K-major
            constexpr uint32_t kL128 = swizzle_layout_type(Swizzle::B128);
            int s = 0;
            uint32_t ph = 0;
            for (int kc = 0; kc < chunks; ++kc) {
                wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t a0 = stage(s), b0 = a0 + kMlpTileBytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int h2 = 0; h2 < NMMA; ++h2)
                            umma_bf16(tmem + 192u * h2, smem_desc(a0 + j * 32, 16, 1024, kL128),
                                      smem_desc(b0 + h2 * 192 * 128 + j * 32, 16, 1024, kL128), idesc, kc > 0 || j > 0);
                    umma_commit(bar(&ctrl->empty[s]));
                }
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!*abort_flag) umma_commit(bar(&ctrl->done));
        }
        __syncwarp();
    } else {
        // ============================================================ epilogue: thread = token
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
        wait_bar(bar(&ctrl->done), 0, abort_flag, prm.dev_status);
        tc_fence_after();
        float z[kMlpMaxC];
#pragma unroll
        for (int c = 0; c < kMlpMaxC; ++c) z[c] = 0.f;
        for (int j16 = 0; j16 < HP / 16; ++j16) {
            if (j16 * 16 >= prm.H) break;
            uint32_t hi[16], mid[16], lo[16];
            tmem_ld_x16(tmem + lane_addr + j16 * 16, hi);
            tmem_ld_x16(tmem + lane_addr + HP + j16 * 16, mid);
            tmem_ld_x16(tmem + lane_addr + 2 * HP + j16 * 16, lo);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 16; ++e) {
                const int j = j16 * 16 + e;
                const float t = (__uint_as_float(lo[e]) + __uint_as_float(mid[e])) + __uint_as_float(hi[e]) + b1s[j];
                const float h = gelu_exact(t);
                const float* w2 = w2s + j * kMlpMaxC;
#pragma unroll
                for (int c = 0; c < kMlpMaxC; ++c)
                    if (c < prm.C) z[c] = fmaf(h, w2[c], z[c]);
            }
        }
        const int64_t i = tok0 + row;
        if (i < prm.N && *abort_flag) prm.r_out[i] = -1;                // a wait ran out: the tile's tokens stay unrouted
        if (i < prm.N && !*abort_flag) {
            float best = 0.f;
            int arg = 0;
#pragma unroll
            for (int c = 0; c < kMlpMaxC; ++c) {
                if (c < prm.C) {
                    float v = z[c];
                    if (prm.b2 != nullptr) v += __ldg(prm.b2 + c);
                    if (prm.logits_out != nullptr) prm.logits_out[i * prm.C + c] = v;
                    if (c == 0 || v > best) { best = v; arg = c; }      // strict '>' keeps the lowest index on ties
                }
            }
            prm.r_out[i] = arg;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// ------------------------------------------------------------------------------------------------ CUDA-core kernel
// One warp per token; lane l takes the input features l, l + 32, ...; HP partial pre-activations per lane.
template <typename T, int HP>
__global__ void __launch_bounds__(128) route_mlp_simple_kernel(const T* __restrict__ x, int64_t N, int d, int64_t ldx,
                                                               const float* __restrict__ W1, const float* __restrict__ b1,
                                                               int H, const float* __restrict__ W2,
                                                               const float* __restrict__ b2, int C,
                                                               int32_t* __restrict__ r_out, float* __restrict__ logits_out)
{
    grid_dependency_sync();
    const int warp = threadIdx.x >> 5, lane = lane_id();
    const int64_t i = (int64_t)blockIdx.x * 4 + warp;
    if (i >= N) return;
    float acc[HP];
#pragma unroll
    for (int j = 0; j < HP; ++j) acc[j] = 0.f;
    for (int k = lane; k < d; k += 32) {
        float xv;
        if constexpr (sizeof(T) == 2) xv = __bfloat162float(x[i * ldx + k]); else xv = x[i * ldx + k];
        const float* w = W1 + (int64_t)k * H;
#pragma unroll
        for (int j = 0; j < HP; ++j)
            if (j < H) acc[j] = fmaf(xv, __ldg(w + j), acc[j]);
    }
    // butterfly sums: afterwards every lane holds every pre-activation; lane c finishes output c
    float zc = 0.f;
#pragma unroll
    for (int j = 0; j < HP; ++j) {
        if (j < H) {
            float t = acc[j];
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
            t += b1 != nullptr ? __ldg(b1 + j) : 0.f;
            const float h = gelu_exact(t);
            if (lane < C) zc = fmaf(h, __ldg(W2 + (int64_t)j * C + lane), zc);
        }
    }
    if (lane < C && b2 != nullptr) zc += __ldg(b2 + lane);
    if (lane < C && logits_out != nullptr) logits_out[i * C + lane] = zc;
    // argmax over lanes 0..C-1, lowest index on ties
    float best = lane < C ? zc : -INFINITY;
    int arg = lane < C ? lane : 0x7fffffff;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, off);
        const int oa = __shfl_xor_sync(0xFFFFFFFFu, arg, off);
        if (ob > best || (ob == best && oa < arg)) { best = ob; arg = oa; }
    }
    if (lane == 0) r_out[i] = arg;
}

// ------------------------------------------------------------------------------------------------ host side
static bool mlp_umma_eligible(molora_dtype_t xdt, int64_t N, int32_t d, int32_t H)
{
    return xdt == MOLORA_BF16 && (d % 64) == 0 && H >= 1 && H <= 128 && N >= 128;
}

size_t route_mlp_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t H)
{
    if (xdt != MOLORA_BF16 || (d % 64) != 0 || H > 128) return 0;
    return (size_t)d * 3 * (H <= 64 ? 64 : 128) * 2;           // the three-term images of W1
}

template <int HP>
static molora_status_t mlp_umma_launch(const void* x, int64_t N, int d, int64_t ldx, const float* W1, const float* b1, int H,
                                       const float* W2, const float* b2, int C, int32_t* r_out, float* logits_out, void* ws,
                                       uint32_t* dev_status, cudaStream_t s)
{
    constexpr int NP = 3 * HP;
    constexpr int STAGES = HP == 64 ? 5 : 3;
    constexpr int SMEM = 1024 + STAGES * (kMlpTileBytes + NP * 128) + 256 + (HP * kMlpMaxC + HP) * 4;
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(route_mlp_umma_kernel<HP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        configured = true;
    }
    __nv_bfloat16* img = static_cast<__nv_bfloat16*>(ws);
    MlpParams prm;
    if (!make_tensor_map_bf16_2d(&prm.tm_x, x, (uint64_t)d, (uint64_t)N, (uint64_t)ldx, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tensor_map_bf16_2d(&prm.tm_w, img, 64, (uint64_t)(d / 64) * NP, 64, 64, 192, CU_TENSOR_MAP_SWIZZLE_128B))
        return MOLORA_ERR_CUDA;
    prm.b1 = b1;
    prm.W2 = W2;
    prm.b2 = b2;
    prm.r_out = r_out;
    prm.logits_out = logits_out;
    prm.dev_status = dev_status;
    prm.N = N;
    prm.d = d;
    prm.H = H;
    prm.C = C;
    const int64_t elems = (int64_t)d * HP;
    if (launch_kernel(gate_umma_split_kernel<HP>, dim3((unsigned)std::min<int64_t>(ceil_div64(elems, 256), 148 * 4)), dim3(256),
                      0, s, 1, false, W1, d, H, img) != cudaSuccess)
        return MOLORA_ERR_CUDA;
    return cuda_ok(launch_kernel(route_mlp_umma_kernel<HP>, dim3((unsigned)ceil_div64(N, 128)), dim3(kMlpThreads), SMEM, s, 1,
                                 true, prm));
}

template <typename T>
static molora_status_t mlp_simple_launch(const void* x, int64_t N, int d, int64_t ldx, const float* W1, const float* b1,
                                         int H, const float* W2, const float* b2, int C, int32_t* r_out, float* logits_out,
                                         cudaStream_t s)
{
    const dim3 grid((unsigned)ceil_div64(N, 4));
    const T* xt = static_cast<const T*>(x);
    cudaError_t e;
    if (H <= 16) e = launch_kernel(route_mlp_simple_kernel<T, 16>, grid, dim3(128), 0, s, 1, false, xt, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out);
    else if (H <= 64) e = launch_kernel(route_mlp_simple_kernel<T, 64>, grid, dim3(128), 0, s, 1, false, xt, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out);
    else e = launch_kernel(route_mlp_simple_kernel<T, 128>, grid, dim3(128), 0, s, 1, false, xt, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out);
    return cuda_ok(e);
}

molora_status_t launch_route_mlp(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* W1,
                                 const float* b1, int32_t H, const float* W2, const float* b2, int32_t C, int32_t* r_out,
                                 float* logits_out, void* ws, size_t ws_bytes, uint32_t* dev_status, cudaStream_t s)
{
    if (N == 0) return MOLORA_OK;
    if (mlp_umma_eligible(xdt, N, d, H)) {
        if (ws == nullptr || ws_bytes < route_mlp_workspace_bytes(xdt, d, H) || !aligned16(ws)) return MOLORA_ERR_WORKSPACE;
        return H <= 64 ? mlp_umma_launch<64>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, ws, dev_status, s)
                       : mlp_umma_launch<128>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, ws, dev_status, s);
    }
    return xdt == MOLORA_BF16 ? mlp_simple_launch<__nv_bfloat16>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, s)
                              : mlp_simple_launch<float>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, s);
}

}  // namespace molora
