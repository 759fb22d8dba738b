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
// output bias and the argmax.  The hidden activations never leave the SM.  Calls with few tiles split the input
// dimension of a tile over a cluster of 2 or 4 CTAs (see SPLIT below): measured on B200, graph replay, both launches,
// 4096 tokens 2048 -> 64 -> 4: 25.8 -> 17.8 us; 2560 -> 128 -> 4: 47.6 -> 29.8 us; 256 tokens: 23.5 -> 16.0 us.
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
    uint64_t full[6], empty[6], done, parts;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ float gelu_exact(float t) { return 0.5f * t * (1.f + erff(t * 0.70710678118654752f)); }

// HP: padded hidden width, 64 or 128.
// SPLIT: the input dimension of a 128-token tile is split over a cluster of S = 2 or 4 CTAs (calls with so few tiles that
// the chunks a CTA walks, ~0.7 us each, set the time).  Every CTA accumulates its slice of d, turns the three terms into
// partial pre-activations (lo + mid) + hi, and sends the rows [128 o / S, 128 (o + 1) / S) to CTA o (asynchronous stores
// that count their bytes on o's barrier; its own rows go into its own slot); CTA o sums the S partials in rank order and
// finishes its 128 / S tokens -- bias, GELU, second layer, argmax -- with all four epilogue warps, each a slice of the
// hidden units.
template <int HP, bool SPLIT>
struct MlpCfg {
    static constexpr int NP = 3 * HP;
    static constexpr int STAGE = kMlpTileBytes + NP * 128;
    static constexpr int STAGES = SPLIT ? (HP == 64 ? 4 : 2) : (HP == 64 ? 5 : 3);
    static constexpr int RECV = SPLIT ? 128 * HP * 4 : 0;            // [S slots][HP / 4][128 / S tokens] float4
    static constexpr int SMEM = 1024 + STAGES * STAGE + 256 + (HP * kMlpMaxC + HP) * 4 + RECV;
};

template <int HP, bool SPLIT>
__global__ void __launch_bounds__(kMlpThreads, 1) route_mlp_umma_kernel(const __grid_constant__ MlpParams prm)
{
    using Cfg = MlpCfg<HP, SPLIT>;
    constexpr int NP = 3 * HP;                      // accumulator columns: three term blocks of HP hidden units
    constexpr int STAGE = Cfg::STAGE;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int NMMA = NP / 192;                  // MMAs of N = 192 per k step
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    MlpCtrl* ctrl = reinterpret_cast<MlpCtrl*>(smem_raw + (base + STAGES * STAGE - raw));
    float* w2s = reinterpret_cast<float*>(smem_raw + (base + STAGES * STAGE + 256 - raw));   // [HP][C], then b1[HP]
    float* b1s = w2s + HP * kMlpMaxC;
    float4* recv = reinterpret_cast<float4*>(b1s + HP);                                       // SPLIT only
    const uint32_t S = SPLIT ? cluster_nctarank() : 1u, crank = SPLIT ? cluster_ctarank() : 0u;
    volatile int* abort_flag = &ctrl->abort_flag;
    auto stage = [&](int s) { return base + (uint32_t)s * STAGE; };
    auto bar = [&](const uint64_t* b) { return smem_u32(b); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int all_chunks = prm.d / 64;
    const int kc0 = (int)(crank * all_chunks / S), kc1 = (int)((crank + 1) * all_chunks / S);   // my slice of d
    const int64_t tok0 = (int64_t)(blockIdx.x / S) * 128;

    if (tid == 0) {
        prefetch_tensormap(&prm.tm_x);
        prefetch_tensormap(&prm.tm_w);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(&ctrl->full[s]), 1);
            mbar_init(bar(&ctrl->empty[s]), 1);
        }
        mbar_init(bar(&ctrl->done), 1);
        mbar_init(bar(&ctrl->parts), 1);        // SPLIT: the peers' partial rows arrive as asynchronous stores counted in bytes
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
    // "I am running and my barriers are initialised": the matching wait comes right before the first store into a peer
    if (SPLIT) cluster_arrive_relaxed();
    const uint32_t tmem = ctrl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 1;
            bool images_ready = false;
            for (int kc = kc0; kc < kc1; ++kc) {
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
            for (int kc = kc0; kc < kc1; ++kc) {
                wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t a0 = stage(s), b0 = a0 + kMlpTileBytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int h2 = 0; h2 < NMMA; ++h2)
                            umma_bf16(tmem + 192u * h2, smem_desc(a0 + j * 32, 16, 1024, kL128),
                                      smem_desc(b0 + h2 * 192 * 128 + j * 32, 16, 1024, kL128), idesc, kc > kc0 || j > 0);
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
        if constexpr (SPLIT) {
            const int et = tid - 64;                               // 0..127 among the epilogue threads
            const int RO = 128 / (int)S;                           // tokens a CTA finishes
            const int owner = row / RO, tl = row - owner * RO;
            const int nj16 = (prm.H + 15) / 16;
            cluster_wait();                                        // every CTA of the cluster is running
            if (et == 0) mbar_arrive_expect_tx(bar(&ctrl->parts), (S - 1) * (uint32_t)(RO * nj16 * 16 * 4));
            {
                // my partial pre-activations, 16 hidden units at a time, to the slot `crank` of the row's owner
                const uint32_t slot = smem_u32(recv) + crank * (uint32_t)(RO * HP * 4);
                const uint32_t dst0 = (uint32_t)owner == crank ? slot : map_to_cta(slot, (uint32_t)owner);
                const uint32_t pb = map_to_cta(bar(&ctrl->parts), (uint32_t)owner);
                for (int j16 = 0; j16 < nj16; ++j16) {
                    uint32_t hi[16], mid[16], lo[16];
                    tmem_ld_x16(tmem + lane_addr + j16 * 16, hi);
                    tmem_ld_x16(tmem + lane_addr + HP + j16 * 16, mid);
                    tmem_ld_x16(tmem + lane_addr + 2 * HP + j16 * 16, lo);
                    tmem_wait_ld();
#pragma unroll
                    for (int e4 = 0; e4 < 4; ++e4) {
                        uint32_t pv[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            pv[e] = __float_as_uint((__uint_as_float(lo[4 * e4 + e]) + __uint_as_float(mid[4 * e4 + e])) +
                                                    __uint_as_float(hi[4 * e4 + e]));
                        const uint32_t a = dst0 + (uint32_t)((j16 * 4 + e4) * RO + tl) * 16u;
                        if ((uint32_t)owner == crank)
                            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(pv[0]), "r"(pv[1]), "r"(pv[2]), "r"(pv[3]) : "memory");
                        else
                            st_async_cluster_u32x4(a, pv[0], pv[1], pv[2], pv[3], pb);
                    }
                }
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");         // my CTA's own rows are in its slot
            wait_bar_cluster(bar(&ctrl->parts), 0, abort_flag, prm.dev_status);   // ... and the peers' partials of them
            // finish my RO tokens: thread (token tl2, part) takes a slice of the hidden units
            const int parts = 128 / RO, tl2 = et % RO, part = et / RO;
            const int hp = HP / parts;                             // hidden units per thread: 16 ... 64
            for (int j4 = part * hp / 4; j4 < (part + 1) * hp / 4; ++j4) {
                if (j4 * 4 >= nj16 * 16) break;
                float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
                for (uint32_t r2 = 0; r2 < S; ++r2) {                                   // rank order
                    const float4 v = recv[(size_t)r2 * (RO * HP / 4) + (size_t)j4 * RO + tl2];
                    t.x += v.x;
                    t.y += v.y;
                    t.z += v.z;
                    t.w += v.w;
                }
                const float tt[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int j = j4 * 4 + e;
                    const float h = gelu_exact(tt[e] + b1s[j]);
                    const float* w2 = w2s + j * kMlpMaxC;
#pragma unroll
                    for (int c = 0; c < kMlpMaxC; ++c)
                        if (c < prm.C) z[c] = fmaf(h, w2[c], z[c]);
                }
            }
            // the parts of a token meet in the (now idle) ring: [part][token][adapter]
            float* zbuf = reinterpret_cast<float*>(smem_raw + (base - raw));
#pragma unroll
            for (int c = 0; c < kMlpMaxC; ++c)
                if (c < prm.C) zbuf[(part * RO + tl2) * kMlpMaxC + c] = z[c];
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (part == 0) {
                const int64_t i = tok0 + (int64_t)crank * RO + tl2;
                if (i < prm.N && *abort_flag) prm.r_out[i] = -1;        // a wait ran out: the tile's tokens stay unrouted
                if (i < prm.N && !*abort_flag) {
                    float best = 0.f;
                    int arg = 0;
                    for (int c = 0; c < prm.C; ++c) {
                        float v = 0.f;
                        for (int p2 = 0; p2 < parts; ++p2) v += zbuf[(p2 * RO + tl2) * kMlpMaxC + c];
                        if (prm.b2 != nullptr) v += __ldg(prm.b2 + c);
                        if (prm.logits_out != nullptr) prm.logits_out[i * prm.C + c] = v;
                        if (c == 0 || v > best) { best = v; arg = c; }   // strict '>' keeps the lowest index on ties
                    }
                    prm.r_out[i] = arg;
                }
            }
        } else {
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
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 512);
    if constexpr (SPLIT) {
        // the warps that took no part in the exchange complete the start-up barrier; one closing barrier keeps every CTA
        // alive until the stores addressed to it have been issued and taken
        if (warp < 2) cluster_wait();
        cluster_sync_all();
    }
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
                                       uint32_t* dev_status, cudaStream_t s, int image)
{
    constexpr int NP = 3 * HP;
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(route_mlp_umma_kernel<HP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 MlpCfg<HP, false>::SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(route_mlp_umma_kernel<HP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 MlpCfg<HP, true>::SMEM) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        configured = true;
    }
    // CTAs per 128-token tile (split along d) while the tiles alone leave most SMs idle; at least four chunks each
    const int64_t tiles = ceil_div64(N, 128);
    unsigned split = 1;
    if (tiles * 4 <= 148 && d / 64 / 4 >= 4) split = 4;
    else if (tiles * 2 <= 148 && d / 64 / 2 >= 4) split = 2;
    __nv_bfloat16* img = static_cast<__nv_bfloat16*>(ws);
    {
        const int64_t elems = (int64_t)d * HP;
        if (image != kImageUseOnly &&
            launch_kernel(gate_umma_split_kernel<HP>, dim3((unsigned)std::min<int64_t>(ceil_div64(elems, 256), 148 * 4)), dim3(256),
                          0, s, 1, false, W1, d, H, img) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        if (image == kImageBuildOnly) return MOLORA_OK;
    }
    const bool chained = image == kImageBuildAndUse;       // overlap with the tail of the preparation kernel
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
    if (split > 1)
        return cuda_ok(launch_kernel(route_mlp_umma_kernel<HP, true>, dim3((unsigned)tiles * split), dim3(kMlpThreads),
                                     MlpCfg<HP, true>::SMEM, s, split, chained, prm));
    return cuda_ok(launch_kernel(route_mlp_umma_kernel<HP, false>, dim3((unsigned)tiles), dim3(kMlpThreads),
                                 MlpCfg<HP, false>::SMEM, s, 1, chained, prm));
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
                                 float* logits_out, void* ws, size_t ws_bytes, uint32_t* dev_status, cudaStream_t s, int image)
{
    if (N == 0 && image != kImageBuildOnly) return MOLORA_OK;
    if (mlp_umma_eligible(xdt, image == kImageBuildOnly ? 128 : N, d, H)) {
        if (ws == nullptr || ws_bytes < route_mlp_workspace_bytes(xdt, d, H) || !aligned16(ws)) return MOLORA_ERR_WORKSPACE;
        return H <= 64 ? mlp_umma_launch<64>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, ws, dev_status, s, image)
                       : mlp_umma_launch<128>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, ws, dev_status, s, image);
    }
    if (image == kImageBuildOnly) return MOLORA_OK;          // the CUDA-core router reads W1 as it is
    return xdt == MOLORA_BF16 ? mlp_simple_launch<__nv_bfloat16>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, s)
                              : mlp_simple_launch<float>(x, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, s);
}

}  // namespace molora
