// Linear gate with top-1 argmax (Eq. 8, k = 1) on the 5th-generation tensor cores, for bf16 activations,
// more than four adapters and calls of at least 1024 tokens.
//
// z = x G is a [N, d] x [d, C] product with a tiny C: its cost is streaming x once.  One CTA owns 128
// consecutive tokens (rows of x are contiguous, so an x chunk [128, 64] is ONE 2-D TMA load into the
// 128-byte-swizzled K-major layout) and accumulates D[128, 3*CP] in TMEM over all of d with tcgen05.mma.
// G stays fp32 in the interface: a preparation kernel splits every value into three bf16 terms
// hi + mid + lo (24 mantissa bits) and writes, per 64-wide k chunk, the K-major operand image
// [3*CP rows (term, adapter)][64 k] into the workspace, so that the B operand of a chunk is one TMA load
// too.  bf16 x bf16 products are exact in fp32 and the three column blocks are summed in the epilogue
// ((lo + mid) + hi), the same accuracy class as an fp32 FMA chain.
//
// A call with few 128-token tiles is split over a cluster of S = 2 or 4 CTAs along d: rank q accumulates the q-th
// slice of the k chunks, ranks > 0 push their partial logits into rank 0's shared memory, one hardware cluster
// barrier (reached by every thread), and rank 0 adds the partials in rank order and finishes the tokens.
//
// Warp roles (192 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-5 epilogue (one
// thread per token: reads its TMEM lane, adds the terms and the bias, takes the argmax, lowest index on ties).
// Waits are bounded as in the apply kernel.
#include <algorithm>

#include "common.cuh"
#include "gate_image.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace molora {

using namespace ptx;

constexpr int kGuThreads = 192;
constexpr int kGuStages = 6;
constexpr int kGuTileBytes = 128 * 128;          // x chunk: 128 tokens x 64 bf16
constexpr int kGuMaxSplit = 4;

struct GateUmmaParams {
    CUtensorMap tm_x, tm_g;
    const float* bias;
    int32_t* r_out;
    float* logits_out;
    uint32_t* dev_status;
    int64_t N;
    int32_t d, C;
};

struct GateCtrl {
    uint64_t full[kGuStages], empty[kGuStages], done, parts;
    uint32_t tmem_base;
    int abort_flag;
};

template <int CP>
__global__ void __launch_bounds__(kGuThreads, 1) route_gate_umma_kernel(const __grid_constant__ GateUmmaParams prm)
{
    constexpr int NP = 3 * CP;                      // MMA N: three term blocks of CP adapters
    constexpr int GBYTES = NP * 128;                // G image of one chunk
    constexpr int STAGE = kGuTileBytes + GBYTES;
    constexpr int STAGES = CP == 16 ? kGuStages : kGuStages - 1;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    GateCtrl* ctrl = reinterpret_cast<GateCtrl*>(smem_raw + (base + STAGES * STAGE - raw));
    float* partials = reinterpret_cast<float*>(smem_raw + (base + STAGES * STAGE + 256 - raw));   // [S-1][NP][128]
    const uint32_t S = cluster_nctarank(), crank = cluster_ctarank();
    volatile int* abort_flag = &ctrl->abort_flag;
    auto stage = [&](int s) { return base + (uint32_t)s * STAGE; };
    auto bar = [&](const uint64_t* b) { return smem_u32(b); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int all_chunks = prm.d / 64;
    const int kc0 = (int)(crank * all_chunks / S), kc1 = (int)((crank + 1) * all_chunks / S);   // my slice of d
    const int64_t tok0 = (int64_t)(blockIdx.x / S) * 128;

    if (tid == 0) {
        prefetch_tensormap(&prm.tm_x);
        prefetch_tensormap(&prm.tm_g);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(&ctrl->full[s]), 1);
            mbar_init(bar(&ctrl->empty[s]), 1);
        }
        mbar_init(bar(&ctrl->done), 1);
        mbar_init(bar(&ctrl->parts), 1);       // rank 0: the peers' partial logits arrive as asynchronous stores counted in bytes
        ctrl->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), 128);      // NP <= 96 accumulator columns
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // "I am running and my barriers are initialised": the matching wait comes right before the first store into a peer
    if (S > 1) cluster_arrive_relaxed();
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
                tma_load_2d(stage(s) + kGuTileBytes, &prm.tm_g, 0, kc * NP, fb);
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(128, NP, 0, 0);               // both operands K-major
            constexpr uint32_t kL128 = swizzle_layout_type(Swizzle::B128);
            int s = 0;
            uint32_t ph = 0;
            for (int kc = kc0; kc < kc1; ++kc) {
                wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t a0 = stage(s), b0 = a0 + kGuTileBytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        umma_bf16(tmem, smem_desc(a0 + j * 32, 16, 1024, kL128), smem_desc(b0 + j * 32, 16, 1024, kL128),
                                  idesc, kc > kc0 || j > 0);
                    umma_commit(bar(&ctrl->empty[s]));
                }
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!*abort_flag) umma_commit(bar(&ctrl->done));
        }
        __syncwarp();
    }
    // every thread of every CTA of the cluster takes the same path from here on (the cluster barrier below)
    uint32_t v[NP];
    const int q = warp & 3;
    const int row = q * 32 + lane;
    const bool epi = warp >= 2;
    if (epi) {
        wait_bar(bar(&ctrl->done), 0, abort_flag, prm.dev_status);
        tc_fence_after();
#pragma unroll
        for (int c16 = 0; c16 < NP / 16; ++c16) tmem_ld_x16(tmem + ((uint32_t)(q * 32) << 16) + c16 * 16, v + c16 * 16);
        tmem_wait_ld();
        if (S > 1) {
            cluster_wait();          // every CTA of the cluster is running
            if (crank != 0) {
                // push my partial logits into rank 0's shared memory, slot crank - 1, as [NP / 4][128] 16-byte pieces; the
                // stores are asynchronous and count their bytes on rank 0's barrier (a warp's plain stores into a peer's
                // memory complete one after the other, ~0.14 us each)
                const uint32_t dst = map_to_cta(smem_u32(partials + (size_t)(crank - 1) * NP * 128) + (uint32_t)row * 16u, 0);
                const uint32_t pb = map_to_cta(bar(&ctrl->parts), 0);
#pragma unroll
                for (int c4 = 0; c4 < NP / 4; ++c4)
                    st_async_cluster_u32x4(dst + (uint32_t)c4 * 128u * 16u, v[4 * c4], v[4 * c4 + 1], v[4 * c4 + 2], v[4 * c4 + 3], pb);
            } else {
                if (warp == 2 && lane == 0) mbar_arrive_expect_tx(bar(&ctrl->parts), (S - 1) * (uint32_t)(NP * 128 * 4));
                wait_bar_cluster(bar(&ctrl->parts), 0, abort_flag, prm.dev_status);
            }
        }
    }
    if (epi && crank == 0) {
        const int64_t i = tok0 + row;
        if (i < prm.N && *abort_flag) prm.r_out[i] = -1;                // a wait ran out: the tile's tokens stay unrouted
        if (i < prm.N && !*abort_flag) {
            for (uint32_t p2 = 1; p2 < S; ++p2) {                       // rank order
                const float4* src = reinterpret_cast<const float4*>(partials + (size_t)(p2 - 1) * NP * 128) + row;
#pragma unroll
                for (int c4 = 0; c4 < NP / 4; ++c4) {
                    const float4 pv = src[c4 * 128];
                    v[4 * c4] = __float_as_uint(__uint_as_float(v[4 * c4]) + pv.x);
                    v[4 * c4 + 1] = __float_as_uint(__uint_as_float(v[4 * c4 + 1]) + pv.y);
                    v[4 * c4 + 2] = __float_as_uint(__uint_as_float(v[4 * c4 + 2]) + pv.z);
                    v[4 * c4 + 3] = __float_as_uint(__uint_as_float(v[4 * c4 + 3]) + pv.w);
                }
            }
            float best = 0.f;
            int arg = 0;
#pragma unroll
            for (int c = 0; c < CP; ++c) {
                if (c < prm.C) {
                    float z = (__uint_as_float(v[2 * CP + c]) + __uint_as_float(v[CP + c])) + __uint_as_float(v[c]);
                    if (prm.bias != nullptr) z += __ldg(prm.bias + c);
                    if (prm.logits_out != nullptr) prm.logits_out[i * prm.C + c] = z;
                    if (c == 0 || z > best) { best = z; arg = c; }      // strict '>' keeps the lowest index on ties
                }
            }
            prm.r_out[i] = arg;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, 128);
    if (S > 1) {
        // the warps that took no part in the exchange complete the start-up barrier; then one closing barrier keeps rank 0
        // alive until every peer's stores have been issued and the peers until rank 0 has taken them
        if (!epi) cluster_wait();
        cluster_sync_all();
    }
}

template <int CP>
static molora_status_t gate_umma_launch(const void* x, int64_t N, int d, int64_t ldx, const float* G, const float* bias,
                                        int C, int32_t* r_out, float* logits_out, void* ws, uint32_t* dev_status,
                                        cudaStream_t s, int image)
{
    constexpr int NP = 3 * CP;
    constexpr int STAGES = CP == 16 ? kGuStages : kGuStages - 1;
    // CTAs per 128-token tile (split along d): enough to put ~128 CTAs to work, at least 8 k chunks each
    int split = 1;
    const int64_t tiles = ceil_div64(N, 128);
    while (split < (CP == 16 ? kGuMaxSplit : 2) && tiles * split * 2 <= 148 && (d / 64) / (split * 2) >= 8) split *= 2;
    const int SMEM = 1024 + STAGES * (kGuTileBytes + NP * 128) + 256 + (kGuMaxSplit - 1) * NP * 128 * 4 * (CP == 16 ? 1 : 0) +
                     (CP == 16 ? 0 : NP * 128 * 4);
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        if (cudaFuncSetAttribute(route_gate_umma_kernel<CP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        configured = true;
    }
    __nv_bfloat16* img = static_cast<__nv_bfloat16*>(ws);
    const int64_t elems = (int64_t)d * CP;
    if (image != kImageUseOnly &&
        launch_kernel(gate_umma_split_kernel<CP>, dim3((unsigned)std::min<int64_t>(ceil_div64(elems, 256), 148 * 4)),
                      dim3(256), 0, s, 1, false, G, d, C, img) != cudaSuccess)
        return MOLORA_ERR_CUDA;
    if (image == kImageBuildOnly) return MOLORA_OK;
    GateUmmaParams prm;
    if (!make_tensor_map_bf16_2d(&prm.tm_x, x, (uint64_t)d, (uint64_t)N, (uint64_t)ldx, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_tensor_map_bf16_2d(&prm.tm_g, img, 64, (uint64_t)(d / 64) * NP, 64, 64, NP, CU_TENSOR_MAP_SWIZZLE_128B))
        return MOLORA_ERR_CUDA;
    prm.bias = bias;
    prm.r_out = r_out;
    prm.logits_out = logits_out;
    prm.dev_status = dev_status;
    prm.N = N;
    prm.d = d;
    prm.C = C;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles * split), 1, 1);
    cfg.blockDim = dim3(kGuThreads, 1, 1);
    cfg.dynamicSmemBytes = SMEM;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // overlap with the tail of the preparation kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (chained_launch_enabled() && image == kImageBuildAndUse) ? 2 : 1;   // chained to the preparation kernel only
    note_launch();
    return cuda_ok(cudaLaunchKernelEx(&cfg, route_gate_umma_kernel<CP>, prm));
}

// (with four adapters or fewer the shared-memory-resident CUDA-core gate needs no preparation launch and is
// as fast up to about 16k tokens)
bool gate_umma_eligible(int64_t N, int32_t d, int32_t C) { return C > 4 && C <= 32 && (d % 64) == 0 && N >= 1024; }

size_t route_gate_umma_workspace_bytes(int32_t d, int32_t C)
{
    if (C <= 4 || (d % 64) != 0) return 0;
    return (size_t)d * 3 * (C <= 16 ? 16 : 32) * 2;
}

molora_status_t launch_route_gate_umma(const void* x, int64_t N, int32_t d, int64_t ldx, const float* G,
                                       const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                       uint32_t* dev_status, cudaStream_t s, int image)
{
    if (N == 0 && image != kImageBuildOnly) return MOLORA_OK;
    if (C <= 16) return gate_umma_launch<16>(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, dev_status, s, image);
    return gate_umma_launch<32>(x, N, d, ldx, G, bias, C, r_out, logits_out, ws, dev_status, s, image);
}

}  // namespace molora
