// Grouped LoRA shrink -> expand on the 5th-generation tensor cores (tcgen05 + TMEM), for segments large
// enough to be a real dense contraction (prefill).  bf16 storage, fp32 accumulation.
//
// One CTA owns a tile of up to 128 positions of one segment (all rows share adapter c) and runs Eq. 2
// for it as two chained MMAs whose intermediate never leaves the SM:
//
//   shrink   T[128, R]   = X[128, d_in] * A_c[d_in, R]      accumulator in TMEM, K streamed in chunks of 64
//   split    T = T_hi + T_lo (two bf16 tiles in shared memory; keeps ~16 mantissa bits of the fp32 T)
//   expand   D[128, 64]  = T_hi * B_c[:, n0:n0+64] + T_lo * B_c[:, n0:n0+64]   per 64-column chunk of d_out
//   epilogue y[rows, n0:n0+64] += D    (fp32 add, one rounding to bf16, written back at the original rows)
//
// Data movement.  The token rows of a tile are NOT contiguous (they come from perm).  The row-gather form of
// the tensor copy moves only four 128-byte rows per instruction and measured ~75 cycles per instruction on
// B200 (about 13 GB/s per SM), so rows are gathered with 16-byte cp.async copies instead: eight lanes fetch one
// 128-byte row segment (a full line) and write it straight into the 128-byte-swizzled K-major layout that
// tcgen05.mma reads.  A_c / B_c chunks are plain 2-D tiled TMA loads and are used as MN-major B operands
// exactly as they lie in memory ([d_in, R] and [R, d_out] row-major), so no transposition pass exists.
// Results leave through shared memory too: the epilogue adds D to the Y chunk in place (thread = row, the
// swizzle makes that conflict-free), then the same threads copy the chunk out with the row-segment mapping
// so that every global store instruction writes full 128-byte lines.
//
// Warp roles (416 threads): warps 0-3 gather X and Y chunks, warp 4 issues the MMAs and owns TMEM, warps
// 5-8 and 9-12 are two epilogue groups that take alternate 64-column chunks.  X chunks and Y chunks travel
// through ONE ring of shared-memory stages, so Y prefetch overlaps the shrink and the shrink -> expand
// hand-over.  Every mbarrier wait is bounded: after ~1 s a waiter raises an abort flag (and
// MOLORA_DEV_TIMEOUT in the status word); from then on all waits fall through and no further copies are
// issued, so control flow stays convergent, TMEM is freed and the kernel returns.
#include <cuda.h>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kProducerWarps = 4;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kMmaWarp = kProducerWarps;
constexpr int kEpiGroups = 2;
constexpr int kEpiWarp0 = kMmaWarp + 1;
constexpr int kUmmaThreads = (kEpiWarp0 + 4 * kEpiGroups) * 32;   // 416
constexpr int kTileM = 128;                 // rows per tile = TMEM lanes
constexpr int kChunkCols = 64;              // bf16 columns per stage: one 128-byte swizzle row
constexpr int kTileBytes = kTileM * 128;    // 16 KB: X or Y chunk
constexpr int kDBufs = 4;                   // expand accumulators in flight (64 TMEM columns each)
constexpr int kTmemCols = 512;
constexpr int kLag = 3;                     // cp.async groups a producer thread keeps in flight
constexpr long long kTimeoutCycles = 2000000000LL;

struct UmmaProj {
    CUtensorMap tm_a, tm_b;
    const __nv_bfloat16* x;
    __nv_bfloat16* y;
    int64_t ldx, ldy;
    int32_t d_in, d_out, rank;
    float scale;
};
struct UmmaParams {
    UmmaProj p[MOLORA_MAX_PROJECTIONS];
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t P, C, min_rows;
};

template <int R>
struct UmmaCfg {
    static constexpr int kWBytes = 64 * R * 2;                       // A chunk [64, R] or B chunk [R, 64]
    static constexpr int kStageBytes = kTileBytes + kWBytes;
    static constexpr int kStages = R == 64 ? 7 : 8;
    static constexpr int kTRowBytes = R * 2;                          // one row of T_hi / T_lo
    static constexpr int kTBytes = kTileM * kTRowBytes;
    static constexpr int kSwzBits = R == 64 ? 3 : R == 32 ? 2 : 1;    // swizzle width of R*2-byte rows
    static constexpr uint32_t kWLayout = swizzle_layout_type(static_cast<Swizzle>(kSwzBits));
    static constexpr int kCtrlBytes = 1024;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kTBytes + kCtrlBytes;
};

struct Ctrl {                         // lives in shared memory after the tiles
    uint64_t full[8], empty[8], t_full, t_ready, d_full[kDBufs], d_empty[kDBufs];
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) int32_t rows[kTileM];
};
static_assert(sizeof(Ctrl) <= 1024, "control block must fit its slot");

// Bounded wait on an mbarrier phase.  Falls through once the CTA has aborted.
__device__ __forceinline__ void wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t* dev_status)
{
    if (*abort_flag) return;
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (*abort_flag) return;
        if (clock64() - t0 > kTimeoutCycles) {
            *abort_flag = 1;
            if (dev_status != nullptr) atomicOr(dev_status, MOLORA_DEV_TIMEOUT);
            return;
        }
    }
}

template <int R>
__global__ void __launch_bounds__(kUmmaThreads, 1) apply_umma_kernel(const __grid_constant__ UmmaParams prm)
{
    using Cfg = UmmaCfg<R>;
    extern __shared__ uint8_t smem_raw[];
    const UmmaProj& pj = prm.p[blockIdx.y];
    if (pj.rank != R) return;
    int seg, row0, rows;
    if (!find_tile(prm.offsets, prm.C, kTileM, blockIdx.x, prm.min_rows, INT32_MAX, seg, row0, rows)) return;

    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t thi = base + Cfg::kStages * Cfg::kStageBytes;
    const uint32_t tlo = thi + Cfg::kTBytes;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw + (tlo + Cfg::kTBytes - raw));
    volatile int* abort_flag = &ctrl->abort_flag;
    auto stage = [&](int s) { return base + (uint32_t)s * Cfg::kStageBytes; };
    auto bar = [&](const uint64_t* b) { return smem_u32(b); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int KX = pj.d_in / kChunkCols, NY = pj.d_out / kChunkCols;
    const int total = KX + NY;

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        prefetch_tensormap(&pj.tm_a);
        prefetch_tensormap(&pj.tm_b);
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(bar(&ctrl->full[s]), kProducerThreads + 1);   // every gathering thread + the weight-chunk arrival
            mbar_init(bar(&ctrl->empty[s]), 1);
        }
        mbar_init(bar(&ctrl->t_full), 1);
        mbar_init(bar(&ctrl->t_ready), kTileM);
        for (int b = 0; b < kDBufs; ++b) {
            mbar_init(bar(&ctrl->d_full[b]), 1);
            mbar_init(bar(&ctrl->d_empty[b]), kTileM);
        }
        ctrl->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    if (tid < kTileM) ctrl->rows[tid] = tid < rows ? __ldg(prm.perm + row0 + tid) : -1;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctrl->tmem_base;
    const uint32_t tmem_T = tmem;                               // columns [0, R)
    auto tmem_D = [&](int b) { return tmem + 64u + 64u * (uint32_t)b; };

    if (warp < kProducerWarps) {
        // ============================================================ gather producer
        // Thread t moves the 16-byte piece (t & 7) of rows (t >> 3) + 16 i, i = 0..7, of every chunk: eight lanes
        // cover one 128-byte row segment.  Completion: each thread waits for its own copies (kLag chunks
        // later), makes them visible to the tensor-core (async) proxy and arrives on the stage's barrier.
        const int piece = tid & 7;
        int64_t xoff[8], yoff[8];
        uint32_t soff[8];
        bool valid[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = (tid >> 3) + 16 * i;
            const int tok = ctrl->rows[r];
            valid[i] = tok >= 0;
            xoff[i] = (int64_t)(valid[i] ? tok : 0) * pj.ldx + piece * 8;
            yoff[i] = (int64_t)(valid[i] ? tok : 0) * pj.ldy + piece * 8;
            soff[i] = swizzle_offset((uint32_t)r * 128u + piece * 16, 3);
        }
        for (int it = 0; it < total + kLag; ++it) {
            if (it < total) {
                const int s = it % Cfg::kStages;
                const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
                wait_bar(bar(&ctrl->empty[s]), ph ^ 1u, abort_flag, prm.dev_status);
                const bool is_x = it < KX;
                const int chunk = is_x ? it : it - KX;
                const uint32_t dst = stage(s);
                if (!*abort_flag) {
                    if (tid == 0) {
                        const uint32_t fb = bar(&ctrl->full[s]);
                        mbar_arrive_expect_tx(fb, (uint32_t)Cfg::kWBytes);
                        if (is_x) tma_load_2d(dst + kTileBytes, &pj.tm_a, 0, seg * pj.d_in + chunk * kChunkCols, fb);
                        else tma_load_2d(dst + kTileBytes, &pj.tm_b, chunk * kChunkCols, seg * R, fb);
                    }
                    const __nv_bfloat16* src = (is_x ? pj.x : pj.y) + chunk * kChunkCols;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (valid[i]) cp_async_16(dst + soff[i], src + (is_x ? xoff[i] : yoff[i]));
                }
            }
            cp_async_commit();
            if (it >= kLag) {
                cp_async_wait<kLag>();
                fence_proxy_async_smem();
                mbar_arrive(bar(&ctrl->full[(it - kLag) % Cfg::kStages]));
            }
        }
    } else if (warp == kMmaWarp) {
        // ============================================================ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_shrink = idesc_bf16_f32(kTileM, R, 0, 1);
            constexpr uint32_t idesc_expand = idesc_bf16_f32(kTileM, kChunkCols, 0, 1);
            constexpr uint32_t kL128 = swizzle_layout_type(Swizzle::B128);
            for (int it = 0; it < KX; ++it) {
                const int s = it % Cfg::kStages;
                const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
                wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t a0 = stage(s), w0 = a0 + kTileBytes;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {   // four K = 16 steps per 64-column chunk
                        const uint64_t ad = smem_desc(a0 + j * 32, 16, 1024, kL128);
                        const uint64_t bd = smem_desc(w0 + j * (16 * Cfg::kTRowBytes), 0, 8 * Cfg::kTRowBytes, Cfg::kWLayout);
                        umma_bf16(tmem_T, ad, bd, idesc_shrink, it > 0 || j > 0);
                    }
                    umma_commit(bar(&ctrl->empty[s]));
                }
            }
            if (!*abort_flag) umma_commit(bar(&ctrl->t_full));
            wait_bar(bar(&ctrl->t_ready), 0, abort_flag, prm.dev_status);
            tc_fence_after();
            for (int nc = 0; nc < NY; ++nc) {
                const int it = KX + nc;
                const int s = it % Cfg::kStages;
                const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
                const int b = nc % kDBufs;
                wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);
                wait_bar(bar(&ctrl->d_empty[b]), ((uint32_t)(nc / kDBufs) & 1u) ^ 1u, abort_flag, prm.dev_status);
                tc_fence_after();
                if (!*abort_flag) {
                    const uint32_t w0 = stage(s) + kTileBytes;
#pragma unroll
                    for (int hl = 0; hl < 2; ++hl) {
                        const uint32_t tb = hl ? tlo : thi;
#pragma unroll
                        for (int j = 0; j < R / 16; ++j) {
                            const uint64_t ad = smem_desc(tb + j * 32, 16, 8 * Cfg::kTRowBytes, Cfg::kWLayout);
                            const uint64_t bd = smem_desc(w0 + j * 2048, 0, 1024, kL128);
                            umma_bf16(tmem_D(b), ad, bd, idesc_expand, hl > 0 || j > 0);
                        }
                    }
                    umma_commit(bar(&ctrl->d_full[b]));
                }
            }
        }
        __syncwarp();
    } else {
        // ============================================================ epilogue groups
        const int group = (warp - kEpiWarp0) >> 2;    // takes chunks group, group + 2, ...
        const int et = tid - (kEpiWarp0 + 4 * group) * 32;   // 0..127 inside the group
        const int q = warp & 3;                       // TMEM lane quarter this warp may access
        const int row = q * 32 + lane;                // tile row = TMEM lane this thread reads
        const uint32_t lane_addr = (uint32_t)(q * 32) << 16;

        if (group == 0) {
            // T -> scaled bf16 hi/lo pair in shared memory, K-major, swizzled like a TMA tile of R*2-byte rows
            wait_bar(bar(&ctrl->t_full), 0, abort_flag, prm.dev_status);
            tc_fence_after();
            uint32_t tv[R];
#pragma unroll
            for (int c = 0; c < R / 16; ++c) tmem_ld_x16(tmem_T + lane_addr + c * 16, tv + c * 16);
            tmem_wait_ld();
#pragma unroll
            for (int c8 = 0; c8 < R / 8; ++c8) {
                float hi[8], lo[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float t = __uint_as_float(tv[c8 * 8 + e]) * pj.scale;
                    hi[e] = __bfloat162float(__float2bfloat16_rn(t));
                    lo[e] = t - hi[e];
                }
                const uint32_t off = swizzle_offset((uint32_t)row * Cfg::kTRowBytes + c8 * 16, Cfg::kSwzBits);
                const uint4 h = pack<__nv_bfloat16>(hi), l = pack<__nv_bfloat16>(lo);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(thi + off), "r"(h.x), "r"(h.y), "r"(h.z), "r"(h.w) : "memory");
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(tlo + off), "r"(l.x), "r"(l.y), "r"(l.z), "r"(l.w) : "memory");
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(&ctrl->t_ready));
        }

        // copy-out mapping: piece (et & 7) of rows (et >> 3) + 16 i
        const int piece = et & 7;
        for (int nc = group; nc < NY; nc += kEpiGroups) {
            const int it = KX + nc;
            const int s = it % Cfg::kStages;
            const uint32_t ph = (uint32_t)(it / Cfg::kStages) & 1u;
            const int b = nc % kDBufs;
            wait_bar(bar(&ctrl->d_full[b]), (uint32_t)(nc / kDBufs) & 1u, abort_flag, prm.dev_status);
            tc_fence_after();
            uint32_t dv[64];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_x16(tmem_D(b) + lane_addr + c * 16, dv + c * 16);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(&ctrl->d_empty[b]));
            wait_bar(bar(&ctrl->full[s]), ph, abort_flag, prm.dev_status);   // the Y chunk of this stage has landed
            const uint32_t ytile = stage(s);
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8) {
                const uint32_t addr = ytile + swizzle_offset((uint32_t)row * 128u + c8 * 16, 3);
                uint4 v;
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
                float yv[8];
                unpack<__nv_bfloat16>(v, yv);
#pragma unroll
                for (int e = 0; e < 8; ++e) yv[e] += __uint_as_float(dv[c8 * 8 + e]);
                v = pack<__nv_bfloat16>(yv);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
            }
            asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
            if (!*abort_flag) {
                __nv_bfloat16* dstc = pj.y + nc * kChunkCols + piece * 8;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int r = (et >> 3) + 16 * i;
                    const int tok = ctrl->rows[r];
                    if (tok >= 0) {
                        const uint32_t addr = ytile + swizzle_offset((uint32_t)r * 128u + piece * 16, 3);
                        uint4 v;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
                        stg128(dstc + (int64_t)tok * pj.ldy, v);
                    }
                }
            }
            asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
            if (et == 0) mbar_arrive(bar(&ctrl->empty[s]));   // the stage may be refilled
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// 2-D bf16 tensor map: `cols` contiguous elements per row, `rows` rows of pitch `ld` elements.
static bool make_map(CUtensorMap* m, const void* ptr, uint64_t cols, uint64_t rows, uint64_t ld, uint32_t box_cols,
                     uint32_t box_rows, CUtensorMapSwizzle swz)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {ld * 2};
    const cuuint32_t box[2] = {box_cols, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool umma_eligible(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    return dt == MOLORA_BF16 && (p.rank == 16 || p.rank == 32 || p.rank == 64) && (p.d_in % kChunkCols) == 0 &&
           (p.d_out % kChunkCols) == 0;
}

template <int R>
static cudaError_t umma_launch(const UmmaParams& prm, int64_t N, cudaStream_t s)
{
    using Cfg = UmmaCfg<R>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(apply_umma_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int64_t tiles = ceil_div64(N, kTileM) + prm.C;
    dim3 grid((unsigned)tiles, (unsigned)prm.P);
    apply_umma_kernel<R><<<grid, kUmmaThreads, Cfg::kSmemBytes, s>>>(prm);
    return cudaGetLastError();
}

molora_status_t launch_apply_umma(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                  const int32_t* offsets, const int32_t* perm, uint32_t* dev_status, int32_t min_rows,
                                  cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    UmmaParams prm;
    bool has[3] = {false, false, false};
    for (int i = 0; i < P; ++i) {
        const molora_proj_desc_t& d = projs[i];
        UmmaProj& u = prm.p[i];
        const CUtensorMapSwizzle wswz = d.rank == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                        : d.rank == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
        bool ok = make_map(&u.tm_a, d.A, d.rank, (uint64_t)C * d.d_in, d.rank, d.rank, kChunkCols, wswz);
        ok = ok && make_map(&u.tm_b, d.B, d.d_out, (uint64_t)C * d.rank, d.d_out, kChunkCols, d.rank,
                            CU_TENSOR_MAP_SWIZZLE_128B);
        if (!ok) return MOLORA_ERR_CUDA;
        u.x = static_cast<const __nv_bfloat16*>(d.x);
        u.y = static_cast<__nv_bfloat16*>(d.y);
        u.ldx = d.ldx;
        u.ldy = d.ldy;
        u.d_in = d.d_in;
        u.d_out = d.d_out;
        u.rank = d.rank;
        u.scale = d.scale;
        has[d.rank == 16 ? 0 : d.rank == 32 ? 1 : 2] = true;
    }
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) prm.p[i].rank = 0;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.P = P;
    prm.C = C;
    prm.min_rows = min_rows;
    cudaError_t e = cudaSuccess;
    if (has[0] && e == cudaSuccess) e = umma_launch<16>(prm, N, s);
    if (has[1] && e == cudaSuccess) e = umma_launch<32>(prm, N, s);
    if (has[2] && e == cudaSuccess) e = umma_launch<64>(prm, N, s);
    return cuda_ok(e);
}

}  // namespace molora
