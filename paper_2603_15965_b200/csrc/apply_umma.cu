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
// Occupancy.  A call with few tiles (N / 128 of them) cannot fill 148 SMs, so a tile may be shared by a
// thread-block cluster of S = 2, 3 or 4 CTAs: CTA q shrinks over the q-th slice of d_in, the S partial T
// tiles (fp32) are exchanged through distributed shared memory and summed in rank order by every CTA (so
// all of them hold the same bits), and CTA q then expands into the q-th slice of d_out.  x, y, A_c and B_c
// are still read exactly once per tile.  The exchange uses mbarriers with remote arrives (bounded waits);
// the only hardware cluster barriers are one after set-up and one before exit, which every thread reaches.
//
// Warp roles (448 threads): warps 0-3 gather X and Y chunks, warp 4 fetches the A_c / B_c chunks, warp 5 issues
// the MMAs and owns TMEM, warps 6-9 and 10-13 are two epilogue groups that take alternate 64-column chunks.  X chunks and Y chunks travel
// through ONE ring of shared-memory stages, so Y prefetch overlaps the shrink and the shrink -> expand
// hand-over.  Every mbarrier wait is bounded: after ~1 s a waiter raises an abort flag (and
// MOLORA_DEV_TIMEOUT in the status word); from then on all waits fall through and no further copies are
// issued, so control flow stays convergent, TMEM is freed and the kernel returns.
#include <cuda.h>
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace molora {

using namespace ptx;

constexpr int kProducerWarps = 4;
constexpr int kProducerThreads = kProducerWarps * 32;
constexpr int kWeightWarp = kProducerWarps;
constexpr int kMmaWarp = kWeightWarp + 1;
constexpr int kEpiGroups = 2;
constexpr int kEpiWarp0 = kMmaWarp + 1;
constexpr int kUmmaThreads = (kEpiWarp0 + 4 * kEpiGroups) * 32;   // 448
constexpr int kTileM = 128;                 // rows per tile = TMEM lanes
constexpr int kChunkCols = 64;              // bf16 columns per stage: one 128-byte swizzle row
constexpr int kTileBytes = kTileM * 128;    // 16 KB: X or Y chunk
constexpr int kDBufs = 4;                   // expand accumulators in flight (64 TMEM columns each)
constexpr int kTmemCols = 512;
constexpr int kMaxSplit = 4;                // largest cluster a tile is split over

struct UmmaProj {
    CUtensorMap tm_a, tm_b;
    const __nv_bfloat16* x;
    __nv_bfloat16* y;
    int64_t ldx, ldy;
    int32_t d_in, d_out, rank;
    float scale;
    const float* row_scale;  // per-token factor on the delta (top-k routing weights) or NULL
    int32_t wide_store;     // y rows are 32-byte aligned: the copy-out uses 256-bit stores
};
struct UmmaParams {
    UmmaProj p[MOLORA_MAX_PROJECTIONS];
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t P, C, min_rows;
    int32_t tile_rows;    // positions per tile: 128, or fewer (the MMA tile stays 128 lanes) to spread a small call over more SMs
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
    // partial T rows received from the cluster peers: (S - 1) * ceil(128 / S) rows of R fp32: 64, 86, 96 rows for
    // S = 2, 3, 4.  Rank 64 stops at S = 3 (shared memory).
    // Ranks 16 and 32 have room for the whole partial of every peer ((S - 1) * 128 rows): one push, every CTA sums
    // for itself.
    static constexpr int kMaxSplitR = R == 64 ? 3 : kMaxSplit;
    static constexpr bool kOnePush = R != 64;
    static constexpr int kRecvBytes = kOnePush ? (kMaxSplit - 1) * kTileM * R * 4 : 86 * R * 4;
    static constexpr int kCtrlBytes = 768;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kTBytes + kRecvBytes + kCtrlBytes;
};

struct Ctrl {                         // lives in shared memory after the tiles
    uint64_t full[8], empty[8], t_full, t_ready, d_full[kDBufs], d_empty[kDBufs], part_full, part_free;
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) int32_t rows[kTileM];
};
static_assert(sizeof(Ctrl) <= 768, "control block must fit its slot");

template <int R>
__global__ void __launch_bounds__(kUmmaThreads, 1) apply_umma_kernel(const __grid_constant__ UmmaParams prm)
{
    using Cfg = UmmaCfg<R>;
    extern __shared__ uint8_t smem_raw[];
    const UmmaProj& pj = prm.p[blockIdx.y];
    if (pj.rank != R) return;
    const uint32_t S = cluster_nctarank(), crank = cluster_ctarank();   // CTAs sharing this tile, and my slice

    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t thi = base + Cfg::kStages * Cfg::kStageBytes;
    const uint32_t tlo = thi + Cfg::kTBytes;
    const uint32_t recv = tlo + Cfg::kTBytes;
    Ctrl* ctrl = reinterpret_cast<Ctrl*>(smem_raw + (recv + Cfg::kRecvBytes - raw));
    volatile int* abort_flag = &ctrl->abort_flag;
    auto stage = [&](int s) { return base + (uint32_t)s * Cfg::kStageBytes; };
    auto bar = [&](const uint64_t* b) { return smem_u32(b); };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // ---------------------------------------------------------------- set-up
    // The segment table is requested first; barriers and TMEM are set up while it is on its way.
    grid_dependency_sync();            // offsets and perm come from the grouping kernel; y from the base projection
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    int32_t offs_v[(MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads];
#pragma unroll
    for (int j = 0; j < (MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads; ++j) {
        const int i = tid + j * kUmmaThreads;
        offs_v[j] = i <= prm.C ? __ldg(prm.offsets + i) : 0;
    }
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
        mbar_init(bar(&ctrl->part_full), 4 * S);     // one arrival per epilogue warp of group 0 of every CTA
        mbar_init(bar(&ctrl->part_free), 4 * S);
        ctrl->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    // which tile is mine: the segment table goes on chip, then the tile is looked up there
#pragma unroll
    for (int j = 0; j < (MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads; ++j) {
        const int i = tid + j * kUmmaThreads;
        if (i <= prm.C) offs_s[i] = offs_v[j];
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    int seg, row0, rows;
    if (!find_tile_smem(offs_s, prm.C, prm.tile_rows, blockIdx.x / S, prm.min_rows, INT32_MAX, seg, row0, rows)) {
        // past the last tile (the grid is sized from an upper bound); the whole cluster takes this exit together
        if (warp == kMmaWarp) tmem_dealloc(ctrl->tmem_base, kTmemCols);
        return;
    }
    const int KXall = pj.d_in / kChunkCols, NYall = pj.d_out / kChunkCols;
    const int kx0 = (int)(crank * KXall / S), KX = (int)((crank + 1) * KXall / S) - kx0;   // my slice of d_in
    const int ny0 = (int)(crank * NYall / S), NY = (int)((crank + 1) * NYall / S) - ny0;   // my slice of d_out
    const int total = KX + NY;
    if (tid < kTileM) ctrl->rows[tid] = tid < rows ? __ldg(prm.perm + row0 + tid) : -1;
    __syncthreads();
    // "I am running and my barriers are initialised": the matching wait comes right before the first access to
    // a peer's shared memory (the T exchange), so the cluster barrier costs nothing here
    if (S > 1) cluster_arrive_relaxed();      // (the barrier initialisation was released by fence_mbar_init)
    const uint32_t tmem = ctrl->tmem_base;
    const uint32_t tmem_T = tmem;                               // columns [0, R)
    auto tmem_D = [&](int b) { return tmem + 64u + 64u * (uint32_t)b; };

    if (warp < kProducerWarps) {
        // ============================================================ gather producer
        // Thread t moves the 16-byte piece (t & 7) of rows (t >> 3) + 16 i, i = 0..7, of every chunk: eight lanes
        // cover one 128-byte row segment.  Each thread's arrival on the stage barrier is triggered by the
        // hardware when its copies have landed, so up to kStages chunks are in flight per SM.
        constexpr int kRowsPerThread = kTileM * 8 / kProducerThreads;
        constexpr int kRowStep = kProducerThreads / 8;
        const int piece = tid & 7;
        const __nv_bfloat16* xsrc[kRowsPerThread];
        const __nv_bfloat16* ysrc[kRowsPerThread];
        uint32_t soff[kRowsPerThread];
        bool valid[kRowsPerThread];
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int r = (tid >> 3) + kRowStep * i;
            const int tok = ctrl->rows[r];
            valid[i] = tok >= 0;
            xsrc[i] = pj.x + (int64_t)(valid[i] ? tok : 0) * pj.ldx + piece * 8 + kx0 * kChunkCols;
            ysrc[i] = pj.y + (int64_t)(valid[i] ? tok : 0) * pj.ldy + piece * 8 + ny0 * kChunkCols;
            soff[i] = swizzle_offset((uint32_t)r * 128u + piece * 16, 3);
        }
        int s = 0;
        uint32_t ph = 1;                                        // parity of the "empty" phase to wait for
        for (int it = 0; it < total; ++it) {
            if (it >= Cfg::kStages) wait_bar(bar(&ctrl->empty[s]), ph, abort_flag, prm.dev_status);   // first round: all free
            const uint32_t dst = stage(s);
            if (!*abort_flag) {
                if (it < KX) {
#pragma unroll
                    for (int i = 0; i < kRowsPerThread; ++i) {
                        if (valid[i]) cp_async_16(dst + soff[i], xsrc[i]);
                        xsrc[i] += kChunkCols;
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kRowsPerThread; ++i) {
                        if (valid[i]) cp_async_16(dst + soff[i], ysrc[i]);
                        ysrc[i] += kChunkCols;
                    }
                }
            }
            cp_async_arrive_noinc(bar(&ctrl->full[s]));
            if (++s == Cfg::kStages) { s = 0; ph ^= 1u; }
        }
    } else if (warp == kWeightWarp) {
        // ============================================================ weight-chunk producer (TMA)
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 1;
            for (int it = 0; it < total; ++it) {
                if (it >= Cfg::kStages) wait_bar(bar(&ctrl->empty[s]), ph, abort_flag, prm.dev_status);
                if (*abort_flag) break;
                const uint32_t fb = bar(&ctrl->full[s]);
                mbar_arrive_expect_tx(fb, (uint32_t)Cfg::kWBytes);
                if (it < KX) tma_load_2d(stage(s) + kTileBytes, &pj.tm_a, 0, seg * pj.d_in + (kx0 + it) * kChunkCols, fb);
                else tma_load_2d(stage(s) + kTileBytes, &pj.tm_b, (ny0 + it - KX) * kChunkCols, seg * R, fb);
                if (++s == Cfg::kStages) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
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
                fence_proxy_async_smem();     // the gathered rows were written through the generic proxy
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
            // LoRA scale times the token's routing weight (1 unless the caller passes per-token factors)
            const int my_tok = ctrl->rows[row];
            const float tscale = pj.scale * ((pj.row_scale != nullptr && my_tok >= 0) ? __ldg(pj.row_scale + my_tok) : 1.f);
            bool t_published = false;
            if (Cfg::kOnePush && S > 1) {
                // Exchange of the partial T tiles in one push through distributed shared memory: every CTA writes its
                // partial into its slot at every peer, one barrier round, and every CTA sums all partials itself in
                // rank order (the same bits in every CTA).  Nothing is read from a peer and nobody touches this CTA's
                // memory afterwards, so the CTAs of a cluster retire independently.
                cluster_wait();                                 // every peer is running, its barriers initialised
                for (uint32_t q2 = 0; q2 < S; ++q2) {
                    if (q2 == crank) continue;
                    const uint32_t slot = crank < q2 ? crank : crank - 1;                   // my slot at CTA q2
                    const uint32_t dst = map_to_cta(recv, q2) + slot * (uint32_t)(kTileM * R * 4);
#pragma unroll
                    for (int c4 = 0; c4 < R / 4; ++c4)
                        st_cluster_u32x4(dst + (uint32_t)(c4 * kTileM + row) * 16u, tv[4 * c4], tv[4 * c4 + 1], tv[4 * c4 + 2],
                                         tv[4 * c4 + 3]);
                }
                __syncwarp();                                   // the warp's rows are sent; lane q2 tells CTA q2
                if ((uint32_t)lane < S) mbar_arrive_remote(map_to_cta(bar(&ctrl->part_full), (uint32_t)lane));
                wait_bar_cluster(bar(&ctrl->part_full), 0, abort_flag, prm.dev_status);
#pragma unroll
                for (int c4 = 0; c4 < R / 4; ++c4) {            // rank order, in place
                    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (uint32_t q2 = 0; q2 < S; ++q2) {
                        float4 v;
                        if (q2 == crank) {
                            v = make_float4(__uint_as_float(tv[4 * c4]), __uint_as_float(tv[4 * c4 + 1]),
                                            __uint_as_float(tv[4 * c4 + 2]), __uint_as_float(tv[4 * c4 + 3]));
                        } else {
                            const uint32_t src = recv + (q2 < crank ? q2 : q2 - 1) * (uint32_t)(kTileM * R * 4);
                            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                                         : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                         : "r"(src + (uint32_t)(c4 * kTileM + row) * 16u)
                                         : "memory");
                        }
                        a.x += v.x;
                        a.y += v.y;
                        a.z += v.z;
                        a.w += v.w;
                    }
                    tv[4 * c4] = __float_as_uint(a.x);
                    tv[4 * c4 + 1] = __float_as_uint(a.y);
                    tv[4 * c4 + 2] = __float_as_uint(a.z);
                    tv[4 * c4 + 3] = __float_as_uint(a.w);
                }
                // tv now holds the full T row: the local conversion below finishes it
            } else if (S > 1) {
                // Exchange of the partial T tiles in two pushes through distributed shared memory.  CTA o owns the
                // tile rows [o*128/S, (o+1)*128/S): (1) every CTA sends its partial of a row to the row's owner;
                // (2) the owner sums the partials in rank order (the same bits whoever computes them), scales,
                // splits into bf16 hi + lo and writes the finished row into the T_hi / T_lo tiles of every CTA.
                // Nothing is ever read from a peer, and after step 2 nobody touches this CTA's memory again, so
                // the CTAs of a cluster retire independently.
                const int rows_max = (kTileM + (int)S - 1) / (int)S;
                int owner = 0;
#pragma unroll
                for (int o = 1; o < kMaxSplit; ++o)
                    if ((uint32_t)o < S && row >= o * kTileM / (int)S) owner = o;
                const int own_lo = owner * kTileM / (int)S;
                cluster_wait();                                 // every peer is running, its barriers initialised
                if ((uint32_t)owner != crank) {
                    const uint32_t slot = crank < (uint32_t)owner ? crank : crank - 1;      // my slot at the owner
                    const uint32_t dst = map_to_cta(recv, (uint32_t)owner) + slot * (uint32_t)(rows_max * R * 4);
#pragma unroll
                    for (int c4 = 0; c4 < R / 4; ++c4)
                        st_cluster_u32x4(dst + (uint32_t)(c4 * rows_max + (row - own_lo)) * 16u, tv[4 * c4], tv[4 * c4 + 1],
                                         tv[4 * c4 + 2], tv[4 * c4 + 3]);
                }
                __syncwarp();                                   // the warp's rows are sent; lane q2 tells CTA q2
                if ((uint32_t)lane < S) mbar_arrive_remote(map_to_cta(bar(&ctrl->part_full), (uint32_t)lane));
                wait_bar_cluster(bar(&ctrl->part_full), 0, abort_flag, prm.dev_status);
                if ((uint32_t)owner == crank) {
                    // sum in rank order, in place: lower ranks' partials, mine (registers), higher ranks'
#pragma unroll
                    for (int c4 = 0; c4 < R / 4; ++c4) {
                        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (uint32_t q2 = 0; q2 < S; ++q2) {
                            float4 v;
                            if (q2 == crank) {
                                v = make_float4(__uint_as_float(tv[4 * c4]), __uint_as_float(tv[4 * c4 + 1]),
                                                __uint_as_float(tv[4 * c4 + 2]), __uint_as_float(tv[4 * c4 + 3]));
                            } else {
                                const uint32_t src = recv + (q2 < crank ? q2 : q2 - 1) * (uint32_t)(rows_max * R * 4);
                                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];"
                                             : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                             : "r"(src + (uint32_t)(c4 * rows_max + (row - own_lo)) * 16u)
                                             : "memory");
                            }
                            a.x += v.x;
                            a.y += v.y;
                            a.z += v.z;
                            a.w += v.w;
                        }
                        tv[4 * c4] = __float_as_uint(a.x);
                        tv[4 * c4 + 1] = __float_as_uint(a.y);
                        tv[4 * c4 + 2] = __float_as_uint(a.z);
                        tv[4 * c4 + 3] = __float_as_uint(a.w);
                    }
#pragma unroll
                    for (int c8 = 0; c8 < R / 8; ++c8) {
                        float hi[8], lo[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float t = __uint_as_float(tv[c8 * 8 + e]) * tscale;
                            hi[e] = __bfloat162float(__float2bfloat16_rn(t));
                            lo[e] = t - hi[e];
                        }
                        const uint32_t off = swizzle_offset((uint32_t)row * Cfg::kTRowBytes + c8 * 16, Cfg::kSwzBits);
                        const uint4 h = pack<__nv_bfloat16>(hi), l = pack<__nv_bfloat16>(lo);
                        for (uint32_t q2 = 0; q2 < S; ++q2) {
                            st_cluster_u32x4(map_to_cta(thi + off, q2), h.x, h.y, h.z, h.w);
                            st_cluster_u32x4(map_to_cta(tlo + off, q2), l.x, l.y, l.z, l.w);
                        }
                    }
                }
                __syncwarp();                                   // the warp's rows are published everywhere
                if ((uint32_t)lane < S) mbar_arrive_remote(map_to_cta(bar(&ctrl->part_free), (uint32_t)lane));
                wait_bar_cluster(bar(&ctrl->part_free), 0, abort_flag, prm.dev_status);   // all 128 rows of T are here
                t_published = true;
            }
            if (!t_published) {
#pragma unroll
                for (int c8 = 0; c8 < R / 8; ++c8) {
                    float hi[8], lo[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float t = __uint_as_float(tv[c8 * 8 + e]) * tscale;
                        hi[e] = __bfloat162float(__float2bfloat16_rn(t));
                        lo[e] = t - hi[e];
                    }
                    const uint32_t off = swizzle_offset((uint32_t)row * Cfg::kTRowBytes + c8 * 16, Cfg::kSwzBits);
                    const uint4 h = pack<__nv_bfloat16>(hi), l = pack<__nv_bfloat16>(lo);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(thi + off), "r"(h.x), "r"(h.y), "r"(h.z), "r"(h.w) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(tlo + off), "r"(l.x), "r"(l.y), "r"(l.z), "r"(l.w) : "memory");
                }
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(&ctrl->t_ready));
        }

        // copy-out mapping: piece (et & 7) of rows (et >> 3) + 16 i
        const int piece = et & 7;
        int otok[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) otok[i] = ctrl->rows[(et >> 3) + 16 * i];
        int wtok[4];                                    // 256-bit variant: rows (et >> 2) + 32 i
#pragma unroll
        for (int i = 0; i < 4; ++i) wtok[i] = ctrl->rows[(et >> 2) + 32 * i];
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
            uint8_t* ytile = smem_raw + (stage(s) - raw);
            {
                uint4 yp[8];
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8)
                    yp[c8] = *reinterpret_cast<const uint4*>(ytile + swizzle_offset((uint32_t)row * 128u + c8 * 16, 3));
#pragma unroll
                for (int c8 = 0; c8 < 8; ++c8) {
                    float yv[8];
                    unpack<__nv_bfloat16>(yp[c8], yv);
#pragma unroll
                    for (int e = 0; e < 8; ++e) yv[e] += __uint_as_float(dv[c8 * 8 + e]);
                    *reinterpret_cast<uint4*>(ytile + swizzle_offset((uint32_t)row * 128u + c8 * 16, 3)) =
                        pack<__nv_bfloat16>(yv);
                }
            }
            asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");
            if (!*abort_flag) {
                if (pj.wide_store) {
                    // 32 bytes per lane: four lanes cover a 128-byte row segment, a warp instruction eight rows
                    const int p32 = et & 3;
                    __nv_bfloat16* dstc = pj.y + (ny0 + nc) * kChunkCols + p32 * 16;
                    uint4 lo4[4], hi4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t r = (uint32_t)((et >> 2) + 32 * i);
                        lo4[i] = *reinterpret_cast<const uint4*>(ytile + swizzle_offset(r * 128u + p32 * 32, 3));
                        hi4[i] = *reinterpret_cast<const uint4*>(ytile + swizzle_offset(r * 128u + p32 * 32 + 16, 3));
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        if (wtok[i] >= 0) stg256(dstc + (int64_t)wtok[i] * pj.ldy, lo4[i], hi4[i]);
                } else {
                    __nv_bfloat16* dstc = pj.y + (ny0 + nc) * kChunkCols + piece * 8;
                    uint4 op[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        op[i] = *reinterpret_cast<const uint4*>(
                            ytile + swizzle_offset((uint32_t)((et >> 3) + 16 * i) * 128u + piece * 16, 3));
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (otok[i] >= 0) stg128(dstc + (int64_t)otok[i] * pj.ldy, op[i]);
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
    // threads that took no part in the exchange complete the start-up cluster barrier here (it has long been
    // passed); no closing barrier is needed, see the exchange
    if (S > 1 && !(warp >= kEpiWarp0 && warp < kEpiWarp0 + 4)) cluster_wait();
}

// Self-test of the bounded wait: one warp waits on an mbarrier that nothing ever arrives on, with a limit of
// `limit_cycles`.  The wait must give up, raise the abort flag and MOLORA_DEV_TIMEOUT, and the kernel must return
// normally (no trap, no hang): this is the exit every pipeline role takes if a peer never shows up.
__global__ void bounded_wait_selftest_kernel(uint32_t* dev_status, long long limit_cycles, int32_t* result)
{
    __shared__ uint64_t never;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&never), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    wait_bar(smem_u32(&never), 0, &abort_flag, dev_status, limit_cycles);
    __syncthreads();
    // a second wait after the abort must fall through at once
    const long long t0 = clock64();
    wait_bar(smem_u32(&never), 0, &abort_flag, dev_status, limit_cycles);
    if (threadIdx.x == 0) {
        result[0] = abort_flag;
        result[1] = (clock64() - t0) < limit_cycles ? 1 : 0;
    }
}

molora_status_t launch_bounded_wait_selftest(uint32_t* dev_status, int64_t limit_cycles, int32_t* result, cudaStream_t s)
{
    note_launch();
    bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(dev_status, limit_cycles, result);
    return cuda_ok(cudaGetLastError());
}

// ------------------------------------------------------------------------------------------------ host side
bool umma_eligible(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    return dt == MOLORA_BF16 && (p.rank == 16 || p.rank == 32 || p.rank == 64) && (p.d_in % kChunkCols) == 0 &&
           (p.d_out % kChunkCols) == 0;
}

struct UmmaPlan {
    int split;       // CTAs per tile (cluster size)
    int tile_rows;   // positions per tile
};

template <int R>
static void fill_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int64_t tiles, int P, int split,
                               cudaStream_t s)
{
    cfg.gridDim = dim3((unsigned)(tiles * split), (unsigned)P, 1);
    cfg.blockDim = dim3(kUmmaThreads, 1, 1);
    cfg.dynamicSmemBytes = UmmaCfg<R>::kSmemBytes;
    cfg.stream = s;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

template <int R>
static cudaError_t umma_launch(UmmaParams prm, int64_t N, UmmaPlan plan, cudaStream_t s)
{
    const int split = plan.split;
    prm.tile_rows = plan.tile_rows;
    using Cfg = UmmaCfg<R>;
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(apply_umma_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int64_t tiles = ceil_div64(N, prm.tile_rows) + prm.C;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    fill_launch_config<R>(cfg, attr, tiles, prm.P, split, s);
    note_launch();
    return cudaLaunchKernelEx(&cfg, apply_umma_kernel<R>, prm);
}

// Clusters of `split` CTAs of this kernel that can be resident at once (cached per rank and split).
template <int R>
static int max_active_clusters(int split)
{
    static int cache_dev[kMaxDevices][kMaxSplit + 1] = {};
    int (&cache)[kMaxSplit + 1] = cache_dev[device_slot()];
    if (cache[split] == 0) {
        cudaFuncSetAttribute(apply_umma_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize, UmmaCfg<R>::kSmemBytes);
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        fill_launch_config<R>(cfg, attr, 148, 1, split, nullptr);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, apply_umma_kernel<R>, &cfg) != cudaSuccess || n <= 0) n = 148 / split;
        cache[split] = n;
    }
    return cache[split];
}

// CTAs per tile.  Tiles are 128 rows, so small calls have too few of them for 148 SMs; a tile can be split over
// a cluster of 2 or 4 CTAs.  Pick the split with the smallest estimated time: waves of resident clusters times
// (work per CTA, which shrinks with the split, plus a fixed per-CTA cost and the cost of the exchange).
template <int R>
static UmmaPlan choose_split_for_rank(const UmmaParams& prm, int64_t N)
{
    int min_kx = INT32_MAX, nproj = 0;
    for (int i = 0; i < prm.P; ++i) {
        if (prm.p[i].rank != R) continue;
        min_kx = std::min(min_kx, prm.p[i].d_in / kChunkCols);
        ++nproj;
    }
    // expected tiles: every segment ends in a partial tile
    auto tiles_for = [&](int rows) { return (ceil_div64(N, rows) + prm.C / 2) * nproj; };
    auto cost_for = [&](int rows, int split, double& waves) {
        const int resident = max_active_clusters<R>(split);
        waves = (double)((tiles_for(rows) + resident - 1) / resident);
        return waves * ((rows / 128.0) / split + 0.15 + (split > 1 ? 0.10 : 0.0));
    };
    UmmaPlan best = {1, kTileM};
    const int64_t fsplit = tune(kTuneUmmaSplit), frows = tune(kTuneUmmaTileRows);          // tuning overrides
    if (fsplit > 0 || frows > 0) {
        if (fsplit > 0) best.split = (int)std::max<int64_t>(1, std::min<int64_t>(fsplit, UmmaCfg<R>::kMaxSplitR));
        if (frows > 0) best.tile_rows = (int)std::max<int64_t>(32, std::min<int64_t>(frows, kTileM));
    } else {
        double best_cost = 1e30, best_waves = 0;
        for (int split = 1; split <= UmmaCfg<R>::kMaxSplitR; ++split) {    // cluster sizes need not be powers of two
            double waves;
            const double cost = cost_for(kTileM, split, waves);
            if (cost < best_cost - 1e-9) { best_cost = cost; best_waves = waves; best = {split, kTileM}; }
        }
        // A call that does not even fill one wave can use shorter tiles (the MMA tile keeps 128 lanes, the extra
        // lanes idle) to put more SMs to work, as long as everything still fits in one wave.
        if (best_waves <= 1.0 && tiles_for(kTileM) * best.split < 0.85 * 148) {
            for (int rows = 96; rows >= 64; rows -= 32)
                for (int split = 1; split <= UmmaCfg<R>::kMaxSplitR; ++split) {
                    double waves;
                    const double cost = cost_for(rows, split, waves);
                    if (waves <= 1.0 && cost < best_cost - 1e-9) { best_cost = cost; best = {split, rows}; }
                }
        }
    }
    while (best.split > 1 && min_kx / best.split < 4) --best.split;   // keep at least four chunks of d_in per CTA
    return best;
}

molora_status_t launch_apply_umma(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                  const int32_t* offsets, const int32_t* perm, uint32_t* dev_status, int32_t min_rows,
                                  cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    UmmaParams prm;
    bool has[3] = {false, false, false};
    // CTAs are dispatched projection by projection (blockIdx.y): put the projections that move the most bytes
    // per tile first, so that the last, partly filled wave consists of the cheap tiles.
    int order[MOLORA_MAX_PROJECTIONS];
    for (int i = 0; i < P; ++i) order[i] = i;
    std::stable_sort(order, order + P, [&](int a, int b) {
        return (int64_t)projs[a].d_in + 2 * (int64_t)projs[a].d_out > (int64_t)projs[b].d_in + 2 * (int64_t)projs[b].d_out;
    });
    for (int i = 0; i < P; ++i) {
        const molora_proj_desc_t& d = projs[order[i]];
        UmmaProj& u = prm.p[i];
        const CUtensorMapSwizzle wswz = d.rank == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                        : d.rank == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
        bool ok = make_tensor_map_bf16_2d(&u.tm_a, d.A, d.rank, (uint64_t)C * d.d_in, d.rank, d.rank, kChunkCols, wswz);
        ok = ok && make_tensor_map_bf16_2d(&u.tm_b, d.B, d.d_out, (uint64_t)C * d.rank, d.d_out, kChunkCols, d.rank,
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
        u.row_scale = d.row_scale;
        u.wide_store = ((reinterpret_cast<uintptr_t>(d.y) & 31u) == 0 && ((d.ldy * 2) % 32) == 0) ? 1 : 0;
        has[d.rank == 16 ? 0 : d.rank == 32 ? 1 : 2] = true;
    }
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) prm.p[i].rank = 0;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.P = P;
    prm.C = C;
    prm.min_rows = min_rows;
    prm.tile_rows = kTileM;
    cudaError_t e = cudaSuccess;
    if (has[0] && e == cudaSuccess) e = umma_launch<16>(prm, N, choose_split_for_rank<16>(prm, N), s);
    if (has[1] && e == cudaSuccess) e = umma_launch<32>(prm, N, choose_split_for_rank<32>(prm, N), s);
    if (has[2] && e == cudaSuccess) e = umma_launch<64>(prm, N, choose_split_for_rank<64>(prm, N), s);
    return cuda_ok(e);
}

}  // namespace molora
