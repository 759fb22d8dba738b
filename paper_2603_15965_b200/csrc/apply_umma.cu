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
#include "group_inline.cuh"
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
constexpr int kMaxWideSplit = 8;            // ... by the rank-64 variant for calls with few tiles (portable cluster limit)

struct UmmaProj {
    CUtensorMap tm_a, tm_b;
    const __nv_bfloat16* x;
    __nv_bfloat16* y;
    int64_t ldx, ldy;
    int32_t d_in, d_out, rank;
    float scale;
    const float* row_scale;  // per-token factor on the delta (top-k routing weights) or NULL
    int32_t wide_store;     // y rows are 32-byte aligned: the copy-out uses 256-bit stores
    // Projections of equal shape that read the same x (k / v, gate / up) are neighbours in the launch and their tiles are
    // dispatched interleaved -- tile 0 of each, tile 1 of each, ... -- so that the x rows one of them brings into L2 are
    // still there for the others: first projection of my group and its size (1: no sharing).
    int32_t gfirst, gsize;
};
struct UmmaParams {
    UmmaProj p[MOLORA_MAX_PROJECTIONS];
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t P, C, min_rows;
    int32_t tile_rows;    // positions per tile: 128, or fewer (the MMA tile stays 128 lanes) to spread a small call over more SMs
    // Grouping inside the kernel (r != NULL; at most kUmmaGroupMaxN tokens): every CTA runs Section 3.3 steps 1-3 on the
    // routing decisions in its idle ring stages instead of loading offsets / perm, and the CTAs of projection 0 write
    // counts, offsets and perm out -- the grouping launch in front of a mid-sized call costs as much as a third of it.
    const int32_t* r;
    int32_t N;
    int32_t* counts_out;
    int32_t* offsets_out;
    int32_t* perm_out;
    // Top-k routing in one pass (Eq. 8): a segment is a SET of `parts` adapters (named by set_table, `cbase` adapters
    // in all) and the launch's rank R is parts x the adapters' rank r.  The shrink runs one MMA per part into
    // its own r columns of T (the part's A chunk is its own shared-memory tile), every part of a row of T is scaled by the
    // token's weight for that part (row_scale[part * N + token]), and the expand contracts all R columns against the
    // parts' B chunks stacked by rows -- one read of x and y, one rounding.  parts == 1: plain top-1 routing.
    int32_t parts, cbase;
    const uint8_t* set_table;         // parts > 1: set_table[4 * segment + j] = the j-th adapter of the set
};
constexpr int kUmmaGroupMaxN = 4096;
constexpr int kUmmaMaxParts = 4;


// WIDE (rank 64 only): one ring stage fewer, which makes room for the partial rows of up to seven peers, so that a tile
// can be split over a cluster of up to 8 CTAs -- for calls with so few tiles that the chain of chunks per CTA, not the
// bytes, sets the time.
template <int R, bool WIDE = false>
struct UmmaCfg {
    static_assert(!WIDE || R == 64, "the wide split exists for rank 64");
    static constexpr int kWBytes = 64 * R * 2;                       // A chunk [64, R] or B chunk [R, 64]
    static constexpr int kStageBytes = kTileBytes + kWBytes;
    static constexpr int kStages = R == 64 ? (WIDE ? 6 : 7) : 8;
    static constexpr int kTRowBytes = R * 2;                          // one row of T_hi / T_lo
    static constexpr int kTBytes = kTileM * kTRowBytes;
    static constexpr int kSwzBits = R == 64 ? 3 : R == 32 ? 2 : 1;    // swizzle width of R*2-byte rows
    static constexpr uint32_t kWLayout = swizzle_layout_type(static_cast<Swizzle>(kSwzBits));
    // partial T rows received from the cluster peers: (S - 1) * ceil(128 / S) rows of R fp32: 64, 86, 96 rows for
    // S = 2, 3, 4 and at most 114 (S = 7) up to S = 8.  Rank 64 stops at S = 3 (shared memory) unless WIDE.
    // Ranks 16 and 32 have room for the whole partial of every peer ((S - 1) * 128 rows): one push, every CTA sums
    // for itself.
    static constexpr int kMaxSplitR = R == 64 ? (WIDE ? kMaxWideSplit : 3) : kMaxSplit;
    static constexpr bool kOnePush = R != 64;
    static constexpr int kRecvBytes = kOnePush ? (kMaxSplit - 1) * kTileM * R * 4 : (WIDE ? 114 : 86) * R * 4;
    static constexpr int kCtrlBytes = 768;
    static constexpr int kSmemBytes = 1024 + kStages * kStageBytes + 2 * kTBytes + kRecvBytes + kCtrlBytes;
};

struct Ctrl {                         // lives in shared memory after the tiles
    uint64_t full[8], empty[8], t_full, t_ready, d_full[kDBufs], d_empty[kDBufs], part_full, part_free, peers_done;
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) int32_t rows[kTileM];
};
static_assert(sizeof(Ctrl) <= 768, "control block must fit its slot");

// Sum of the partial rows of T over the CTAs of a cluster, in rank order (the same bits whoever computes them), in place
// in tv (this CTA's partial, NWORDS fp32 words of one row).  The peers' partials lie in shared memory as [slot][R / 4][rows]
// float4 pieces (slot = sender's rank, skipping this CTA); `mine` points at this row's piece 0 of slot 0.  Four
// independent 16-byte loads per sender keep the loop from running at one shared-memory latency per piece.
template <int NWORDS>
__device__ __forceinline__ void sum_partials(uint32_t (&tv)[NWORDS], const float4* mine, int piece_stride, int slot_stride, uint32_t S,
                                             uint32_t crank)
{
    constexpr int R = NWORDS;
    constexpr int kBatch = R / 4 < 4 ? R / 4 : 4;
#pragma unroll
    for (int h = 0; h < R / 4 / kBatch; ++h) {
        float4 acc[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t q2 = 0; q2 < S; ++q2) {
            float4 v[kBatch];
            if (q2 == crank) {
#pragma unroll
                for (int j = 0; j < kBatch; ++j) {
                    const int c4 = h * kBatch + j;
                    v[j] = make_float4(__uint_as_float(tv[4 * c4]), __uint_as_float(tv[4 * c4 + 1]), __uint_as_float(tv[4 * c4 + 2]),
                                       __uint_as_float(tv[4 * c4 + 3]));
                }
            } else {
                const float4* src = mine + (size_t)(q2 < crank ? q2 : q2 - 1) * slot_stride + (size_t)(h * kBatch) * piece_stride;
#pragma unroll
                for (int j = 0; j < kBatch; ++j) v[j] = src[(size_t)j * piece_stride];
            }
#pragma unroll
            for (int j = 0; j < kBatch; ++j) {
                acc[j].x += v[j].x;
                acc[j].y += v[j].y;
                acc[j].z += v[j].z;
                acc[j].w += v[j].w;
            }
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int c4 = h * kBatch + j;
            tv[4 * c4] = __float_as_uint(acc[j].x);
            tv[4 * c4 + 1] = __float_as_uint(acc[j].y);
            tv[4 * c4 + 2] = __float_as_uint(acc[j].z);
            tv[4 * c4 + 3] = __float_as_uint(acc[j].w);
        }
    }
}

// PARTS: adapters per segment (1: top-1 routing; 2 or 4: adapter sets of top-k routing, see UmmaParams) -- a compile-time
// constant so that the top-1 kernel is exactly the code it was before sets existed (a run-time `parts` cost it 13 %).
template <int R, bool WIDE, int PARTS>
__global__ void __launch_bounds__(kUmmaThreads, 1) apply_umma_kernel(const __grid_constant__ UmmaParams prm)
{
    using Cfg = UmmaCfg<R, WIDE>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t S = cluster_nctarank(), crank = cluster_ctarank();   // CTAs sharing this tile, and my slice
    // (tile, projection) of this cluster: blockIdx.y walks the projections, except inside a group that shares x, whose
    // m x (tiles) clusters are renumbered tile-major
    int proj = (int)blockIdx.y, my_tile = (int)(blockIdx.x / S);
    {
        const UmmaProj& p0 = prm.p[blockIdx.y];
        if (p0.rank != R) return;
        if (p0.gsize > 1) {
            const int lc = ((int)blockIdx.y - p0.gfirst) * (int)(gridDim.x / S) + my_tile;
            my_tile = lc / p0.gsize;
            proj = p0.gfirst + lc % p0.gsize;
        }
    }
    const UmmaProj& pj = prm.p[proj];

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
    const bool grouping = prm.r != nullptr;
    // grouping: perm, a scratch table and 256 temporary words live in the ring stages, which are idle until the tile is known
    int32_t* perm_s = reinterpret_cast<int32_t*>(smem_raw + (base - raw));
    int32_t* gtmp_s = perm_s + kUmmaGroupMaxN;
    unsigned char* gscratch = reinterpret_cast<unsigned char*>(gtmp_s + MOLORA_MAX_ADAPTERS);
    static_assert(kUmmaGroupMaxN * 4 + MOLORA_MAX_ADAPTERS * 4 + kGroupInCtaTableMaxC * kUmmaThreads * 4 + 4 * kGroupInCtaTableMaxC <=
                      Cfg::kStages * Cfg::kStageBytes, "the grouping scratch must fit the ring");
    static_assert(kUmmaThreads / 32 * MOLORA_MAX_ADAPTERS * 4 <= kGroupInCtaTableMaxC * kUmmaThreads * 4, "ballot-path scratch");
    int32_t offs_v[(MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads];
#pragma unroll
    for (int j = 0; j < (MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads; ++j) {
        const int i = tid + j * kUmmaThreads;
        offs_v[j] = (!grouping && i <= prm.C) ? __ldg(prm.offsets + i) : 0;
    }
    if (tid == 0) {
        prefetch_tensormap(&pj.tm_a);
        prefetch_tensormap(&pj.tm_b);
        for (int s = 0; s < Cfg::kStages; ++s) {
            mbar_init(bar(&ctrl->full[s]), kProducerThreads + 1);   // every gathering thread + the weight-chunk arrival
            mbar_init(bar(&ctrl->empty[s]), 4);      // the four warps of an epilogue group; the MMA thread arrives for all four
        }
        mbar_init(bar(&ctrl->t_full), 1);
        mbar_init(bar(&ctrl->t_ready), 2 * kTileM);      // both epilogue groups
        for (int b = 0; b < kDBufs; ++b) {
            mbar_init(bar(&ctrl->d_full[b]), 1);
            mbar_init(bar(&ctrl->d_empty[b]), kTileM);
        }
        mbar_init(bar(&ctrl->part_full), 1);         // the partials arrive as asynchronous stores that count their bytes here
        // one push (ranks 16, 32): unused.  Two pushes (rank 64): the finished rows of T arrive by bulk copies that
        // count their bytes here; the one arrival is this CTA's own, which states the byte count
        mbar_init(bar(&ctrl->part_free), 1);
        mbar_init(bar(&ctrl->peers_done), S > 1 ? S - 1 : 1);   // every peer has received the rows this CTA sent it
        ctrl->abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&ctrl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    // which tile is mine: the segment table goes on chip (or is built there), then the tile is looked up there
    if (grouping) {
        group_in_cta<kUmmaThreads, kUmmaGroupMaxN>(prm.r, prm.N, prm.C, offs_s, gtmp_s, perm_s, gscratch, blockIdx.y == 0,
                                                   prm.counts_out, prm.offsets_out, prm.perm_out, prm.dev_status);
    } else {
#pragma unroll
        for (int j = 0; j < (MOLORA_MAX_ADAPTERS + kUmmaThreads) / kUmmaThreads; ++j) {
            const int i = tid + j * kUmmaThreads;
            if (i <= prm.C) offs_s[i] = offs_v[j];
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    int seg, row0, rows;
    if (!find_tile_smem(offs_s, prm.C, prm.tile_rows, my_tile, prm.min_rows, INT32_MAX, seg, row0, rows)) {
        // past the last tile (the grid is sized from an upper bound); the whole cluster takes this exit together
        if (warp == kMmaWarp) tmem_dealloc(ctrl->tmem_base, kTmemCols);
        return;
    }
    // adapters of the segment's set (one adapter when parts == 1) and the rank of each
    constexpr int parts = PARTS, rp = R / PARTS;
    static_assert(rp >= 16 && rp * PARTS == R, "adapters of rank 16, 32 or 64");
    int adapter[kUmmaMaxParts];
#pragma unroll
    for (int j = 0; j < kUmmaMaxParts; ++j)
        adapter[j] = PARTS == 1 ? seg : (j < PARTS ? (int)__ldg(prm.set_table + seg * 4 + j) : 0);
    const int KXall = pj.d_in / kChunkCols, NYall = pj.d_out / kChunkCols;
    const int kx0 = (int)(crank * KXall / S), KX = (int)((crank + 1) * KXall / S) - kx0;   // my slice of d_in
    const int ny0 = (int)(crank * NYall / S), NY = (int)((crank + 1) * NYall / S) - ny0;   // my slice of d_out
    const int total = KX + NY;
    if (tid < kTileM) ctrl->rows[tid] = tid < rows ? (grouping ? perm_s[row0 + tid] : __ldg(prm.perm + row0 + tid)) : -1;
    __syncthreads();                    // (the ring may be filled from here on: nobody reads perm_s any more)
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
                // one box per part: A chunks [64, r] side by side as tiles of their own, B chunks [r, 64] stacked by rows
#pragma unroll
                for (int j = 0; j < PARTS; ++j) {
                    if (it < KX)
                        tma_load_2d(stage(s) + kTileBytes + (uint32_t)(j * kChunkCols * rp * 2), &pj.tm_a, 0,
                                    adapter[j] * pj.d_in + (kx0 + it) * kChunkCols, fb);
                    else
                        tma_load_2d(stage(s) + kTileBytes + (uint32_t)(j * rp * 128), &pj.tm_b, (ny0 + it - KX) * kChunkCols,
                                    adapter[j] * rp, fb);
                }
                if (++s == Cfg::kStages) { s = 0; ph ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ============================================================ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_shrink = idesc_bf16_f32(kTileM, rp, 0, 1);
            // rows of an A chunk are r x 2 bytes: 128-, 64- or 32-byte swizzle
            constexpr uint32_t wlayout = swizzle_layout_type(rp == 64 ? Swizzle::B128 : rp == 32 ? Swizzle::B64 : Swizzle::B32);
            constexpr uint32_t wrow = (uint32_t)rp * 2u;
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
#pragma unroll
                        for (int pt = 0; pt < PARTS; ++pt) {          // part pt -> columns [pt r, (pt + 1) r) of T
                            const uint64_t bd = smem_desc(w0 + (uint32_t)pt * kChunkCols * wrow + j * (16 * wrow), 0, 8 * wrow, wlayout);
                            umma_bf16(tmem_T + (uint32_t)(pt * rp), ad, bd, idesc_shrink, it > 0 || j > 0);
                        }
                    }
                    umma_commit(bar(&ctrl->empty[s]));          // arrives when the MMAs have read the stage ...
#pragma unroll
                    for (int k = 0; k < 3; ++k) mbar_arrive(bar(&ctrl->empty[s]));   // ... and completes the count of four
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

        {
            // T -> scaled bf16 hi/lo pair in shared memory, K-major, swizzled like a TMA tile of R*2-byte rows.  Both
            // epilogue groups take part, group g with the columns [g R/2, (g+1) R/2) of every row: a lone warp runs the
            // few hundred dependent instructions of a row at one every four cycles, and its stores into a peer's shared
            // memory at one every ~0.14 us, so the work per thread is what this step costs.
            constexpr int RH = R / 2;
            const int col0 = group * RH;
            wait_bar(bar(&ctrl->t_full), 0, abort_flag, prm.dev_status);
            tc_fence_after();
            uint32_t tv[RH];
            if constexpr (RH == 8) {
                tmem_ld_x8(tmem_T + lane_addr + col0, tv);
            } else {
#pragma unroll
                for (int c = 0; c < RH / 16; ++c) tmem_ld_x16(tmem_T + lane_addr + col0 + c * 16, tv + c * 16);
            }
            tmem_wait_ld();
            // LoRA scale times the token's routing weight (1 unless the caller passes per-token factors)
            const int my_tok = ctrl->rows[row];
            float tscale[kUmmaMaxParts];
#pragma unroll
            for (int j = 0; j < kUmmaMaxParts; ++j)
                tscale[j] = pj.scale * ((pj.row_scale != nullptr && my_tok >= 0 && j < parts)
                                            ? __ldg(pj.row_scale + (int64_t)j * prm.N + my_tok) : 1.f);
            // my half row -> T_hi / T_lo of this CTA
            auto publish_local = [&]() {
#pragma unroll
                for (int c8 = 0; c8 < RH / 8; ++c8) {
                    float hi[8], lo[8];
                    const int tpart = (col0 + c8 * 8) / rp;       // (r is a multiple of 16: a block of 8 columns has one part)
                    const float ts = PARTS == 1 ? tscale[0] : tpart == 0 ? tscale[0] : tpart == 1 ? tscale[1] : tpart == 2 ? tscale[2] : tscale[3];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float t = __uint_as_float(tv[c8 * 8 + e]) * ts;
                        hi[e] = __bfloat162float(__float2bfloat16_rn(t));
                        lo[e] = t - hi[e];
                    }
                    const uint32_t off = swizzle_offset((uint32_t)row * Cfg::kTRowBytes + (uint32_t)(col0 / 8 + c8) * 16, Cfg::kSwzBits);
                    const uint4 h = pack<__nv_bfloat16>(hi), l = pack<__nv_bfloat16>(lo);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(thi + off), "r"(h.x), "r"(h.y), "r"(h.z), "r"(h.w) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(tlo + off), "r"(l.x), "r"(l.y), "r"(l.z), "r"(l.w) : "memory");
                }
            };
            const float4* recv_p = reinterpret_cast<const float4*>(smem_raw + (recv - raw));
            if (Cfg::kOnePush && S > 1) {
                // Exchange of the partial T tiles in one push through distributed shared memory: every CTA writes its
                // partial into its slot at every peer, one barrier round, and every CTA sums all partials itself in
                // rank order (the same bits in every CTA).  Nothing is read from a peer and nobody touches this CTA's
                // memory afterwards, so the CTAs of a cluster retire independently.
                cluster_wait();                                 // every peer is running, its barriers initialised
                if (group == 0 && et == 0) mbar_arrive_expect_tx(bar(&ctrl->part_full), (S - 1) * (uint32_t)(kTileM * R * 4));
                for (uint32_t q2 = 0; q2 < S; ++q2) {
                    if (q2 == crank) continue;
                    const uint32_t slot = crank < q2 ? crank : crank - 1;                   // my slot at CTA q2
                    const uint32_t dst = map_to_cta(recv, q2) + slot * (uint32_t)(kTileM * R * 4);
                    const uint32_t pb = map_to_cta(bar(&ctrl->part_full), q2);              // counts the bytes it receives
#pragma unroll
                    for (int c4 = 0; c4 < RH / 4; ++c4)
                        st_async_cluster_u32x4(dst + (uint32_t)((col0 / 4 + c4) * kTileM + row) * 16u, tv[4 * c4], tv[4 * c4 + 1],
                                               tv[4 * c4 + 2], tv[4 * c4 + 3], pb);
                }
                wait_bar_cluster(bar(&ctrl->part_full), 0, abort_flag, prm.dev_status);
                sum_partials<RH>(tv, recv_p + (col0 / 4) * kTileM + row, kTileM, kTileM * R / 4, S, crank);
                publish_local();                                // tv holds the full half row
            } else if (S > 1) {
                // Exchange of the partial T tiles in two pushes through distributed shared memory.  CTA o owns the
                // tile rows [o*128/S, (o+1)*128/S): (1) every CTA sends its partial of a row to the row's owner;
                // (2) the owner sums the partials in rank order (the same bits whoever computes them), scales,
                // splits into bf16 hi + lo and writes the finished rows into its own T_hi / T_lo tiles; (3) bulk copies
                // carry them into the tiles of every peer.  Nothing is ever read from a peer by a thread; a CTA retires
                // once every peer has confirmed the arrival of its rows (peers_done, waited for at the very end).
                const int rows_max = (kTileM + (int)S - 1) / (int)S;
                int owner = 0;
#pragma unroll
                for (int o = 1; o < Cfg::kMaxSplitR; ++o)
                    if ((uint32_t)o < S && row >= o * kTileM / (int)S) owner = o;
                const int own_lo = owner * kTileM / (int)S;
                cluster_wait();                                 // every peer is running, its barriers initialised
                if (group == 0 && et == 0) {                    // what the peers will send me: their partials of my rows
                    const int mine = (int)(crank + 1) * kTileM / (int)S - (int)crank * kTileM / (int)S;
                    mbar_arrive_expect_tx(bar(&ctrl->part_full), (S - 1) * (uint32_t)(mine * R * 4));
                }
                if ((uint32_t)owner != crank) {
                    const uint32_t slot = crank < (uint32_t)owner ? crank : crank - 1;      // my slot at the owner
                    const uint32_t dst = map_to_cta(recv, (uint32_t)owner) + slot * (uint32_t)(rows_max * R * 4);
                    const uint32_t pb = map_to_cta(bar(&ctrl->part_full), (uint32_t)owner); // counts the bytes it receives
#pragma unroll
                    for (int c4 = 0; c4 < RH / 4; ++c4)
                        st_async_cluster_u32x4(dst + (uint32_t)((col0 / 4 + c4) * rows_max + (row - own_lo)) * 16u, tv[4 * c4],
                                               tv[4 * c4 + 1], tv[4 * c4 + 2], tv[4 * c4 + 3], pb);
                }
                wait_bar_cluster(bar(&ctrl->part_full), 0, abort_flag, prm.dev_status);
                if ((uint32_t)owner == crank) {
                    sum_partials<RH>(tv, recv_p + (col0 / 4) * rows_max + (row - own_lo), rows_max, rows_max * R / 4, S, crank);
                    publish_local();
                }
                // (3) my rows are a contiguous piece of each T tile (the swizzle permutes inside a row): two bulk copies
                // per peer carry them over and count their bytes on the peer's barrier
                fence_proxy_async_smem();                       // my rows, written above, are read by the copy engine
                asm volatile("bar.sync 3, 256;" ::: "memory");  // the eight epilogue warps
                if (group == 0) {
                    const int mine_lo = (int)crank * kTileM / (int)S, mine_hi = (int)(crank + 1) * kTileM / (int)S;
                    const uint32_t out_off = (uint32_t)mine_lo * Cfg::kTRowBytes;
                    const uint32_t out_bytes = (uint32_t)(mine_hi - mine_lo) * Cfg::kTRowBytes;
                    if (et == 0) mbar_arrive_expect_tx(bar(&ctrl->part_free), 2u * ((uint32_t)kTileM * Cfg::kTRowBytes - out_bytes));
                    if (warp == kEpiWarp0 && (uint32_t)lane < S && (uint32_t)lane != crank && !*abort_flag) {   // lane q2 serves CTA q2
                        const uint32_t pb = map_to_cta(bar(&ctrl->part_free), (uint32_t)lane);
                        bulk_copy_to_peer(map_to_cta(thi + out_off, (uint32_t)lane), thi + out_off, out_bytes, pb);
                        bulk_copy_to_peer(map_to_cta(tlo + out_off, (uint32_t)lane), tlo + out_off, out_bytes, pb);
                    }
                    wait_bar_cluster(bar(&ctrl->part_free), 0, abort_flag, prm.dev_status);   // all 128 rows of T are here
                    // tell every peer that its rows have arrived: it must not retire while the copy engine still reads them
                    if (warp == kEpiWarp0 && (uint32_t)lane < S && (uint32_t)lane != crank)
                        mbar_arrive_remote(map_to_cta(bar(&ctrl->peers_done), (uint32_t)lane));
                }
            } else {
                publish_local();
            }
            fence_proxy_async_smem();
            tc_fence_before();
            mbar_arrive(bar(&ctrl->t_ready));
        }

        // Copy-out mapping: a warp finishes and stores its OWN 32 rows (the TMEM lanes it reads), so the four warps of a
        // group never wait for one another inside a chunk: piece (lane & 7) of rows q*32 + (lane >> 3) + 4 i.
        const int piece = lane & 7;
        int otok[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) otok[i] = ctrl->rows[q * 32 + (lane >> 3) + 4 * i];
        int wtok[4];                                    // 256-bit variant: rows q*32 + (lane >> 2) + 8 i
#pragma unroll
        for (int i = 0; i < 4; ++i) wtok[i] = ctrl->rows[q * 32 + (lane >> 2) + 8 * i];
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
            __syncwarp();                              // my warp's 32 rows are finished in the stage
            if (!*abort_flag) {
                if (pj.wide_store) {
                    // 32 bytes per lane: four lanes cover a 128-byte row segment, a warp instruction eight rows
                    const int p32 = lane & 3;
                    __nv_bfloat16* dstc = pj.y + (ny0 + nc) * kChunkCols + p32 * 16;
                    uint4 lo4[4], hi4[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t r = (uint32_t)(q * 32 + (lane >> 2) + 8 * i);
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
                            ytile + swizzle_offset((uint32_t)(q * 32 + (lane >> 3) + 4 * i) * 128u + piece * 16, 3));
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        if (otok[i] >= 0) stg128(dstc + (int64_t)otok[i] * pj.ldy, op[i]);
                }
            }
            __syncwarp();                              // every lane has read its pieces
            if (lane == 0) mbar_arrive(bar(&ctrl->empty[s]));   // one of four: the stage may be refilled when all warps are done
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem, kTmemCols);
    // threads that took no part in the exchange complete the start-up cluster barrier here (it has long been
    // passed); no closing barrier is needed, see the exchange
    if (S > 1 && warp < kEpiWarp0) cluster_wait();
    // two-push exchange: my rows of T were copied out of my shared memory by the copy engine; every peer has confirmed
    // their arrival long ago, this wait only makes it certain before the memory is given up
    if (!Cfg::kOnePush && S > 1 && tid == 0) wait_bar_cluster(bar(&ctrl->peers_done), 0, abort_flag, prm.dev_status);
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

template <int R, bool WIDE, int PARTS = 1>
static void fill_launch_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int64_t tiles, int P, int split,
                               cudaStream_t s)
{
    cfg.gridDim = dim3((unsigned)(tiles * split), (unsigned)P, 1);
    cfg.blockDim = dim3(kUmmaThreads, 1, 1);
    cfg.dynamicSmemBytes = UmmaCfg<R, WIDE>::kSmemBytes;
    cfg.stream = s;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

template <int R, bool WIDE, int PARTS>
static cudaError_t umma_launch_variant(UmmaParams prm, int64_t N, UmmaPlan plan, cudaStream_t s)
{
    const int split = plan.split;
    prm.tile_rows = plan.tile_rows;
    using Cfg = UmmaCfg<R, WIDE>;
    static bool configured_dev[kMaxDevices] = {};
    bool& configured = configured_dev[device_slot()];
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(apply_umma_kernel<R, WIDE, PARTS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Cfg::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int64_t tiles = ceil_div64(N, prm.tile_rows) + prm.C;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    fill_launch_config<R, WIDE>(cfg, attr, tiles, prm.P, split, s);
    note_launch();
    return cudaLaunchKernelEx(&cfg, apply_umma_kernel<R, WIDE, PARTS>, prm);
}

// adapters per segment -> the instantiation (stacked rank R = parts x 16 | 32 | 64)
template <int R, bool WIDE>
static cudaError_t umma_launch_parts(const UmmaParams& prm, int64_t N, UmmaPlan plan, cudaStream_t s)
{
    if constexpr (R >= 32) {
        if (prm.parts == 2) return umma_launch_variant<R, WIDE, 2>(prm, N, plan, s);
    }
    if constexpr (R == 64) {
        if (prm.parts == 4) return umma_launch_variant<R, WIDE, 4>(prm, N, plan, s);
    }
    if (prm.parts != 1) return cudaErrorInvalidValue;
    return umma_launch_variant<R, WIDE, 1>(prm, N, plan, s);
}

template <int R>
static cudaError_t umma_launch(const UmmaParams& prm, int64_t N, UmmaPlan plan, cudaStream_t s)
{
    if constexpr (R == 64) {
        if (plan.split > UmmaCfg<64, false>::kMaxSplitR) return umma_launch_parts<64, true>(prm, N, plan, s);
    }
    return umma_launch_parts<R, false>(prm, N, plan, s);
}

// Clusters of `split` CTAs of this kernel that can be resident at once (cached per rank and split).
template <int R, bool WIDE>
static int max_active_clusters_variant(int split)
{
    static int cache_dev[kMaxDevices][kMaxWideSplit + 1] = {};
    int (&cache)[kMaxWideSplit + 1] = cache_dev[device_slot()];
    if (cache[split] == 0) {
        cudaFuncSetAttribute(apply_umma_kernel<R, WIDE, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             UmmaCfg<R, WIDE>::kSmemBytes);
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        fill_launch_config<R, WIDE>(cfg, attr, 148, 1, split, nullptr);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, apply_umma_kernel<R, WIDE, 1>, &cfg) != cudaSuccess || n <= 0) n = 148 / split;
        cache[split] = n;
    }
    return cache[split];
}

template <int R>
static int max_active_clusters(int split)
{
    if constexpr (R == 64) {
        if (split > UmmaCfg<64, false>::kMaxSplitR) return max_active_clusters_variant<64, true>(split);
    }
    return max_active_clusters_variant<R, false>(split);
}

// Largest cluster a tile of rank R may be split over (rank 64: through the variant with the larger exchange buffer).
template <int R>
constexpr int max_split_for_rank() { return R == 64 ? kMaxWideSplit : UmmaCfg<R>::kMaxSplitR; }

// CTAs per tile.  Tiles are 128 rows, so small calls have too few of them for 148 SMs; a tile can be split over a
// cluster (up to 4 CTAs; up to 8 at rank 64).  Pick the split with the smallest estimated time, in microseconds, from a
// model fitted to one-projection 4096 -> 4096 calls at rank 64 (64 ... 4096 tokens, every split, graph replay): a wave of
// resident clusters costs a fixed 9 us (launch, tile look-up, first arrival, last stores), 3 us more for the exchange
// of the partial T tiles, and 0.40 us per 64-column chunk a CTA walks (shrink chunks + expand chunks divided by the
// split); shorter tiles make a chunk only a little cheaper (the gathers are bound by requests in flight, not bytes).
template <int R>
static UmmaPlan choose_split_for_rank(const UmmaParams& prm, int64_t N)
{
    int min_kx = INT32_MAX, nproj = 0;
    double chunks[MOLORA_MAX_PROJECTIONS];         // 64-column chunks a tile of each projection of this rank walks
    for (int i = 0; i < prm.P; ++i) {
        if (prm.p[i].rank != R) continue;
        min_kx = std::min(min_kx, prm.p[i].d_in / kChunkCols);
        chunks[nproj++] = (double)((prm.p[i].d_in + prm.p[i].d_out) / kChunkCols);
    }
    // expected tiles per projection: every segment has at least one and ends in a partial one
    auto tiles_for = [&](int rows) { return std::max<int64_t>(prm.C, ceil_div64(N, rows) + prm.C / 2); };
    // Estimated time of the launch: the CTAs are dispatched heaviest projection first onto the resident clusters, so the
    // launch lasts as long as its heaviest tile or as the whole work spread over the cluster slots (plus a quarter of a
    // light tile of imbalance), whichever is longer; with equal tiles it is whole waves.
    auto cost_for = [&](int rows, int split, bool& one_wave) {
        const int resident = max_active_clusters<R>(split);
        const int64_t tiles = tiles_for(rows);
        // (a chunk costs up to 1.4 times as much once every SM streams: 35 GB/s per SM instead of ~50)
        const double load = std::min(1.0, (double)(tiles * nproj * split) / 148.0);
        const double fixed = 9.0 + (split > 1 ? 3.0 : 0.0);
        const double per_chunk = 0.40 * (1.0 + 0.4 * load * load) * (0.7 + 0.3 * rows / 128.0) / split;
        double cmax = 0.0, cmin = 1e30, total = 0.0;
        for (int i = 0; i < nproj; ++i) {
            const double c = fixed + per_chunk * chunks[i];
            cmax = std::max(cmax, c);
            cmin = std::min(cmin, c);
            total += c * (double)tiles;
        }
        one_wave = tiles * nproj * 1.1 <= resident;         // (margin: the tile count is an estimate)
        if (one_wave) return cmax;
        if (cmax - cmin < 1e-9) return cmax * (double)((tiles * nproj + resident - 1) / resident);
        return std::max(cmax, total / resident + 0.25 * cmin);
    };
    UmmaPlan best = {1, kTileM};
    const int64_t fsplit = tune(kTuneUmmaSplit), frows = tune(kTuneUmmaTileRows);          // tuning overrides
    if (fsplit > 0 || frows > 0) {
        if (fsplit > 0) best.split = (int)std::max<int64_t>(1, std::min<int64_t>(fsplit, max_split_for_rank<R>()));
        if (frows > 0) best.tile_rows = (int)std::max<int64_t>(32, std::min<int64_t>(frows, kTileM));
    } else if (nproj > 0) {
        double best_cost = 1e30;
        bool best_one_wave = false;
        for (int split = 1; split <= max_split_for_rank<R>(); ++split) {    // cluster sizes need not be powers of two
            bool one_wave;
            const double cost = cost_for(kTileM, split, one_wave);
            if (cost < best_cost - 1e-9) { best_cost = cost; best_one_wave = one_wave; best = {split, kTileM}; }
        }
        // A call that does not even fill one wave can use shorter tiles (the MMA tile keeps 128 lanes, the extra
        // lanes idle) to put more SMs to work, as long as everything still fits in one wave.
        if (best_one_wave && tiles_for(kTileM) * nproj * best.split < 0.85 * 148) {
            for (int rows = 96; rows >= 64; rows -= 32)
                for (int split = 1; split <= max_split_for_rank<R>(); ++split) {
                    bool one_wave;
                    const double cost = cost_for(rows, split, one_wave);
                    if (one_wave && cost < best_cost - 1e-9) { best_cost = cost; best = {split, rows}; }
                }
        }
    }
    while (best.split > 1 && min_kx / best.split < 4) --best.split;   // keep at least four chunks of d_in per CTA
    return best;
}

bool group_apply_umma_eligible(int64_t N, int32_t C) { return N >= 1 && N <= kUmmaGroupMaxN && C <= kUmmaAllSegmentsMaxC; }

molora_status_t launch_apply_umma(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                  const int32_t* offsets, const int32_t* perm, uint32_t* dev_status, int32_t min_rows,
                                  cudaStream_t s, const int32_t* r, int32_t* counts_out, int32_t parts, int32_t cbase,
                                  const uint8_t* set_table)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    if (parts < 1 || parts > kUmmaMaxParts) return MOLORA_ERR_INVALID_ARG;
    UmmaParams prm;
    prm.parts = parts;
    prm.cbase = parts > 1 ? cbase : C;
    prm.set_table = set_table;
    if (parts > 1 && set_table == nullptr) return MOLORA_ERR_INVALID_ARG;
    const int32_t n_adapters = parts > 1 ? cbase : C;          // C counts adapter SETS when parts > 1
    // r given: the kernel groups on chip and writes counts / offsets / perm (the pointers are then outputs); one launch
    // only, so every projection must have the same rank
    prm.r = r;
    prm.N = (int32_t)N;
    prm.counts_out = counts_out;
    prm.offsets_out = const_cast<int32_t*>(offsets);
    prm.perm_out = const_cast<int32_t*>(perm);
    if (r != nullptr) {
        if (!group_apply_umma_eligible(N, C) || min_rows > 1) return MOLORA_ERR_UNSUPPORTED;
        for (int i = 1; i < P; ++i)
            if (projs[i].rank != projs[0].rank) return MOLORA_ERR_UNSUPPORTED;
    }
    bool has[3] = {false, false, false};
    // CTAs are dispatched projection by projection (blockIdx.y): put the projections that move the most bytes
    // per tile first, so that the last, partly filled wave consists of the cheap tiles.
    int sorted[MOLORA_MAX_PROJECTIONS], order[MOLORA_MAX_PROJECTIONS], gfirst[MOLORA_MAX_PROJECTIONS], gsize[MOLORA_MAX_PROJECTIONS];
    for (int i = 0; i < P; ++i) sorted[i] = i;
    std::stable_sort(sorted, sorted + P, [&](int a, int b) {
        return (int64_t)projs[a].d_in + 2 * (int64_t)projs[a].d_out > (int64_t)projs[b].d_in + 2 * (int64_t)projs[b].d_out;
    });
    // ... and pull the projections that read the same x (same pointer, pitch, width, rank) and cost the same (same d_out:
    // interleaving tiles of unequal cost would undo the heaviest-first order, which matters more -- two projections of
    // 2048 -> 2048 and 2048 -> 6144 at 16384 tokens: 149 us interleaved against 124 us) next to each other
    {
        bool placed[MOLORA_MAX_PROJECTIONS] = {};
        int n = 0;
        for (int a = 0; a < P; ++a) {
            if (placed[sorted[a]]) continue;
            const int first = n;
            const molora_proj_desc_t& pa = projs[sorted[a]];
            for (int b = a; b < P; ++b) {
                const molora_proj_desc_t& pb = projs[sorted[b]];
                if (placed[sorted[b]] || pb.x != pa.x || pb.ldx != pa.ldx || pb.d_in != pa.d_in || pb.rank != pa.rank ||
                    pb.d_out != pa.d_out)
                    continue;
                placed[sorted[b]] = true;
                order[n++] = sorted[b];
            }
            for (int k = first; k < n; ++k) {
                gfirst[k] = first;
                gsize[k] = n - first;
            }
        }
    }
    for (int i = 0; i < P; ++i) {
        const molora_proj_desc_t& d = projs[order[i]];
        UmmaProj& u = prm.p[i];
        const int32_t rr = d.rank / parts;                    // the adapters' own rank (d.rank is the stacked rank of a set)
        if (rr * parts != d.rank || (rr != 16 && rr != 32 && rr != 64)) return MOLORA_ERR_UNSUPPORTED;
        const CUtensorMapSwizzle wswz = rr == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                        : rr == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
        bool ok = make_tensor_map_bf16_2d(&u.tm_a, d.A, rr, (uint64_t)n_adapters * d.d_in, rr, rr, kChunkCols, wswz);
        ok = ok && make_tensor_map_bf16_2d(&u.tm_b, d.B, d.d_out, (uint64_t)n_adapters * rr, d.d_out, kChunkCols, rr,
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
        u.gfirst = gfirst[i];
        u.gsize = gsize[i];
        has[d.rank == 16 ? 0 : d.rank == 32 ? 1 : 2] = true;
    }
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) {
        prm.p[i].rank = 0;
        prm.p[i].gfirst = i;
        prm.p[i].gsize = 1;
    }
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
