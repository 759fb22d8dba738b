// Grouped LoRA shrink -> expand for decode-sized calls (a few hundred tokens, segments of tens of rows), bf16.
//
// Here the bytes are dominated by y (read + write) and by the adapter stacks, every (segment, projection) pair
// is a small problem, and the whole layer should finish in a few microseconds.  What decides the time is the
// number of dependent memory round trips, the number of CTA waves and how many bytes each SM keeps in flight,
// so the path is two launches of independent CTAs that move whole row segments with bulk asynchronous copies
// (one request per row of a tile, kilobytes each, tracked by an mbarrier instead of registers):
//
//   shrink_kernel   work item = (projection, tile of <= 32 positions of one segment, slice of d_in).  The grid is
//                   at most one wave of persistent CTAs; each brings offsets and perm on chip once, derives the
//                   list of items from them and takes every gridDim.x-th item.  Per item one warp requests the
//                   x row segments of the tile and the matching rows of A_c into shared memory; the 8 warps then
//                   take interleaved 32-wide k blocks (ldmatrix + mma.sync), their fp32 partial t[32, R] are
//                   summed in warp order and the CTA's partial goes to the workspace
//                   [projection][slice][position][R].
//   expand_kernel   work item = (projection, tile, slice of d_out), persistent CTAs again.  It is launched
//                   programmatically: while the shrink kernel still runs it reads offsets and perm and requests
//                   the y row segments and the B_c rows of its first item; then it waits for the shrink kernel,
//                   sums the partial t of its tile in slice order (the same bits in every CTA), scales, splits
//                   into bf16 hi + lo, runs the MMAs, updates y in shared memory (fp32 add, one rounding) and
//                   writes the row segments back with bulk stores.
//
// Reading offsets, perm, B_c and y before the dependency wait is safe because the predecessor of the expand
// kernel in the stream is always the shrink kernel of the same call, which writes none of them and which lets
// its successor start only after its own dependency wait, i.e. after everything enqueued before it has finished.
//
// mma.sync.m16n8k16 is the legacy tensor path on sm_100a; it is used here because a decode tile has 1-32 valid
// rows, far below the 128-row tcgen05 tile, and the flops (~0.3 GFLOP per layer) are irrelevant next to the bytes.
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "group_inline.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kTpThreads = 256;
constexpr int kTpWarps = 8;
constexpr int kTpRows = 32;               // positions per tile (two 16-row MMA tiles)
constexpr int kTpPermCache = 1024;        // calls with at most this many tokens keep perm in shared memory
constexpr int kTpMaxSlices = 16;          // slices of d_in (longer reductions loop inside the CTA)
constexpr int kTpBulkPiece = 16384;       // largest single bulk copy issued for a contiguous region

struct TwoPhaseParams {
    molora_proj_desc_t p[MOLORA_MAX_PROJECTIONS];
    int64_t t_off[MOLORA_MAX_PROJECTIONS];    // first float of the projection's partials in tws
    int32_t ks[MOLORA_MAX_PROJECTIONS];       // slices of d_in of the projection
    float* tws;                               // [projection][slice][position][R] fp32
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t N, P, C, max_rows;                // segments with at least max_rows rows belong to the tcgen05 kernel
    // grouping variant only: the routing decisions and where counts / offsets / perm are written (as by molora_group)
    const int32_t* r;
    int32_t* counts_out;
    int32_t* offsets_out;
    int32_t* perm_out;
};
// Work-item units: (projection, slice) pairs of the projections of the launch's rank; projection p owns the unit
// indices [start[p], start[p + 1]).
struct TpUnits {
    int32_t start[MOLORA_MAX_PROJECTIONS + 1];
};
__device__ __forceinline__ void tp_unit(const TpUnits& u, int P, int idx, int& proj, int& slice)
{
    proj = 0;
#pragma unroll
    for (int p = 1; p < MOLORA_MAX_PROJECTIONS; ++p)
        if (p < P && idx >= u.start[p]) proj = p;
    slice = idx - u.start[proj];
}

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

// Shared-memory plan of the two kernels.  Row pitches carry 16 extra bytes so that the eight rows of an
// ldmatrix 8x8 matrix (and the eight fragment rows of a 4-byte y access) fall into different banks.
template <int R>
struct TpCfg {
    static constexpr int KBLOCKS = R == 16 ? 32 : 16;            // 32-wide k blocks of a shrink item (one slice)
    static constexpr int XP = KBLOCKS * 64 + 16;                 // pitch of a staged x row (bytes)
    static constexpr int XBYTES = kTpRows * XP;
    static constexpr int ABYTES = KBLOCKS * 32 * R * 2;          // the slice's rows of A_c, dense [k][R]
    static constexpr int TFLOATS = kTpRows * R;                  // one fp32 copy of t
    static constexpr int PARTBYTES = kTpWarps * TFLOATS * 4;     // per-warp partials; reuse the x / A_c area
    static constexpr int SHRINK_SMEM = (XBYTES + ABYTES > PARTBYTES ? XBYTES + ABYTES : PARTBYTES) + 16;
    static constexpr int COLS = R == 16 ? 1024 : 512;            // output columns of an expand item
    static constexpr int YP = COLS * 2 + 16;                     // pitch of a staged y row and of a staged B_c row
    static constexpr int YBYTES = kTpRows * YP;
    static constexpr int BBYTES = R * YP;
    static constexpr int EXPAND_SMEM = YBYTES + BBYTES + TFLOATS * 4 + 16;
};

// Segment table and (for small calls) the permutation on chip in one memory round trip.  Returns the number of
// tiles of the segments that belong to this path (1 <= rows < max_rows): work items are (tile, unit) pairs.
// GROUP: the call starts from the routing decisions r (at most kTpPermCache tokens): every CTA of both kernels runs
// the grouping itself (group_in_cta) in the staging area, which is idle at this point; the shrink kernel's CTAs also
// write counts, offsets and perm out.  The expand kernel recomputes rather than reads them, so that it can still
// request its first item before the shrink kernel has finished.
template <bool GROUP>
__device__ __forceinline__ int tp_load_tables(const TwoPhaseParams& prm, int32_t* offs_s, int32_t* tstart_s, int32_t* perm_s,
                                              unsigned char* scratch, bool write_out)
{
    const int tid = threadIdx.x;
    if constexpr (GROUP) {
        group_in_cta<kTpThreads, kTpPermCache>(prm.r, prm.N, prm.C, offs_s, tstart_s, perm_s, scratch, write_out, prm.counts_out,
                                               prm.offsets_out, prm.perm_out, prm.dev_status);
    } else {
        for (int i = tid; i <= prm.C; i += kTpThreads) offs_s[i] = __ldg(prm.offsets + i);
        if (prm.N <= kTpPermCache)
            for (int i = tid; i < prm.N; i += kTpThreads) perm_s[i] = __ldg(prm.perm + i);
    }
    __syncthreads();
    if (tid < 32) tile_starts(offs_s, prm.C, kTpRows, 1, prm.max_rows, tstart_s);
    __syncthreads();
    return tstart_s[prm.C];
}
struct TpTile {
    int seg, row0, rows;
};
__device__ __forceinline__ int tp_token(const TwoPhaseParams& prm, const int32_t* perm_s, int pos)
{
    return prm.N <= kTpPermCache ? perm_s[pos] : __ldg(prm.perm + pos);
}
// After a wait has given up: give the copies still in flight into this CTA's shared memory one more bounded
// chance to land before the CTA returns.
__device__ __forceinline__ void tp_drain(uint32_t bar, uint32_t parity)
{
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < kTimeoutCycles) {
    }
}

// ------------------------------------------------------------------------------------------------ shrink
template <int R, bool GROUP>
__global__ void __launch_bounds__(kTpThreads, 2) shrink_kernel(const __grid_constant__ TwoPhaseParams prm,
                                                               const __grid_constant__ TpUnits units)
{
    using Cfg = TpCfg<R>;
    constexpr int NT = R / 8;                      // n8 tiles
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t tstart_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t perm_s[kTpPermCache];
    __shared__ __align__(8) uint64_t bar_s;
    __shared__ int abort_s;
    extern __shared__ __align__(128) unsigned char dsm[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const uint32_t bar = smem_u32(&bar_s);
    if (tid == 0) {
        mbar_init(bar, 1);
        abort_s = 0;
        fence_mbar_init();
    }
    grid_dependency_sync();                        // offsets and perm come from the grouping kernel
    const int T = tp_load_tables<GROUP>(prm, offs_s, tstart_s, perm_s, dsm, true);
    const int nitems = T * units.start[prm.P];

    const uint32_t xs = smem_u32(dsm), as = xs + Cfg::XBYTES;
    float* tparts = reinterpret_cast<float*>(dsm);                       // reuses the staging area after the MMAs
    float* tpart = tparts + warp * Cfg::TFLOATS;
    uint32_t parity = 0;
    int dead = 0;

    for (int item = blockIdx.x; item < nitems && !dead; item += (int)gridDim.x) {
        const int unit = item / T, tile = item - unit * T;
        int proj, ks;
        tp_unit(units, prm.P, unit, proj, ks);
        TpTile t;
        find_tile_bisect(offs_s, tstart_s, prm.C, kTpRows, tile, t.seg, t.row0, t.rows);
        const molora_proj_desc_t& pd = prm.p[proj];
        const bool two = t.rows > 16;              // second 16-row MMA tile holds valid rows
        const int kblocks = pd.d_in / 32, KS = prm.ks[proj];
        const int kb0 = (int)((int64_t)ks * kblocks / KS), kb1 = (int)((int64_t)(ks + 1) * kblocks / KS);
        const char* xrow = static_cast<const char*>(pd.x) +
                           (lane < t.rows ? (int64_t)tp_token(prm, perm_s, t.row0 + lane) * pd.ldx * 2 : 0);
        const char* Ac = static_cast<const char*>(pd.A) + (int64_t)t.seg * pd.d_in * R * 2;

        float acc[2][NT][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][n][i] = 0.f;

        // passes of at most KBLOCKS blocks over my slice (one pass unless d_in is very long)
        for (int pb = kb0; pb < kb1; pb += Cfg::KBLOCKS) {
            const int nb = min(Cfg::KBLOCKS, kb1 - pb);
            const uint32_t xbytes = (uint32_t)nb * 64u, abytes = (uint32_t)nb * 32u * R * 2u;
            if (warp == 0) {
                fence_proxy_async_smem();          // earlier accesses to the staging area are ordered before the copies
                if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)t.rows * xbytes + abytes);
                __syncwarp();
                if (lane < t.rows) bulk_load(xs + lane * Cfg::XP, xrow + (int64_t)pb * 64, xbytes, bar);
                for (uint32_t c = lane * kTpBulkPiece; c < abytes; c += 32 * kTpBulkPiece)
                    bulk_load(as + c, Ac + (int64_t)pb * 32 * R * 2 + c, min((uint32_t)kTpBulkPiece, abytes - c), bar);
            }
            wait_bar(bar, parity, &abort_s, prm.dev_status);
            dead = __syncthreads_or(abort_s);
            if (dead) break;
            parity ^= 1u;
            for (int b = warp; b < nb; b += kTpWarps) {
#pragma unroll
                for (int s = 0; s < 2; ++s) {                           // two k16 steps per block
                    uint32_t bf[NT / 2][4];
                    const int m = lane >> 3;                            // matrix of the x4 load this lane addresses
#pragma unroll
                    for (int n16 = 0; n16 < NT / 2; ++n16)
                        ldmatrix_x4_trans(bf[n16], as + (b * 32 + s * 16 + (m & 1) * 8 + (lane & 7)) * (R * 2) +
                                                       (n16 * 16 + (m >> 1) * 8) * 2);
#pragma unroll
                    for (int mt = 0; mt < 2; ++mt) {
                        if (mt == 0 || two) {
                            uint32_t a[4];
                            ldmatrix_x4(a, xs + (mt * 16 + (lane & 15)) * Cfg::XP + (b * 32 + s * 16 + (lane >> 4) * 8) * 2);
#pragma unroll
                            for (int n16 = 0; n16 < NT / 2; ++n16) {
                                mma16816(acc[mt][2 * n16], a, bf[n16][0], bf[n16][1]);
                                mma16816(acc[mt][2 * n16 + 1], a, bf[n16][2], bf[n16][3]);
                            }
                        }
                    }
                }
            }
            __syncthreads();                       // the staging area is free again
        }
        if (dead) break;
        // per-warp partials -> CTA partial (warp order) -> workspace
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                const int c = n * 8 + 2 * q;
                *reinterpret_cast<float2*>(&tpart[(mt * 16 + g) * R + c]) = make_float2(acc[mt][n][0], acc[mt][n][1]);
                *reinterpret_cast<float2*>(&tpart[(mt * 16 + g + 8) * R + c]) = make_float2(acc[mt][n][2], acc[mt][n][3]);
            }
        __syncthreads();
        float* out = prm.tws + prm.t_off[proj] + ((int64_t)ks * prm.N + t.row0) * R;   // rows of a tile are contiguous
        for (int e4 = tid; e4 < t.rows * R / 4; e4 += kTpThreads) {
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int w = 0; w < kTpWarps; ++w) {
                const float4 v = *reinterpret_cast<const float4*>(&tparts[w * Cfg::TFLOATS + e4 * 4]);
                s.x += v.x;
                s.y += v.y;
                s.z += v.z;
                s.w += v.w;
            }
            *reinterpret_cast<float4*>(out + e4 * 4) = s;
        }
        __syncthreads();                           // the partials may be overwritten by the next item's copies
    }
    if (dead && tid == 0) tp_drain(bar, parity);
}

// ------------------------------------------------------------------------------------------------ expand
template <int R, bool GROUP>
__global__ void __launch_bounds__(kTpThreads, 2) expand_kernel(const __grid_constant__ TwoPhaseParams prm,
                                                               const __grid_constant__ TpUnits units)
{
    using Cfg = TpCfg<R>;
    constexpr int KB = R / 16;                     // k16 blocks
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t tstart_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t perm_s[kTpPermCache];
    __shared__ __align__(8) uint64_t bar_s;
    __shared__ int abort_s;
    extern __shared__ __align__(128) unsigned char dsm[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, q = lane & 3;
    const uint32_t bar = smem_u32(&bar_s);
    if (tid == 0) {
        mbar_init(bar, 1);
        abort_s = 0;
        fence_mbar_init();
    }
    // Nothing read before the dependency wait below is written by the shrink kernel (see the file header).
    const int T = tp_load_tables<GROUP>(prm, offs_s, tstart_s, perm_s, dsm, false);
    const int nitems = T * units.start[prm.P];

    const uint32_t ys = smem_u32(dsm), bs = ys + Cfg::YBYTES;
    unsigned char* ysp = dsm;
    float* tfin = reinterpret_cast<float*>(dsm + Cfg::YBYTES + Cfg::BBYTES);

    // ---- the item in flight
    int proj = 0, ncols = 0;
    TpTile t = {0, 0, 1};
    char* yrow = nullptr;                          // lane r: start of the item's segment of tile row r in y

    auto request = [&](int item) {                 // decode the item; one warp requests its y row segments and B_c rows
        const int unit = item / T, tile = item - unit * T;
        int slice;
        tp_unit(units, prm.P, unit, proj, slice);
        find_tile_bisect(offs_s, tstart_s, prm.C, kTpRows, tile, t.seg, t.row0, t.rows);
        const molora_proj_desc_t& pd = prm.p[proj];
        const int col0 = slice * Cfg::COLS;
        ncols = min(Cfg::COLS, pd.d_out - col0);
        yrow = static_cast<char*>(pd.y) + (int64_t)col0 * 2 +
               (lane < t.rows ? (int64_t)tp_token(prm, perm_s, t.row0 + lane) * pd.ldy * 2 : 0);
        if (warp == 0) {
            const char* Bc = static_cast<const char*>(pd.B) + ((int64_t)t.seg * R * pd.d_out + col0) * 2;
            const uint32_t rowbytes = (uint32_t)ncols * 2u;
            fence_proxy_async_smem();              // earlier accesses to the staging area are ordered before the copies
            if (lane == 0) mbar_arrive_expect_tx(bar, (uint32_t)(t.rows + R) * rowbytes);
            __syncwarp();
            if (lane < t.rows) bulk_load(ys + lane * Cfg::YP, yrow, rowbytes, bar);
            for (int k = lane; k < R; k += 32) bulk_load(bs + k * Cfg::YP, Bc + (int64_t)k * pd.d_out * 2, rowbytes, bar);
        }
    };

    int item = blockIdx.x;
    if (item < nitems) request(item);
    grid_dependency_sync();                        // the partial t of the shrink kernel are complete and visible

    uint32_t parity = 0;
    int dead = 0;
    while (item < nitems) {
        // t of my tile: partials summed in slice order, scaled
        {
            const int KS = prm.ks[proj];
            const float scale = prm.p[proj].scale;
            const float* rscale = prm.p[proj].row_scale;
            const float* part = prm.tws + prm.t_off[proj] + (int64_t)t.row0 * R;
            const int64_t slice_stride = (int64_t)prm.N * R;
            for (int e4 = tid; e4 < Cfg::TFLOATS / 4; e4 += kTpThreads) {
                float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
                if (e4 * 4 < t.rows * R) {
                    for (int k0 = 0; k0 < KS; k0 += 4) {           // four slices in flight at once, summed in slice order
                        float4 v[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (k0 + k < KS) v[k] = __ldcg(reinterpret_cast<const float4*>(part + (k0 + k) * slice_stride + e4 * 4));
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (k0 + k < KS) {
                                s.x += v[k].x;
                                s.y += v[k].y;
                                s.z += v[k].z;
                                s.w += v[k].w;
                            }
                    }
                }
                float sc = scale;                   // times the token's routing weight, if the caller passes per-token factors
                if (rscale != nullptr && e4 * 4 < t.rows * R) sc *= __ldg(rscale + tp_token(prm, perm_s, t.row0 + e4 * 4 / R));
                *reinterpret_cast<float4*>(&tfin[e4 * 4]) = make_float4(s.x * sc, s.y * sc, s.z * sc, s.w * sc);
            }
        }
        wait_bar(bar, parity, &abort_s, prm.dev_status);
        dead = __syncthreads_or(abort_s);          // also publishes t
        if (dead) break;
        parity ^= 1u;
        // A fragments of t: bf16 hi and lo parts
        uint32_t thi[2][KB][4], tlo[2][KB][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = mt * 16 + g + 8 * (i & 1);
                    const int c = kb * 16 + 2 * q + 8 * (i >> 1);
                    const float2 tv = *reinterpret_cast<const float2*>(&tfin[r * R + c]);
                    const float h0 = __bfloat162float(__float2bfloat16_rn(tv.x)), h1 = __bfloat162float(__float2bfloat16_rn(tv.y));
                    thi[mt][kb][i] = f32x2_to_bf16x2(h0, h1);
                    tlo[mt][kb][i] = f32x2_to_bf16x2(tv.x - h0, tv.y - h1);
                }
        const bool two = t.rows > 16;
        for (int grp = warp; grp < ncols / 32; grp += kTpWarps) {       // my 32-column groups
            float d[2][4][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) d[mt][nt][i] = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                uint32_t bf[2][4];                                      // [n16 pair][b0,b1 of tile 2p, b0,b1 of tile 2p+1]
                const int m = lane >> 3;
#pragma unroll
                for (int p2 = 0; p2 < 2; ++p2)
                    ldmatrix_x4_trans(bf[p2], bs + (kb * 16 + (m & 1) * 8 + (lane & 7)) * Cfg::YP +
                                                  (grp * 32 + p2 * 16 + (m >> 1) * 8) * 2);
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    if (mt == 0 || two) {
#pragma unroll
                        for (int p2 = 0; p2 < 2; ++p2) {
                            mma16816(d[mt][2 * p2], thi[mt][kb], bf[p2][0], bf[p2][1]);
                            mma16816(d[mt][2 * p2], tlo[mt][kb], bf[p2][0], bf[p2][1]);
                            mma16816(d[mt][2 * p2 + 1], thi[mt][kb], bf[p2][2], bf[p2][3]);
                            mma16816(d[mt][2 * p2 + 1], tlo[mt][kb], bf[p2][2], bf[p2][3]);
                        }
                    }
                }
            }
            // y += delta in shared memory: accumulator (row g + 8h, columns 2q, 2q+1 of n8 tile nt), one rounding
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int r = mt * 16 + g + 8 * h;
                    if (r < t.rows) {
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt) {
                            uint32_t* w = reinterpret_cast<uint32_t*>(ysp + r * Cfg::YP + (grp * 32 + nt * 8 + 2 * q) * 2);
                            const uint32_t v = *w;
                            *w = f32x2_to_bf16x2(bf16lo_to_f32(v) + d[mt][nt][2 * h], bf16hi_to_f32(v) + d[mt][nt][2 * h + 1]);
                        }
                    }
                }
        }
        fence_proxy_async_smem();                  // my updates of y are visible to the bulk stores
        __syncthreads();
        if (warp == 0) {
            if (lane < t.rows) bulk_store(yrow, ys + lane * Cfg::YP, (uint32_t)ncols * 2u);
            bulk_commit_group();
            bulk_wait_group_read<0>();             // the staging area may be overwritten
        }
        __syncthreads();
        item += (int)gridDim.x;
        if (item < nitems) request(item);
    }
    if (warp == 0) bulk_wait_group<0>();           // my stores have completed
    if (dead && tid == 0) tp_drain(bar, parity);
}

// ------------------------------------------------------------------------------------------------ host side
bool decode_eligible(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    return dt == MOLORA_BF16 && (p.rank == 16 || p.rank == 32 || p.rank == 64) && (p.d_in % 32) == 0 && (p.d_out % 32) == 0;
}

static int shrink_slices(int d_in, int rank)
{
    const int per_item = rank == 16 ? TpCfg<16>::KBLOCKS : rank == 32 ? TpCfg<32>::KBLOCKS : TpCfg<64>::KBLOCKS;
    return std::max(1, std::min(kTpMaxSlices, ceil_div(d_in / 32, per_item)));
}

static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

size_t decode_workspace_bytes(int64_t N, int32_t d_in, int32_t rank)
{
    return align256((size_t)shrink_slices(d_in, rank) * (size_t)N * (size_t)rank * sizeof(float));
}

template <int R, bool GROUP>
static cudaError_t twophase_launch(const TwoPhaseParams& prm, int64_t N, cudaStream_t s)
{
    static_assert(kGroupInCtaTableMaxC * kTpThreads * 4 + 4 * kGroupInCtaTableMaxC <= TpCfg<R>::SHRINK_SMEM &&
                      kGroupInCtaTableMaxC * kTpThreads * 4 + 4 * kGroupInCtaTableMaxC <= TpCfg<R>::EXPAND_SMEM,
                  "the grouping scratch fits the staging areas");
    using Cfg = TpCfg<R>;
    // resident CTAs of each kernel on this device: the size of a wave
    static int wave_dev[kMaxDevices][2] = {};
    int (&wave)[2] = wave_dev[device_slot()];
    if (wave[0] == 0) {
        cudaError_t e = cudaFuncSetAttribute(shrink_kernel<R, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SHRINK_SMEM);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(expand_kernel<R, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::EXPAND_SMEM);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0, occ_s = 0, occ_e = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_s, shrink_kernel<R, GROUP>, kTpThreads, Cfg::SHRINK_SMEM);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_e, expand_kernel<R, GROUP>, kTpThreads, Cfg::EXPAND_SMEM);
        wave[1] = std::max(1, sms * occ_e);
        wave[0] = std::max(1, sms * occ_s);
    }
    // every segment adds at most one partial tile; with a row cap only min(N, C * cap) rows can come here
    const int64_t cap_rows = prm.max_rows == INT32_MAX ? N : std::min<int64_t>(N, (int64_t)prm.C * prm.max_rows);
    const int64_t tiles = ceil_div64(cap_rows, kTpRows) + prm.C;
    TpUnits su, eu;                                // (projection, slice) pairs of this rank's projections
    su.start[0] = eu.start[0] = 0;
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        const bool mine = i < prm.P && prm.p[i].rank == R;
        su.start[i + 1] = su.start[i] + (mine ? prm.ks[i] : 0);
        eu.start[i + 1] = eu.start[i] + (mine ? ceil_div(prm.p[i].d_out, Cfg::COLS) : 0);
    }
    const unsigned grid_s = (unsigned)std::min<int64_t>(tiles * su.start[prm.P], wave[0]);
    const unsigned grid_e = (unsigned)std::min<int64_t>(tiles * eu.start[prm.P], wave[1]);
    cudaError_t e = launch_kernel(shrink_kernel<R, GROUP>, dim3(grid_s), dim3(kTpThreads), Cfg::SHRINK_SMEM, s, 1, false, prm, su);
    if (e != cudaSuccess) return e;
    return launch_kernel(expand_kernel<R, GROUP>, dim3(grid_e), dim3(kTpThreads), Cfg::EXPAND_SMEM, s, 1, true, prm, eu);
}

static molora_status_t decode_enqueue(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C, TwoPhaseParams& prm,
                                      void* ws, size_t ws_bytes, bool group, cudaStream_t s)
{
    bool has[3] = {false, false, false};
    size_t need = 0;
    for (int i = 0; i < P; ++i) {
        prm.p[i] = projs[i];
        prm.ks[i] = shrink_slices(projs[i].d_in, projs[i].rank);
        prm.t_off[i] = (int64_t)(need / sizeof(float));
        need += decode_workspace_bytes(N, projs[i].d_in, projs[i].rank);
        has[projs[i].rank == 16 ? 0 : projs[i].rank == 32 ? 1 : 2] = true;
    }
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) {
        prm.p[i] = molora_proj_desc_t{};
        prm.ks[i] = 0;
        prm.t_off[i] = 0;
    }
    if (ws == nullptr || ws_bytes < need || !aligned16(ws)) return MOLORA_ERR_WORKSPACE;
    prm.tws = static_cast<float*>(ws);
    prm.P = P;
    prm.C = C;
    prm.N = (int32_t)N;
    cudaError_t e = cudaSuccess;
    if (group) {                                   // one rank only (checked by the caller)
        if (has[0]) e = twophase_launch<16, true>(prm, N, s);
        else if (has[1]) e = twophase_launch<32, true>(prm, N, s);
        else e = twophase_launch<64, true>(prm, N, s);
        return cuda_ok(e);
    }
    if (has[0] && e == cudaSuccess) e = twophase_launch<16, false>(prm, N, s);
    if (has[1] && e == cudaSuccess) e = twophase_launch<32, false>(prm, N, s);
    if (has[2] && e == cudaSuccess) e = twophase_launch<64, false>(prm, N, s);
    return cuda_ok(e);
}

molora_status_t launch_apply_decode(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                    const int32_t* offsets, const int32_t* perm, int32_t max_rows, void* ws,
                                    size_t ws_bytes, uint32_t* dev_status, cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    TwoPhaseParams prm;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.max_rows = max_rows;
    prm.r = nullptr;
    prm.counts_out = prm.offsets_out = prm.perm_out = nullptr;
    return decode_enqueue(projs, P, N, C, prm, ws, ws_bytes, false, s);
}

bool group_apply_decode_eligible(int64_t N) { return N >= 1 && N <= kTpPermCache; }

molora_status_t launch_group_apply_decode(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                          int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm, void* ws,
                                          size_t ws_bytes, uint32_t* dev_status, cudaStream_t s)
{
    TwoPhaseParams prm;
    prm.offsets = nullptr;
    prm.perm = nullptr;
    prm.dev_status = dev_status;
    prm.max_rows = INT32_MAX;
    prm.r = r;
    prm.counts_out = counts;
    prm.offsets_out = offsets;
    prm.perm_out = perm;
    return decode_enqueue(projs, P, N, C, prm, ws, ws_bytes, true, s);
}

}  // namespace molora
