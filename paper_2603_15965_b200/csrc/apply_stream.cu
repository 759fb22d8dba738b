// Grouped LoRA shrink -> expand for calls below the tcgen05 crossover (Eq. 2, Section 3.3 step 4), bf16, one launch.
//
// A work item is (projection, slice of d_out, tile of <= 32 positions of one segment) and belongs to ONE CTA from
// its first byte to its last: the CTA streams the tile's x rows and A_c through a ring of shared-memory stages,
// keeps t[32, R] on chip, then streams the tile's y rows and B_c through the same ring, updates y in shared memory
// and stores it back.  Nothing is exchanged between CTAs, there is no workspace and no second launch; a projection
// wider than one item re-computes the (cheap, L2-served) shrink per output slice.
//
//   warps 8-11 (copy)    walk the list of chunk jobs of the CTA's items in order -- shrink chunks (512 columns of
//                        the x rows + the matching rows of A_c), then expand chunks (512 columns of the y rows +
//                        B_c) -- and keep the ring full with bulk asynchronous copies, one request per row (each warp
//                        a quarter of the rows and of the weight rows; the SM accepts a request every ~25 cycles and
//                        a warp's lanes issue theirs one after the other), completion counted in bytes on the
//                        stage's "full" mbarrier.  Before a warp refills a stage it waits for the stage's "done"
//                        mbarrier and, if the job in it was an expand chunk, issues the bulk stores of its updated
//                        y rows and waits until they have been read out.  Because the job list runs across items,
//                        the x rows of the next item are in flight while this one expands.
//   warps 0-7 (compute)  shrink chunk: interleaved 32-wide k blocks, ldmatrix + mma.sync.m16n8k16, fp32 partial
//                        t per warp in registers.  After the last shrink chunk the partials are summed in warp order
//                        through that stage's memory (it has been consumed), scaled (and multiplied by the
//                        token's routing weight, if given) and split into bf16 hi + lo A-fragments.
//                        expand chunk: interleaved 32-column groups, y += t B_c in shared memory (fp32 add, one
//                        rounding), then the warp arrives on "done".
//
// Variants: GROUP starts from the routing decisions r and groups on chip (group_inline.cuh) instead of loading offsets
// and perm; SHORT (rank 16) uses 16-row tiles and 1024-column chunks for small calls.
//
// mma.sync is the legacy tensor path on sm_100a; a 32-row tile is far below the 128-row tcgen05 tile, and this path
// is bound by the bytes it moves, not by its flops.  Every wait is bounded; after a time-out the CTA stops issuing
// copies, lets the ones in flight land (bounded again) and returns with MOLORA_DEV_TIMEOUT set.
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "group_inline.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kFsMaxRows = 32;            // most positions of a tile (two 16-row MMA tiles)
constexpr int kFsWarps = 8;               // compute warps
constexpr int kFsCopyWarps = 4;            // each moves 8 rows of the tile and a quarter of the weight rows
constexpr int kFsThreads = (kFsWarps + kFsCopyWarps) * 32;
constexpr double kFsShortFill = 1.25;     // rank 16: short tiles while (16-row tiles x projections) <= this x SMs
constexpr int kFsPermCache = 4096;        // calls with at most this many tokens keep perm in shared memory

struct StreamParams {
    molora_proj_desc_t p[MOLORA_MAX_PROJECTIONS];
    int32_t och[MOLORA_MAX_PROJECTIONS];      // chunks of d_out per item of the projection
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t N, P, C, max_rows;                // segments with at least max_rows rows belong to the tcgen05 kernel
    // Top-k routing in one pass (Eq. 8): a segment is a SET of `parts` adapters (set_table[4 * segment + j] names them, in
    // ascending order), the launch's rank R is parts x the adapters' rank, A_c and B_c are gathered from the
    // parts' adapters, and row_scale holds the routing weights [parts][N].  parts == 1: plain top-1 routing.
    int32_t parts, cbase;
    const uint8_t* set_table;
    // grouping variant only: the routing decisions and where counts / offsets / perm are written (as by molora_group)
    const int32_t* r;
    int32_t* counts_out;
    int32_t* offsets_out;
    int32_t* perm_out;
};
// adapter of part j of segment `seg`
// (set_tab: the kernel's shared-memory copy of prm.set_table)
__device__ __forceinline__ int fs_part_adapter(const StreamParams& prm, const uint8_t* set_tab, int seg, int j)
{
    return prm.parts == 1 ? seg : (int)set_tab[seg * 4 + j];
}
// (projection, slice of d_out) pairs of the projections of the launch's rank; projection p owns [start[p], start[p + 1]).
struct FsUnits {
    int32_t start[MOLORA_MAX_PROJECTIONS + 1];
};

// SHORT (rank 16 only): 16-row tiles and 1024-column chunks instead of 32 rows and 512 columns.
template <int R, bool SHORT>
struct FsCfg {
    static_assert(!SHORT || R == 16, "the short tile exists for rank 16");
    // The SM accepts one bulk-copy request per ~25 cycles whatever its size, so 1 KB requests cap an SM at ~40 B/cycle
    // and an item with a long reduction is bound by them.  The short tile moves 2 KB per request and needs fewer
    // output slices (each of which recomputes the shrink) to fill the SMs of a small call; it reads the weight chunks
    // twice as often per row, which costs more than it saves once every SM has several tiles.
    static constexpr int ROWS = SHORT ? 16 : 32;                 // positions per tile
    static constexpr int MT = ROWS / 16;                         // 16-row MMA tiles
    static constexpr int RPW = ROWS / kFsCopyWarps;              // rows of the tile a copy warp moves
    static constexpr int CH = SHORT ? 1024 : 512;                // columns of a chunk (of d_in or of d_out)
    static constexpr int NSTAGE = SHORT ? 3 : R == 16 ? 4 : R == 32 ? 3 : 2;
    static constexpr int RP = CH * 2 + 16;                       // pitch of a staged x / y / B_c row: 16 bytes of padding
    static constexpr int ROWBYTES = ROWS * RP;                //   keep the 8 rows of an ldmatrix in distinct banks
    static constexpr int ABYTES = CH * R * 2;                    // the chunk's rows of A_c, dense [k][R]
    static constexpr int BBYTES = R * RP;
    static constexpr int STAGE = ROWBYTES + (ABYTES > BBYTES ? ABYTES : BBYTES);
    static constexpr int TFLOATS = ROWS * R;                  // one fp32 copy of t
    static constexpr int SMEM = NSTAGE * STAGE + TFLOATS * 4 + 16;
    static_assert(kFsWarps * TFLOATS * 4 <= STAGE, "the per-warp partials are summed through one stage");
};

namespace {

__device__ __forceinline__ void fs_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void fs_ldsm(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void fs_ldsm_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// barrier of the compute warps only (the copy warp never joins it)
__device__ __forceinline__ void fs_compute_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kFsWarps * 32) : "memory"); }

// One work item, decoded the same way by the copy warp and the compute warps.
struct FsItem {
    int proj, seg, row0, rows;
    int nks;        // shrink chunks
    int ne;         // expand chunks
    int col0;       // first output column
};
__device__ __forceinline__ FsItem fs_item(const StreamParams& prm, const FsUnits& units, const int32_t* offs_s,
                                          const int32_t* tstart_s, int T, int item, int CH, int ROWS)
{
    FsItem it;
    const int unit = item / T, tile = item - unit * T;
    it.proj = 0;
#pragma unroll
    for (int p = 1; p < MOLORA_MAX_PROJECTIONS; ++p)
        if (p < prm.P && unit >= units.start[p]) it.proj = p;
    const int slice = unit - units.start[it.proj];
    it.seg = 0;
    it.row0 = 0;
    it.rows = 1;
    find_tile_bisect(offs_s, tstart_s, prm.C, ROWS, tile, it.seg, it.row0, it.rows);
    const molora_proj_desc_t& pd = prm.p[it.proj];
    it.nks = (pd.d_in + CH - 1) / CH;
    it.col0 = slice * prm.och[it.proj] * CH;
    it.ne = min(prm.och[it.proj], (pd.d_out - it.col0 + CH - 1) / CH);
    return it;
}
__device__ __forceinline__ int fs_token(const StreamParams& prm, const int32_t* perm_s, int pos)
{
    return prm.N <= kFsPermCache ? perm_s[pos] : __ldg(prm.perm + pos);
}

}  // namespace

// GROUP: the call starts from the routing decisions r instead of offsets / perm (at most kFsPermCache tokens).  Every
// CTA then runs the whole grouping (Section 3.3 steps 1-3: histogram, exclusive scan, stable permutation -- the
// algorithm of group_cluster_kernel on one CTA) into its own shared memory before its first copy request, which
// replaces the table load and saves the grouping launch; the CTAs also write counts, offsets and perm out, bit-equal
// to molora_group's, each a slice of perm.
template <int R, bool GROUP, bool SHORT>
__global__ void __launch_bounds__(kFsThreads, 1) apply_stream_kernel(const __grid_constant__ StreamParams prm,
                                                                    const __grid_constant__ FsUnits units)
{
    using Cfg = FsCfg<R, SHORT>;
    constexpr int NS = Cfg::NSTAGE;
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t tstart_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t perm_s[kFsPermCache];
    __shared__ __align__(8) uint64_t full_s[NS], done_s[NS];
    __shared__ unsigned long long st_dst[NS][kFsMaxRows];   // expand job in the stage: where its y rows go back to
    __shared__ uint32_t st_bytes[kFsCopyWarps][NS];      // bytes per row to store (0: a shrink job, nothing to store)
    __shared__ int st_rows[kFsCopyWarps][NS];
    __shared__ int abort_s;
    __shared__ __align__(16) uint8_t set_tab_s[MOLORA_MAX_ADAPTERS * 4];   // adapter sets of top-k routing: set -> adapters
    extern __shared__ __align__(128) unsigned char dsm[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_s[s]), kFsCopyWarps);
            mbar_init(smem_u32(&done_s[s]), kFsWarps);
        }
        abort_s = 0;
        fence_mbar_init();
    }
    if (prm.parts > 1)                         // (visible after the block-wide barriers of the prologue below)
        for (int i = tid; i < prm.C; i += kFsThreads)
            reinterpret_cast<uint32_t*>(set_tab_s)[i] = __ldg(reinterpret_cast<const uint32_t*>(prm.set_table) + i);
    if constexpr (GROUP) {
        // the grouping itself, on this CTA, while the ring is idle (its memory is the scratch)
        group_in_cta<kFsThreads, kFsPermCache>(prm.r, prm.N, prm.C, offs_s, tstart_s, perm_s, dsm, true, prm.counts_out,
                                               prm.offsets_out, prm.perm_out, prm.dev_status);
    } else {
        // segment table and (small calls) the permutation on chip in one memory round trip
        for (int i = tid; i <= prm.C; i += kFsThreads) offs_s[i] = __ldg(prm.offsets + i);
        if (prm.N <= kFsPermCache)
            for (int i = tid; i < prm.N; i += kFsThreads) perm_s[i] = __ldg(prm.perm + i);
        __syncthreads();
    }
    // tiles of the segments before each segment (those with 1 <= rows < max_rows own tiles here), so that an item finds
    // its tile by bisection instead of a walk over all segments
    if (warp == 0) tile_starts(offs_s, prm.C, Cfg::ROWS, 1, prm.max_rows, tstart_s);
    __syncthreads();
    const int T = tstart_s[prm.C];
    const int nitems = T * units.start[prm.P];
    const uint32_t stage0 = smem_u32(dsm);
    float* tfin = reinterpret_cast<float*>(dsm + NS * Cfg::STAGE);

    if (warp >= kFsWarps) {
        // ------------------------------------------------------------------------------------------ copy warps
        // Copy warp w owns RPW consecutive rows of the tile (its first RPW lanes, one bulk request each) and a quarter of the
        // weight rows (lanes 8 ..); the four warps run the same job list without talking to one another -- each
        // arrives once per job on the stage's "full" barrier with the bytes it requested.
        const int cw = warp - kFsWarps;
        constexpr int RPW = Cfg::RPW;
        const int myrow = cw * RPW + (lane % RPW);
        // the stage's previous job is finished: write back my y rows if it was an expand chunk
        auto retire = [&](uint32_t k) {
            const uint32_t s = k % NS;
            wait_bar(smem_u32(&done_s[s]), (k / NS) & 1u, &abort_s, prm.dev_status);
            const uint32_t nb = st_bytes[cw][s];
            if (nb != 0 && !abort_s) {
                if (lane < RPW && myrow < st_rows[cw][s])
                    bulk_store(reinterpret_cast<void*>(st_dst[s][myrow]), stage0 + s * Cfg::STAGE + myrow * Cfg::RP, nb);
                bulk_commit_group();
                bulk_wait_group_read<0>();     // the stage may be overwritten
            }
            __syncwarp();                      // every lane has read the stage's record before lane 0 rewrites it
        };
        uint32_t g = 0;                        // jobs issued so far; job k lives in stage k % NS
        for (int item = blockIdx.x; item < nitems && !abort_s; item += (int)gridDim.x) {
            const FsItem it = fs_item(prm, units, offs_s, tstart_s, T, item, Cfg::CH, Cfg::ROWS);
            const molora_proj_desc_t& pd = prm.p[it.proj];
            const bool rowlane = lane < RPW && myrow < it.rows;
            const int64_t tok = rowlane ? fs_token(prm, perm_s, it.row0 + myrow) : 0;
            const char* xrow = static_cast<const char*>(pd.x) + tok * pd.ldx * 2;
            char* yrow = static_cast<char*>(pd.y) + tok * pd.ldy * 2 + (int64_t)it.col0 * 2;
            const int parts = prm.parts, pr = R / parts;            // adapters per segment, rank of each
            // my weight source: lane RPW + j loads part j's rows of A; the lanes after RPW load one row of B each
            const int apart = min(max(lane - RPW, 0), parts - 1);
            const char* Ac = static_cast<const char*>(pd.A) + (int64_t)fs_part_adapter(prm, set_tab_s, it.seg, apart) * pd.d_in * pr * 2;
            const int brow = cw * (R / kFsCopyWarps) + max(lane - RPW, 0);          // my row of the stacked B (lanes RPW ..)
            const int bpart = min(brow / pr, parts - 1);
            const char* Bc = static_cast<const char*>(pd.B) +
                             (((int64_t)fs_part_adapter(prm, set_tab_s, it.seg, bpart) * pr + (brow - bpart * pr)) * pd.d_out + it.col0) * 2;
            const int myrows = max(0, min(RPW, it.rows - cw * RPW));
            for (int j = 0; j < it.nks + it.ne; ++j, ++g) {
                const uint32_t s = g % NS;
                if (g >= (uint32_t)NS) retire(g - NS);
                if (abort_s) break;
                const uint32_t sb = stage0 + s * Cfg::STAGE, bar = smem_u32(&full_s[s]);
                fence_proxy_async_smem();      // earlier accesses to the stage are ordered before the copies
                if (j < it.nks) {
                    const int k0 = j * Cfg::CH, kc = min(Cfg::CH, pd.d_in - k0);
                    const uint32_t xbytes = (uint32_t)kc * 2u;
                    // my quarter of the chunk's rows of A_c (kc is a multiple of 32: a quarter is a multiple of 16 bytes)
                    const uint32_t ablock = (uint32_t)kc * pr * 2u;                // one part's rows of A for this chunk
                    const uint32_t aq = ablock / kFsCopyWarps;
                    if (lane == 0) {
                        st_bytes[cw][s] = 0;
                        mbar_arrive_expect_tx(bar, (uint32_t)myrows * xbytes + (uint32_t)parts * aq);
                    }
                    __syncwarp();
                    if (rowlane) bulk_load(sb + myrow * Cfg::RP, xrow + (int64_t)k0 * 2, xbytes, bar);
                    if (lane >= RPW && lane < RPW + parts)
                        bulk_load(sb + Cfg::ROWBYTES + apart * ablock + cw * aq, Ac + (int64_t)k0 * pr * 2 + cw * aq, aq, bar);
                } else {
                    const int c0 = (j - it.nks) * Cfg::CH, nc = min(Cfg::CH, pd.d_out - it.col0 - c0);
                    const uint32_t rowbytes = (uint32_t)nc * 2u;
                    if (rowlane) st_dst[s][myrow] = reinterpret_cast<unsigned long long>(yrow + (int64_t)c0 * 2);
                    if (lane == 0) {
                        st_bytes[cw][s] = rowbytes;
                        st_rows[cw][s] = it.rows;
                        mbar_arrive_expect_tx(bar, (uint32_t)(myrows + R / kFsCopyWarps) * rowbytes);
                    }
                    __syncwarp();
                    if (rowlane) bulk_load(sb + myrow * Cfg::RP, yrow + (int64_t)c0 * 2, rowbytes, bar);
                    if (lane >= RPW && lane < RPW + R / kFsCopyWarps) {
                        const int k = cw * (R / kFsCopyWarps) + lane - RPW;
                        bulk_load(sb + Cfg::ROWBYTES + k * Cfg::RP, Bc + (int64_t)c0 * 2, rowbytes, bar);
                    }
                }
            }
        }
        // the jobs still in the ring
        const uint32_t first = g > (uint32_t)NS ? g - NS : 0;
        if (!abort_s)
            for (uint32_t k = first; k < g; ++k) retire(k);
        if (abort_s) {
            // stopped early: give the copies in flight into this CTA's shared memory a bounded chance to land
            for (uint32_t k = first; k < g; ++k) {
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(&full_s[k % NS]), (k / NS) & 1u) && clock64() - t0 < kTimeoutCycles) {
                }
            }
        }
        bulk_wait_group<0>();                  // my stores have completed
        return;
    }

    // ---------------------------------------------------------------------------------------------- compute warps
    constexpr int NT = R / 8;                  // n8 tiles of t
    constexpr int KB = R / 16;                 // k16 blocks of the expand
    constexpr int MT = Cfg::MT;
    const int g4 = lane >> 2, q = lane & 3;
    uint32_t g = 0;
    for (int item = blockIdx.x; item < nitems; item += (int)gridDim.x) {
        const FsItem it = fs_item(prm, units, offs_s, tstart_s, T, item, Cfg::CH, Cfg::ROWS);
        const molora_proj_desc_t& pd = prm.p[it.proj];
        const bool two = MT == 2 && it.rows > 16;   // the second 16-row MMA tile holds valid rows

        // ---- shrink: t = x A_c, fp32 partial per warp
        float acc[MT][NT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][n][i] = 0.f;
        for (int j = 0; j < it.nks; ++j, ++g) {
            const uint32_t s = g % NS;
            const uint32_t xs = stage0 + s * Cfg::STAGE, as = xs + Cfg::ROWBYTES;
            wait_bar(smem_u32(&full_s[s]), (g / NS) & 1u, &abort_s, prm.dev_status);
            const int kcols = min(Cfg::CH, pd.d_in - j * Cfg::CH), nb = kcols / 32;
            const int pr = R / prm.parts;
            for (int b = warp; b < nb; b += kFsWarps) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {                           // two k16 steps per block
                    uint32_t bf[NT / 2][4];
                    const int m = lane >> 3;                            // matrix of the x4 load this lane addresses
#pragma unroll
                    for (int n16 = 0; n16 < NT / 2; ++n16)
                        {
                            // the chunk's rows of A: one dense [k][pr] block per part (pr >= 16: an n16 tile lies in one part)
                            const int part = (n16 * 16) / pr, pc = n16 * 16 - part * pr;
                            fs_ldsm_t(bf[n16], as + part * (kcols * pr * 2) + (b * 32 + h * 16 + (m & 1) * 8 + (lane & 7)) * (pr * 2) +
                                                   (pc + (m >> 1) * 8) * 2);
                        }
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        if (mt == 0 || two) {
                            uint32_t a[4];
                            fs_ldsm(a, xs + (mt * 16 + (lane & 15)) * Cfg::RP + (b * 32 + h * 16 + (lane >> 4) * 8) * 2);
#pragma unroll
                            for (int n16 = 0; n16 < NT / 2; ++n16) {
                                fs_mma(acc[mt][2 * n16], a, bf[n16][0], bf[n16][1]);
                                fs_mma(acc[mt][2 * n16 + 1], a, bf[n16][2], bf[n16][3]);
                            }
                        }
                    }
                }
            }
            if (j + 1 < it.nks) {
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&done_s[s]));
            } else {
                // last chunk: sum the per-warp partials in warp order through this stage, then release it
                float* tparts = reinterpret_cast<float*>(dsm + s * Cfg::STAGE);
                float* tpart = tparts + warp * Cfg::TFLOATS;
                fs_compute_sync();                 // every warp has finished reading the stage (and the previous item's t)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        const int c = n * 8 + 2 * q;
                        *reinterpret_cast<float2*>(&tpart[(mt * 16 + g4) * R + c]) = make_float2(acc[mt][n][0], acc[mt][n][1]);
                        *reinterpret_cast<float2*>(&tpart[(mt * 16 + g4 + 8) * R + c]) = make_float2(acc[mt][n][2], acc[mt][n][3]);
                    }
                fs_compute_sync();
                const float* rscale = pd.row_scale;
                for (int e4 = tid; e4 < Cfg::TFLOATS / 4; e4 += kFsWarps * 32) {
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int w = 0; w < kFsWarps; ++w) {
                        const float4 u = *reinterpret_cast<const float4*>(&tparts[w * Cfg::TFLOATS + e4 * 4]);
                        v.x += u.x;
                        v.y += u.y;
                        v.z += u.z;
                        v.w += u.w;
                    }
                    const int row = e4 * 4 / R;
                    float sc = pd.scale;           // times the token's routing weight, if the caller passes per-token factors
                    if (row >= it.rows) v = make_float4(0.f, 0.f, 0.f, 0.f);   // rows past the tile hold stale shared memory
                    else if (rscale != nullptr)    // (top-k in one pass: the weight of the part this column belongs to)
                        sc *= __ldg(rscale + (int64_t)((e4 * 4 % R) / (R / prm.parts)) * prm.N + fs_token(prm, perm_s, it.row0 + row));
                    *reinterpret_cast<float4*>(&tfin[e4 * 4]) = make_float4(v.x * sc, v.y * sc, v.z * sc, v.w * sc);
                }
                fence_proxy_async_smem();          // my writes to the stage are ordered before the copies that refill it
                fs_compute_sync();                 // t is complete; the stage is free
                if (lane == 0) mbar_arrive(smem_u32(&done_s[s]));
            }
        }

        // ---- A fragments of t: bf16 hi and lo parts
        uint32_t thi[MT][KB][4], tlo[MT][KB][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = mt * 16 + g4 + 8 * (i & 1);
                    const int c = kb * 16 + 2 * q + 8 * (i >> 1);
                    const float2 tv = *reinterpret_cast<const float2*>(&tfin[r * R + c]);
                    const float h0 = __bfloat162float(__float2bfloat16_rn(tv.x)), h1 = __bfloat162float(__float2bfloat16_rn(tv.y));
                    thi[mt][kb][i] = f32x2_to_bf16x2(h0, h1);
                    tlo[mt][kb][i] = f32x2_to_bf16x2(tv.x - h0, tv.y - h1);
                }

        // ---- expand: y += t B_c, chunk by chunk, in shared memory
        for (int e = 0; e < it.ne; ++e, ++g) {
            const uint32_t s = g % NS;
            const uint32_t ys = stage0 + s * Cfg::STAGE, bs = ys + Cfg::ROWBYTES;
            unsigned char* ysp = dsm + s * Cfg::STAGE;
            wait_bar(smem_u32(&full_s[s]), (g / NS) & 1u, &abort_s, prm.dev_status);
            const int ncols = min(Cfg::CH, pd.d_out - it.col0 - e * Cfg::CH);
            // my 32-column groups, GI at a time: y words first, then the MMAs, then add, round once and write back.
            // Rows past the tile hold stale shared memory; they are updated like the others and never stored.
            constexpr int GI = 1;
            const int ngroups = ncols / 32;
            for (int grp0 = warp; grp0 < ngroups; grp0 += GI * kFsWarps) {
                uint32_t yv[GI][MT][2][4];
                float d[GI][MT][4][4];
#pragma unroll
                for (int gi = 0; gi < GI; ++gi) {
                    const int grp = grp0 + gi * kFsWarps;
                    if (grp < ngroups) {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int nt = 0; nt < 4; ++nt)
                                    yv[gi][mt][h][nt] = *reinterpret_cast<const uint32_t*>(
                                        ysp + (mt * 16 + g4 + 8 * h) * Cfg::RP + (grp * 32 + nt * 8 + 2 * q) * 2);
                    }
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) d[gi][mt][nt][i] = 0.f;
                }
#pragma unroll
                for (int gi = 0; gi < GI; ++gi) {
                    const int grp = grp0 + gi * kFsWarps;
                    if (grp < ngroups) {
#pragma unroll
                        for (int kb = 0; kb < KB; ++kb) {
                            uint32_t bf[2][4];                              // [n16 pair][b0,b1 of tile 2p, b0,b1 of tile 2p+1]
                            const int m = lane >> 3;
#pragma unroll
                            for (int p2 = 0; p2 < 2; ++p2)
                                fs_ldsm_t(bf[p2], bs + (kb * 16 + (m & 1) * 8 + (lane & 7)) * Cfg::RP + (grp * 32 + p2 * 16 + (m >> 1) * 8) * 2);
#pragma unroll
                            for (int mt = 0; mt < MT; ++mt) {
                                if (mt == 0 || two) {
#pragma unroll
                                    for (int p2 = 0; p2 < 2; ++p2) {
                                        fs_mma(d[gi][mt][2 * p2], thi[mt][kb], bf[p2][0], bf[p2][1]);
                                        fs_mma(d[gi][mt][2 * p2 + 1], thi[mt][kb], bf[p2][2], bf[p2][3]);
                                    }
#pragma unroll
                                    for (int p2 = 0; p2 < 2; ++p2) {
                                        fs_mma(d[gi][mt][2 * p2], tlo[mt][kb], bf[p2][0], bf[p2][1]);
                                        fs_mma(d[gi][mt][2 * p2 + 1], tlo[mt][kb], bf[p2][2], bf[p2][3]);
                                    }
                                }
                            }
                        }
                    }
                }
                // accumulator element (row g4 + 8h, columns 2q, 2q+1 of n8 tile nt)
#pragma unroll
                for (int gi = 0; gi < GI; ++gi) {
                    const int grp = grp0 + gi * kFsWarps;
                    if (grp < ngroups) {
#pragma unroll
                        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int nt = 0; nt < 4; ++nt) {
                                    const uint32_t v = yv[gi][mt][h][nt];
                                    *reinterpret_cast<uint32_t*>(ysp + (mt * 16 + g4 + 8 * h) * Cfg::RP + (grp * 32 + nt * 8 + 2 * q) * 2) =
                                        f32x2_to_bf16x2(bf16lo_to_f32(v) + d[gi][mt][nt][2 * h], bf16hi_to_f32(v) + d[gi][mt][nt][2 * h + 1]);
                                }
                    }
                }
            }
            fence_proxy_async_smem();              // my updates of y are visible to the bulk stores
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&done_s[s]));
        }
    }
}

// ------------------------------------------------------------------------------------------------ host side
bool stream_eligible(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    return dt == MOLORA_BF16 && (p.rank == 16 || p.rank == 32 || p.rank == 64) && (p.d_in % 32) == 0 && (p.d_out % 32) == 0;
}

template <int R, bool GROUP, bool SHORT>
static cudaError_t stream_launch(StreamParams prm, int64_t N, cudaStream_t s)
{
    using Cfg = FsCfg<R, SHORT>;
    static int slots_dev[kMaxDevices] = {};        // resident CTAs per device: the size of a wave
    int& slots = slots_dev[device_slot()];
    if (slots == 0) {
        cudaError_t e = cudaFuncSetAttribute(apply_stream_kernel<R, GROUP, SHORT>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0, occ = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, apply_stream_kernel<R, GROUP, SHORT>, kFsThreads, Cfg::SMEM);
        slots = std::max(1, sms * occ);
    }
    // every segment adds at most one partial tile; with a row cap only min(N, C * cap) rows can come here
    const int64_t cap_rows = prm.max_rows == INT32_MAX ? N : std::min<int64_t>(N, (int64_t)prm.C * prm.max_rows);
    const int64_t tiles_max = ceil_div64(cap_rows, Cfg::ROWS) + prm.C;
    // Output slices per projection: start with one item per (projection, tile); while the items certainly fit into
    // one wave, split the widest item once more (its shrink is then recomputed per slice).  A second round of
    // items costs more than the imbalance it removes.
    int slices[MOLORA_MAX_PROJECTIONS], chunks[MOLORA_MAX_PROJECTIONS];
    int total = 0;
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        const bool mine = i < prm.P && prm.p[i].rank == R;
        chunks[i] = mine ? ceil_div(prm.p[i].d_out, Cfg::CH) : 0;
        slices[i] = mine ? 1 : 0;
        total += slices[i];
    }
    for (;;) {
        int widest = -1, width = 1;
        for (int i = 0; i < prm.P; ++i) {
            const int w = slices[i] > 0 ? ceil_div(chunks[i], slices[i]) : 0;
            if (w > width) {
                width = w;
                widest = i;
            }
        }
        if (widest < 0 || tiles_max * (total + 1) > slots) break;
        ++slices[widest];
        ++total;
    }
    FsUnits u;
    u.start[0] = 0;
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        prm.och[i] = slices[i] > 0 ? ceil_div(chunks[i], slices[i]) : 0;
        u.start[i + 1] = u.start[i] + (slices[i] > 0 ? ceil_div(chunks[i], prm.och[i]) : 0);
    }
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(tiles_max * u.start[prm.P], slots));
    return launch_kernel(apply_stream_kernel<R, GROUP, SHORT>, dim3(grid), dim3(kFsThreads), Cfg::SMEM, s, 1, false, prm, u);
}

static molora_status_t stream_enqueue(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C, StreamParams& prm,
                                      bool group, cudaStream_t s)
{
    bool has[3] = {false, false, false};
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        prm.p[i] = i < P ? projs[i] : molora_proj_desc_t{};
        prm.och[i] = 0;
        if (i < P) has[projs[i].rank == 16 ? 0 : projs[i].rank == 32 ? 1 : 2] = true;
    }
    prm.P = P;
    prm.C = C;
    prm.N = (int32_t)N;
    if (prm.parts < 1) prm.parts = 1;
    // rank 16: the short tile while its tiles of all projections (nearly) fit one wave of CTAs
    int p16 = 0;
    for (int i = 0; i < P; ++i) p16 += projs[i].rank == 16;
    int sms = 148;
    {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    }
    const int64_t cap_rows = prm.max_rows == INT32_MAX ? N : std::min<int64_t>(N, (int64_t)C * prm.max_rows);
    bool short16 = (ceil_div64(cap_rows, 16) + C) * p16 <= (int64_t)(sms * kFsShortFill);
    if (const int64_t forced = tune(kTuneStreamTile)) short16 = forced == 16;
    cudaError_t e = cudaSuccess;
    if (group) {                                   // one rank only (checked by the caller): one launch does it all
        if (has[0]) e = short16 ? stream_launch<16, true, true>(prm, N, s) : stream_launch<16, true, false>(prm, N, s);
        else if (has[1]) e = stream_launch<32, true, false>(prm, N, s);
        else e = stream_launch<64, true, false>(prm, N, s);
        return cuda_ok(e);
    }
    if (has[0] && e == cudaSuccess)
        e = short16 ? stream_launch<16, false, true>(prm, N, s) : stream_launch<16, false, false>(prm, N, s);
    if (has[1] && e == cudaSuccess) e = stream_launch<32, false, false>(prm, N, s);
    if (has[2] && e == cudaSuccess) e = stream_launch<64, false, false>(prm, N, s);
    return cuda_ok(e);
}

molora_status_t launch_apply_stream(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                    const int32_t* offsets, const int32_t* perm, int32_t max_rows, uint32_t* dev_status,
                                    cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    StreamParams prm;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.max_rows = max_rows;
    prm.r = nullptr;
    prm.counts_out = prm.offsets_out = prm.perm_out = nullptr;
    prm.parts = 1;
    prm.cbase = C;
    prm.set_table = nullptr;
    return stream_enqueue(projs, P, N, C, prm, false, s);
}

// Top-k routing in one pass: `projs` carry the STACKED rank (parts x the adapters' rank) and row_scale = weights
// [parts][N]; offsets / perm group the tokens by adapter set, C_sets = cbase^parts segments.
molora_status_t launch_apply_stream_sets(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t n_sets, int32_t parts,
                                         const uint8_t* set_table, const int32_t* offsets, const int32_t* perm,
                                         uint32_t* dev_status, cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    StreamParams prm;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.max_rows = INT32_MAX;
    prm.r = nullptr;
    prm.counts_out = prm.offsets_out = prm.perm_out = nullptr;
    prm.parts = parts;
    prm.cbase = 0;
    prm.set_table = set_table;
    return stream_enqueue(projs, P, N, n_sets, prm, false, s);
}

// ... and started from the set indices (at most 4096 tokens): grouping by set and apply in one launch.  (Forming the sets
// inside this kernel as well was measured and lost: every CTA repeats the sort, 23.2 against 21.5 us at 4096 tokens.)
molora_status_t launch_group_apply_stream_sets(const int32_t* sets, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                               int32_t n_sets, int32_t parts, const uint8_t* set_table, int32_t* counts,
                                               int32_t* offsets, int32_t* perm, uint32_t* dev_status, cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    StreamParams prm;
    prm.offsets = nullptr;
    prm.perm = nullptr;
    prm.dev_status = dev_status;
    prm.max_rows = INT32_MAX;
    prm.r = sets;
    prm.counts_out = counts;
    prm.offsets_out = offsets;
    prm.perm_out = perm;
    prm.parts = parts;
    prm.cbase = 0;
    prm.set_table = set_table;
    return stream_enqueue(projs, P, N, n_sets, prm, true, s);
}

bool group_apply_stream_eligible(int64_t N) { return N >= 1 && N <= kFsPermCache; }

molora_status_t launch_group_apply_stream(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                          int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm,
                                          uint32_t* dev_status, cudaStream_t s)
{
    StreamParams prm;
    prm.offsets = nullptr;
    prm.perm = nullptr;
    prm.dev_status = dev_status;
    prm.max_rows = INT32_MAX;
    prm.r = r;
    prm.counts_out = counts;
    prm.offsets_out = offsets;
    prm.perm_out = perm;
    prm.parts = 1;
    prm.cbase = C;
    prm.set_table = nullptr;
    return stream_enqueue(projs, P, N, C, prm, true, s);
}

}  // namespace molora
