// Grouped LoRA shrink -> expand for decode-sized calls (Eq. 2, Section 3.3 step 4), bf16, ONE launch whose CTAs share
// the work of every (segment tile, projection) pair instead of owning one each.
//
// A decode layer is a few hundred tokens and several projections: with one CTA per (tile, projection) the launch
// lasts as long as its longest item (a 6144-long reduction, or a 6144-wide expand) while most SMs are done early.
// Here the unit of work is a JOB of one staged chunk (~64 KB of rows + weights):
//
//   shrink job (x-group, tile, chunk of d_in)   x-group = up to 64 / R projections that read the same x (q / k / v,
//       gate / up): the tile's x rows are loaded ONCE and multiplied against the chunk's rows of every member's A_c.
//       The fp32 partial t[16, R] of every member goes to the workspace as 64-bit records {value, tag of this launch}:
//       a 64-bit store is indivisible, so a reader that finds the tag has the value -- no flag, no fence, no second
//       round trip.
//   expand job (projection, tile, chunk of d_out)   its y rows and B_c chunk are requested at once (they depend on
//       nothing); the CTA's t warp polls (bounded) the records of every shrink chunk of its (x-group, tile) until all
//       carry the tag, sums them in chunk order (deterministic), scales, splits into bf16 hi + lo and stages them beside
//       the chunk; the compute warps then update y in shared memory (fp32 add, one rounding) and the copy warps store
//       the rows.
//
// Jobs are numbered shrink jobs first and CTA b takes jobs b, b + gridDim.x, ... in that order, streaming them through
// a ring of three shared-memory stages exactly as the single-launch streaming kernel does (four copy warps issue one
// bulk copy per row, eight compute warps run ldmatrix + mma.sync.m16n8k16).  A shrink job never waits for another CTA,
// and every CTA runs its jobs in increasing order, so every wait on a counter ends as long as all CTAs are resident:
// the launch is cooperative (grid <= resident CTAs), and every wait is bounded in any case.
//
// Workspace (caller-owned, zero-filled before its first use): [control: CTAs finished, launches so far | records].  The
// tag of a launch is 1 + the number of launches that have used the workspace, which the last CTA to finish counts up
// (and it clears the CTA counter), so records left by earlier launches -- of any shape -- never carry the current tag and
// nothing has to be cleared between calls.
#include <algorithm>

#include "common.cuh"
#include "group_inline.cuh"
#include "pipeline.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kJbRows = 16;                // positions per tile (one 16-row MMA tile)
constexpr int kJbWarps = 8;                // compute warps: two teams of four that take alternate jobs of the CTA
constexpr int kJbTeams = 2;
constexpr int kJbTeamWarps = kJbWarps / kJbTeams;
constexpr int kJbCopyWarps = 4;            // each moves 4 rows of the tile and a quarter of the weight rows
constexpr int kJbThreads = (kJbWarps + kJbCopyWarps + 1) * 32;    // + the t warp
constexpr int kJbMaxTokens = 1024;         // perm stays in shared memory
constexpr int kJbStages = 3;
constexpr int kJbStageData = 66048;        // rows + weights of one job
constexpr int kJbMaxChunk = 1024;          // columns of a chunk at most
constexpr int kJbMaxUnits = 256;           // (x-group, chunk) and (projection, chunk) pairs of a launch at most
constexpr int kJbMaxUnitsPerProj = kJbMaxUnits / MOLORA_MAX_PROJECTIONS;
constexpr int kJbCtlBytes = 256;           // control words at the start of the workspace: [0] CTAs finished, [1] launches
constexpr int kJbMaxTiles = kJbMaxTokens / kJbRows + MOLORA_MAX_ADAPTERS;   // every segment adds at most one partial tile

template <int R>
struct JbCfg {
    static constexpr int MAXM = 64 / R;                    // projections that share x in one shrink job
    static constexpr int TP = R * 2 + 16;                  // pitch of a staged row of t (bf16), conflict-free for ldmatrix
    static constexpr int TBYTES = 2 * kJbRows * TP;        // hi and lo
    static constexpr int STAGE = kJbStageData + (TBYTES + 127) / 128 * 128;
    static constexpr int SMEM = kJbStages * STAGE;
    static_assert(kJbTeamWarps * MAXM * kJbRows * R * 4 <= kJbStageData, "the per-warp partials are summed through one stage");
};

struct JobParams {
    molora_proj_desc_t p[MOLORA_MAX_PROJECTIONS];
    int32_t ng;                                            // x-groups
    int32_t gm[MOLORA_MAX_PROJECTIONS];                    // members of the group
    int32_t gmem[MOLORA_MAX_PROJECTIONS][4];               // their projection indices
    int32_t gch[MOLORA_MAX_PROJECTIONS];                   // columns per shrink chunk
    int32_t sstart[MOLORA_MAX_PROJECTIONS + 1];            // shrink chunks of the groups before g
    int32_t pgroup[MOLORA_MAX_PROJECTIONS], pslot[MOLORA_MAX_PROJECTIONS];
    int32_t ech[MOLORA_MAX_PROJECTIONS];                   // columns per expand chunk
    int32_t estart[MOLORA_MAX_PROJECTIONS + 1];            // expand chunks of the projections before p
    int64_t part_off[MOLORA_MAX_PROJECTIONS];              // first record of the group's partials
    uint32_t* ctl;                                         // [0]: CTAs that have finished, [1]: launches that have used the workspace
    unsigned long long* partials;                          // per group: [tile][chunk][member][16][R] records {value, tag}
    const int32_t* offsets;
    const int32_t* perm;
    uint32_t* dev_status;
    int32_t N, P, C, Tmax;
    // grouping variant only: the routing decisions and where counts / offsets / perm are written (as by molora_group)
    const int32_t* r;
    int32_t* counts_out;
    int32_t* offsets_out;
    int32_t* perm_out;
};

namespace {

__device__ __forceinline__ void jb_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm(   // a pure function of its registers: the compiler may schedule it freely
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void jb_ldsm(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void jb_ldsm_t(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// barrier of the compute warps of one team
__device__ __forceinline__ void jb_team_sync(int team) { asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "n"(kJbTeamWarps * 32) : "memory"); }

// A record is one 64-bit word {value: low half, tag: high half}; 64-bit accesses are indivisible, so value and tag
// always travel together.  Two records at a 16-byte aligned address, straight from L2 (another SM may have just
// written them):
__device__ __forceinline__ void ld_records(const unsigned long long* p, unsigned long long& r0, unsigned long long& r1)
{
    asm volatile("ld.relaxed.gpu.global.v2.u64 {%0,%1}, [%2];" : "=l"(r0), "=l"(r1) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_record(unsigned long long* p, float value, uint32_t tag)
{
    const unsigned long long rec = (unsigned long long)__float_as_uint(value) | ((unsigned long long)tag << 32);
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(rec) : "memory");
}

// Decoding a job costs a division, two prefix searches and a bisection; every role of the CTA needs every job of the
// CTA, so the two lookups are tabulated once per CTA after the grouping: tile -> (segment, first position, rows) and
// unit -> (shrink / expand, x-group or projection, chunk, first column, columns).
struct JbJob {
    int expand;     // 0: shrink job of x-group `unit`, 1: expand job of projection `unit`
    int unit;       // x-group or projection
    int chunk;
    int tile, seg, row0, rows;
    int c0, nc;     // first column and columns of the chunk (of d_in or of d_out)
};
// Position of a CTA in its job list: job = unit * T + tile, advanced by gridDim.x without dividing.
struct JbCursor {
    int unit, tile;
    __device__ __forceinline__ void start(int job, int T)
    {
        unit = T > 0 ? job / T : 0;
        tile = job - unit * T;
    }
    __device__ __forceinline__ void next(int gq, int gm, int T)
    {
        unit += gq;
        tile += gm;
        if (tile >= T) {
            tile -= T;
            ++unit;
        }
    }
};
__device__ __forceinline__ JbJob jb_decode(const int4* unit_tab, const int4* tile_tab, const JbCursor& c)
{
    const int4 u = unit_tab[c.unit], t = tile_tab[c.tile];
    JbJob jb;
    jb.expand = u.x & 1;
    jb.unit = u.x >> 1;
    jb.chunk = u.y;
    jb.c0 = u.z;
    jb.nc = u.w;
    jb.tile = c.tile;
    jb.seg = t.x;
    jb.row0 = t.y;
    jb.rows = t.z;
    return jb;
}

}  // namespace

template <int R, bool GROUP>
__global__ void __launch_bounds__(kJbThreads, 1) apply_jobs_kernel(const __grid_constant__ JobParams prm)
{
    using Cfg = JbCfg<R>;
    constexpr int NS = kJbStages;
    constexpr int MAXM = Cfg::MAXM;
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t tstart_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t perm_s[kJbMaxTokens];
    __shared__ int4 tile_tab[kJbMaxTiles];
    __shared__ int4 unit_tab[kJbMaxUnits];
    __shared__ __align__(8) uint64_t full_s[NS], done_s[NS], free_s[NS];
    __shared__ unsigned long long st_dst[NS][kJbRows];      // expand job in the stage: where its y rows go back to
    __shared__ uint32_t st_bytes[kJbCopyWarps][NS];         // bytes per row to store (0: a shrink job, nothing to store)
    __shared__ uint32_t st_pitch[kJbCopyWarps][NS];
    __shared__ int st_rows[kJbCopyWarps][NS];
    __shared__ int abort_s;
    extern __shared__ __align__(128) unsigned char dsm[];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* const aborted = &abort_s;
    if (tid == 0) {
        for (int s = 0; s < NS; ++s) {
            mbar_init(smem_u32(&full_s[s]), kJbCopyWarps + 1);      // four copy warps (with their bytes) + the t warp
            mbar_init(smem_u32(&done_s[s]), kJbTeamWarps);
            mbar_init(smem_u32(&free_s[s]), kJbCopyWarps);
        }
        abort_s = 0;
        fence_mbar_init();
    }
    grid_dependency_wait();                                  // (a no-op unless the launch is programmatic)
    // the launch's tag and the routing decisions are requested first (L2 / DRAM round trips) ...
    const uint32_t tag = __ldcg(prm.ctl + 1) + 1u;          // the launches before this one, + 1: never the tag of an old record
    int warm = 0;
    if (GROUP && prm.N > 0) warm = __ldg(prm.r + min(tid, prm.N - 1));
    // ... and while they travel, the unit table (independent of the routing)
    const int n_sunits = prm.sstart[prm.ng], n_units = n_sunits + prm.estart[prm.P];
    for (int u = tid; u < n_units; u += kJbThreads) {
        int4 e;
        if (u < n_sunits) {
            int g = 0;
#pragma unroll
            for (int k = 1; k < MOLORA_MAX_PROJECTIONS; ++k)
                if (k < prm.ng && u >= prm.sstart[k]) g = k;
            e.x = g << 1;
            e.y = u - prm.sstart[g];
            e.z = e.y * prm.gch[g];
            e.w = min(prm.gch[g], prm.p[prm.gmem[g][0]].d_in - e.z);
        } else {
            const int v = u - n_sunits;
            int p = 0;
#pragma unroll
            for (int k = 1; k < MOLORA_MAX_PROJECTIONS; ++k)
                if (k < prm.P && v >= prm.estart[k]) p = k;
            e.x = (p << 1) | 1;
            e.y = v - prm.estart[p];
            e.z = e.y * prm.ech[p];
            e.w = min(prm.ech[p], prm.p[p].d_out - e.z);
        }
        unit_tab[u] = e;
    }
    asm volatile("" ::"r"(warm));
    if constexpr (GROUP) {
        group_in_cta<kJbThreads, kJbMaxTokens>(prm.r, prm.N, prm.C, offs_s, tstart_s, perm_s, dsm, true, prm.counts_out,
                                               prm.offsets_out, prm.perm_out, prm.dev_status);
    } else {
        for (int i = tid; i <= prm.C; i += kJbThreads) offs_s[i] = __ldg(prm.offsets + i);
        for (int i = tid; i < prm.N; i += kJbThreads) perm_s[i] = __ldg(prm.perm + i);
        __syncthreads();
    }
    if (warp == 0) {                                        // tiles per segment, then every tile's (segment, first position, rows)
        tile_starts(offs_s, prm.C, kJbRows, 1, INT32_MAX, tstart_s);
        __syncwarp();
        const int T0 = tstart_s[prm.C];
        for (int t = lane; t < T0; t += 32) {
            int seg = 0, row0 = 0, rows = 1;
            find_tile_bisect(offs_s, tstart_s, prm.C, kJbRows, t, seg, row0, rows);
            tile_tab[t] = make_int4(seg, row0, rows, 0);
        }
    }
    __syncthreads();
    const int T = tstart_s[prm.C];
    const uint32_t stage0 = smem_u32(dsm);
    const int G = (int)gridDim.x;
    const int gq = T > 0 ? G / T : 0, gm = G - gq * T;      // a step of gridDim.x jobs in (unit, tile) coordinates
    JbCursor cur;
    cur.start((int)blockIdx.x, T);
    if (T == 0) cur.unit = n_units;                         // nothing routed: no jobs

    if (warp >= kJbWarps && warp < kJbWarps + kJbCopyWarps) {
        // ------------------------------------------------------------------------------------------ copy warps
        // Copy warp w owns 4 consecutive rows of the tile (its first 4 lanes, one bulk request each) and a quarter of the
        // weight rows (the lanes after them); the four warps run the same job list.
        const int cw = warp - kJbWarps;
        constexpr int RPW = kJbRows / kJbCopyWarps;
        const int myrow = cw * RPW + (lane % RPW);
        auto retire = [&](uint32_t k) {        // the stage's previous job is finished: write back my y rows
            const uint32_t s = k % NS;
            wait_bar(smem_u32(&done_s[s]), (k / NS) & 1u, &abort_s, prm.dev_status);
            const uint32_t nb = st_bytes[cw][s];
            if (nb != 0 && !*aborted) {
                if (lane < RPW && myrow < st_rows[cw][s])
                    bulk_store(reinterpret_cast<void*>(st_dst[s][myrow]), stage0 + s * Cfg::STAGE + myrow * st_pitch[cw][s], nb);
                bulk_commit_group();
                bulk_wait_group_read<0>();     // my rows have been read out
            }
            __syncwarp();
            // The next job lays the stage out by its own chunk width, so a warp's new copies may land on rows another copy
            // warp still has to store: the stage is free only when all four have read their rows out.
            if (lane == 0) mbar_arrive(smem_u32(&free_s[s]));
            wait_bar(smem_u32(&free_s[s]), (k / NS) & 1u, &abort_s, prm.dev_status);
        };
        uint32_t g = 0;
        for (; cur.unit < n_units && !*aborted; cur.next(gq, gm, T), ++g) {
            const JbJob jb = jb_decode(unit_tab, tile_tab, cur);
            const uint32_t s = g % NS;
            if (g >= (uint32_t)NS) retire(g - NS);
            if (*aborted) break;
            const uint32_t sb = stage0 + s * Cfg::STAGE, bar = smem_u32(&full_s[s]);
            const bool rowlane = lane < RPW && myrow < jb.rows;
            const int64_t tok = rowlane ? perm_s[jb.row0 + myrow] : 0;
            const int myrows = max(0, min(RPW, jb.rows - cw * RPW));
            const uint32_t pitch = (uint32_t)jb.nc * 2u + 16u;
            const uint32_t rowbytes = (uint32_t)jb.nc * 2u;
            fence_proxy_async_smem();          // earlier accesses to the stage are ordered before the copies
            if (!jb.expand) {
                const int m = prm.gm[jb.unit];
                const molora_proj_desc_t& p0 = prm.p[prm.gmem[jb.unit][0]];
                const uint32_t wo = (kJbRows * pitch + 127u) & ~127u;
                const uint32_t ablock = (uint32_t)jb.nc * R * 2u;          // one member's rows of A_c for this chunk
                const uint32_t aq = ablock / kJbCopyWarps;                 // nc is a multiple of 32: a multiple of 16 bytes
                if (lane == 0) {
                    st_bytes[cw][s] = 0;
                    mbar_arrive_expect_tx(bar, (uint32_t)myrows * rowbytes + (uint32_t)m * aq);
                }
                __syncwarp();
                if (rowlane)
                    bulk_load(sb + myrow * pitch, static_cast<const char*>(p0.x) + (tok * p0.ldx + jb.c0) * 2, rowbytes, bar);
                if (lane >= RPW && lane < RPW + m) {
                    const int j = lane - RPW;
                    const molora_proj_desc_t& pj = prm.p[prm.gmem[jb.unit][j]];
                    bulk_load(sb + wo + j * ablock + cw * aq,
                              static_cast<const char*>(pj.A) + ((int64_t)jb.seg * pj.d_in + jb.c0) * R * 2 + cw * aq, aq, bar);
                }
            } else {
                const molora_proj_desc_t& pd = prm.p[jb.unit];
                char* yrow = static_cast<char*>(pd.y) + (tok * pd.ldy + jb.c0) * 2;
                if (rowlane) st_dst[s][myrow] = reinterpret_cast<unsigned long long>(yrow);
                if (lane == 0) {
                    st_bytes[cw][s] = rowbytes;
                    st_pitch[cw][s] = pitch;
                    st_rows[cw][s] = jb.rows;
                    mbar_arrive_expect_tx(bar, (uint32_t)(myrows + R / kJbCopyWarps) * rowbytes);
                }
                __syncwarp();
                if (rowlane) bulk_load(sb + myrow * pitch, yrow, rowbytes, bar);
                if (lane >= RPW && lane < RPW + R / kJbCopyWarps) {
                    const int k = cw * (R / kJbCopyWarps) + lane - RPW;
                    bulk_load(sb + (kJbRows + k) * pitch,
                              static_cast<const char*>(pd.B) + (((int64_t)jb.seg * R + k) * pd.d_out + jb.c0) * 2, rowbytes, bar);
                }
            }
        }
        const uint32_t first = g > (uint32_t)NS ? g - NS : 0;      // the jobs still in the ring
        if (!*aborted)
            for (uint32_t k = first; k < g; ++k) retire(k);
        if (*aborted) {
            // stopped early: give the copies in flight into this CTA's shared memory a bounded chance to land
            for (uint32_t k = first; k < g; ++k) {
                const long long t0 = clock64();
                while (!mbar_try_wait(smem_u32(&full_s[k % NS]), (k / NS) & 1u) && clock64() - t0 < kTimeoutCycles) {
                }
            }
        }
        bulk_wait_group<0>();                  // my stores have completed
    } else if (warp == kJbWarps + kJbCopyWarps) {
        // ------------------------------------------------------------------------------------------ t warp
        // For every expand job: wait for the shrink chunks of its (x-group, tile), sum their partials in chunk order,
        // scale, split into bf16 hi + lo and stage them in the job's stage; then arrive on "full" (also for shrink jobs,
        // where there is nothing to stage).  Lane l holds R / 2 consecutive columns of row l / 2.
        constexpr int CPL = R / 2;
        const int trow = lane >> 1, tcol = (lane & 1) * CPL;
        uint32_t g = 0;
        for (; cur.unit < n_units && !*aborted; cur.next(gq, gm, T), ++g) {
            const JbJob jb = jb_decode(unit_tab, tile_tab, cur);
            const uint32_t s = g % NS;
            if (g >= (uint32_t)NS) wait_bar(smem_u32(&done_s[s]), ((g - NS) / NS) & 1u, &abort_s, prm.dev_status);
            if (*aborted) break;
            if (jb.expand) {
                const molora_proj_desc_t& pd = prm.p[jb.unit];
                const int grp = prm.pgroup[jb.unit], slot = prm.pslot[jb.unit], m = prm.gm[grp];
                const int nk = prm.sstart[grp + 1] - prm.sstart[grp];
                // my CPL records of chunk c: [tile][chunk][member][16][R]
                const unsigned long long* rec = prm.partials + prm.part_off[grp] + ((int64_t)jb.tile * nk * m + slot) * (kJbRows * R) + trow * R + tcol;
                const int64_t cstride = (int64_t)m * (kJbRows * R);
                float v[CPL];
#pragma unroll
                for (int i = 0; i < CPL; ++i) v[i] = 0.f;
                // Blocks of CB chunks: request every record of the block, then look at the tags; a block is summed (in
                // chunk order) only once all of its records carry this launch's tag, otherwise it is requested again.
                constexpr int CB = 32 / CPL >= 1 ? 32 / CPL : 1;      // 32 records (64 registers) in flight per lane
                const long long t0 = clock64();
                for (int c0 = 0; c0 < nk && !*aborted;) {
                    unsigned long long rr[CB][CPL];
                    bool ready = true;
#pragma unroll
                    for (int cb = 0; cb < CB; ++cb)
                        if (c0 + cb < nk) {
#pragma unroll
                            for (int i = 0; i < CPL; i += 2) ld_records(rec + (c0 + cb) * cstride + i, rr[cb][i], rr[cb][i + 1]);
                        }
#pragma unroll
                    for (int cb = 0; cb < CB; ++cb)
                        if (c0 + cb < nk) {
#pragma unroll
                            for (int i = 0; i < CPL; ++i) ready = ready && (uint32_t)(rr[cb][i] >> 32) == tag;
                        }
                    if (__all_sync(0xFFFFFFFFu, ready)) {
#pragma unroll
                        for (int cb = 0; cb < CB; ++cb)
                            if (c0 + cb < nk) {
#pragma unroll
                                for (int i = 0; i < CPL; ++i) v[i] += __uint_as_float((uint32_t)rr[cb][i]);
                            }
                        c0 += CB;
                    } else if (clock64() - t0 > kTimeoutCycles) {
                        *aborted = 1;
                        if (prm.dev_status != nullptr && lane == 0) atomicOr(prm.dev_status, MOLORA_DEV_TIMEOUT);
                    }
                }
                float sc = pd.scale;           // times the token's routing weight, if the caller passes per-token factors
                if (trow < jb.rows && pd.row_scale != nullptr) sc *= __ldg(pd.row_scale + perm_s[jb.row0 + trow]);
                unsigned char* tb = dsm + s * Cfg::STAGE + kJbStageData;
#pragma unroll
                for (int i = 0; i < CPL; i += 8) {
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // rows past the tile hold whatever the stale shared memory of the shrink job gave: force them to 0
                        const float a = trow < jb.rows ? v[i + 2 * e] * sc : 0.f, b = trow < jb.rows ? v[i + 2 * e + 1] * sc : 0.f;
                        const float ha = __bfloat162float(__float2bfloat16_rn(a)), hb = __bfloat162float(__float2bfloat16_rn(b));
                        hi[e] = f32x2_to_bf16x2(ha, hb);
                        lo[e] = f32x2_to_bf16x2(a - ha, b - hb);
                    }
                    *reinterpret_cast<uint4*>(tb + trow * Cfg::TP + (tcol + i) * 2) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(tb + (kJbRows + trow) * Cfg::TP + (tcol + i) * 2) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&full_s[s]));
        }
    } else {
        // ------------------------------------------------------------------------------------------ compute warps
        constexpr int NT = R / 8;                  // n8 tiles of t
        constexpr int KB = R / 16;                 // k16 blocks of the expand
        const int g4 = lane >> 2, q = lane & 3;
        const int mi = lane >> 3;                  // matrix of an x4 ldmatrix this lane addresses
        // Two teams of four warps take alternate jobs: a job's load, MMA and store phases use different pipes, and the
        // two teams are in different phases most of the time.
        const int team = warp / kJbTeamWarps, tw = warp % kJbTeamWarps, ttid = tid - team * (kJbTeamWarps * 32);
        uint32_t g = 0;
        for (; cur.unit < n_units; cur.next(gq, gm, T), ++g) {
            if ((int)(g % kJbTeams) != team) continue;
            const JbJob jb = jb_decode(unit_tab, tile_tab, cur);
            const uint32_t s = g % NS;
            const uint32_t sb = stage0 + s * Cfg::STAGE;
            unsigned char* sp = dsm + s * Cfg::STAGE;
            const uint32_t pitch = (uint32_t)jb.nc * 2u + 16u;
            wait_bar(smem_u32(&full_s[s]), (g / NS) & 1u, &abort_s, prm.dev_status);
            // (after a time-out every wait falls through and the team runs its remaining jobs on whatever the stages hold:
            // nothing of it is stored, and no warp is left alone at a team barrier)
            if (!jb.expand) {
                // ---- shrink chunk: partial t of every member, interleaved 32-wide k blocks per warp.  All fragment loads
                // of a block are issued before its MMAs, so the warp pays the shared-memory latency once per block.
                const int m = prm.gm[jb.unit];
                const uint32_t wo = (kJbRows * pitch + 127u) & ~127u;
                const uint32_t ablock = (uint32_t)jb.nc * R * 2u;
                float acc[MAXM][NT][4];
#pragma unroll
                for (int j = 0; j < MAXM; ++j)
#pragma unroll
                    for (int n = 0; n < NT; ++n)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[j][n][i] = 0.f;
                const int nb = jb.nc / 32;
                const uint32_t xa = sb + (lane & 15) * pitch + (lane >> 4) * 16;
                const uint32_t wa = sb + wo + ((mi & 1) * 8 + (lane & 7)) * (R * 2) + (mi >> 1) * 16;
                for (int b = tw; b < nb; b += kJbTeamWarps) {
                    uint32_t a[2][4];
#pragma unroll
                    for (int h = 0; h < 2; ++h) jb_ldsm(a[h], xa + (b * 32 + h * 16) * 2);
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t bf[MAXM][NT / 2][4];
#pragma unroll
                        for (int j = 0; j < MAXM; ++j)
                            if (j < m) {
#pragma unroll
                                for (int n16 = 0; n16 < NT / 2; ++n16)
                                    jb_ldsm_t(bf[j][n16], wa + j * ablock + (b * 32 + h * 16) * (R * 2) + n16 * 32);
                            }
#pragma unroll
                        for (int j = 0; j < MAXM; ++j)
                            if (j < m) {
#pragma unroll
                                for (int n16 = 0; n16 < NT / 2; ++n16) {
                                    jb_mma(acc[j][2 * n16], a[h], bf[j][n16][0], bf[j][n16][1]);
                                    jb_mma(acc[j][2 * n16 + 1], a[h], bf[j][n16][2], bf[j][n16][3]);
                                }
                            }
                    }
                }
                // sum the per-warp partials in warp order through the stage (it has been consumed) and send the result to the
                // workspace as tagged records
                float* tparts = reinterpret_cast<float*>(sp);
                const int tfl = m * kJbRows * R;                            // floats of one warp's partial
                jb_team_sync(team);                // every warp of the team has finished reading the stage
#pragma unroll
                for (int j = 0; j < MAXM; ++j) {
                    if (j < m) {
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            float* tp = tparts + tw * tfl + j * (kJbRows * R) + n * 8 + 2 * q;
                            *reinterpret_cast<float2*>(tp + g4 * R) = make_float2(acc[j][n][0], acc[j][n][1]);
                            *reinterpret_cast<float2*>(tp + (g4 + 8) * R) = make_float2(acc[j][n][2], acc[j][n][3]);
                        }
                    }
                }
                jb_team_sync(team);
                const int grp = jb.unit;
                const int nk = prm.sstart[grp + 1] - prm.sstart[grp];
                unsigned long long* out = prm.partials + prm.part_off[grp] + ((int64_t)jb.tile * nk + jb.chunk) * tfl;
                for (int e = ttid; e < tfl; e += kJbTeamWarps * 32) {
                    float v = 0.f;
#pragma unroll
                    for (int w = 0; w < kJbTeamWarps; ++w) v += tparts[w * tfl + e];
                    st_record(out + e, v, tag);
                }
                fence_proxy_async_smem();          // my accesses to the stage are ordered before the copies that refill it
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&done_s[s]));
            } else {
                // ---- expand chunk: y += t B_c in shared memory, t from the stage's hi / lo tiles
                const uint32_t tb = sb + kJbStageData;
                uint32_t thi[KB][4], tlo[KB][4];
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    jb_ldsm(thi[kb], tb + (lane & 15) * Cfg::TP + (kb * 16 + (lane >> 4) * 8) * 2);
                    jb_ldsm(tlo[kb], tb + (kJbRows + (lane & 15)) * Cfg::TP + (kb * 16 + (lane >> 4) * 8) * 2);
                }
                constexpr int GI = 1;     // one 32-column group per step: measured faster than two (the MMA and the
                                          // shared-memory pipe do not overlap, a longer step only adds registers)
                const int ngroups = jb.nc / 32;
                // my element of y in a 32-column group: rows g4, g4 + 8; my rows of B_c for the transposed fragment loads
                unsigned char* yp = sp + g4 * pitch + q * 4;
                const uint32_t ba = sb + (kJbRows + (mi & 1) * 8 + (lane & 7)) * pitch + (mi >> 1) * 16;
                for (int grp0 = tw; grp0 < ngroups; grp0 += GI * kJbTeamWarps) {
                    uint32_t yv[GI][2][4];
                    uint32_t bf[GI][KB][2][4];
                    float d[GI][4][4];
                    // every load of the iteration first ...
#pragma unroll
                    for (int gi = 0; gi < GI; ++gi) {
                        const int grp = grp0 + gi * kJbTeamWarps;
                        if (grp < ngroups) {
#pragma unroll
                            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                                for (int p2 = 0; p2 < 2; ++p2)
                                    jb_ldsm_t(bf[gi][kb][p2], ba + kb * 16 * pitch + (grp * 32 + p2 * 16) * 2);
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int nt = 0; nt < 4; ++nt)
                                    yv[gi][h][nt] = *reinterpret_cast<const uint32_t*>(yp + h * 8 * pitch + (grp * 32 + nt * 8) * 2);
                        }
                    }
                    // ... then the MMAs: every hi product before the lo products, so that no MMA waits for its predecessor
#pragma unroll
                    for (int gi = 0; gi < GI; ++gi) {
#pragma unroll
                        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                            for (int i = 0; i < 4; ++i) d[gi][nt][i] = 0.f;
                        const int grp = grp0 + gi * kJbTeamWarps;
                        if (grp < ngroups) {
#pragma unroll
                            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                                for (int p2 = 0; p2 < 2; ++p2) {
                                    jb_mma(d[gi][2 * p2], thi[kb], bf[gi][kb][p2][0], bf[gi][kb][p2][1]);
                                    jb_mma(d[gi][2 * p2 + 1], thi[kb], bf[gi][kb][p2][2], bf[gi][kb][p2][3]);
                                }
#pragma unroll
                            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                                for (int p2 = 0; p2 < 2; ++p2) {
                                    jb_mma(d[gi][2 * p2], tlo[kb], bf[gi][kb][p2][0], bf[gi][kb][p2][1]);
                                    jb_mma(d[gi][2 * p2 + 1], tlo[kb], bf[gi][kb][p2][2], bf[gi][kb][p2][3]);
                                }
                        }
                    }
                    // accumulator element (row g4 + 8h, columns 2q, 2q+1 of n8 tile nt): add, round once, write back
#pragma unroll
                    for (int gi = 0; gi < GI; ++gi) {
                        const int grp = grp0 + gi * kJbTeamWarps;
                        if (grp < ngroups) {
#pragma unroll
                            for (int h = 0; h < 2; ++h)
#pragma unroll
                                for (int nt = 0; nt < 4; ++nt) {
                                    const uint32_t v = yv[gi][h][nt];
                                    *reinterpret_cast<uint32_t*>(yp + h * 8 * pitch + (grp * 32 + nt * 8) * 2) =
                                        f32x2_to_bf16x2(bf16lo_to_f32(v) + d[gi][nt][2 * h], bf16hi_to_f32(v) + d[gi][nt][2 * h + 1]);
                                }
                        }
                    }
                }
                fence_proxy_async_smem();          // my updates of y are visible to the bulk stores
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&done_s[s]));
            }
        }
    }

    // ---- the CTA is done: the last one to get here counts the launch (the next launch's tag) and clears the CTA counter
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(prm.ctl, 1u) == (uint32_t)G - 1u) {
            __threadfence();
            prm.ctl[1] = tag;
            prm.ctl[0] = 0u;
        }
    }
}

// ------------------------------------------------------------------------------------------------ host side
namespace {

// largest chunk (multiple of 32 columns) of a shrink job with m members / of an expand job that fits a stage
int jb_max_shrink_chunk(int rank, int m)
{
    int ch = kJbMaxChunk;
    while (ch > 32 && (size_t)kJbRows * (ch * 2 + 16) + 127 + (size_t)m * ch * rank * 2 > (size_t)kJbStageData) ch -= 32;
    return ch;
}
int jb_max_expand_chunk(int rank)
{
    int ch = kJbMaxChunk;
    while (ch > 32 && (size_t)(kJbRows + rank) * (ch * 2 + 16) > (size_t)kJbStageData) ch -= 32;
    return ch;
}
// chunks of equal size (multiples of 32) that cover d with at most max_chunk columns each
void jb_balanced(int d, int max_chunk, int& chunk, int& count)
{
    count = ceil_div(d, max_chunk);
    chunk = ceil_div(ceil_div(d, count), 32) * 32;
    count = ceil_div(d, chunk);
}
int64_t jb_max_tiles(int64_t N, int32_t C) { return ceil_div64(N, kJbRows) + C; }   // every segment adds at most one partial tile

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

}  // namespace

bool jobs_eligible(const molora_proj_desc_t& p, molora_dtype_t dt, int64_t N)
{
    if (dt != MOLORA_BF16 || (p.rank != 16 && p.rank != 32 && p.rank != 64) || (p.d_in % 32) != 0 || (p.d_out % 32) != 0 ||
        N < 1 || N > kJbMaxTokens)
        return false;
    // the chunks of the projection at the smallest chunk a full x-group gets: the unit table of a launch holds
    // kJbMaxUnits entries for at most MOLORA_MAX_PROJECTIONS projections
    int chunk = 0, ns = 0, ne = 0;
    jb_balanced(p.d_in, jb_max_shrink_chunk(p.rank, 64 / p.rank), chunk, ns);
    jb_balanced(p.d_out, jb_max_expand_chunk(p.rank), chunk, ne);
    return ns + ne <= kJbMaxUnitsPerProj;
}

// Upper bound of the partials one projection adds to a job-list launch, whatever projections it is grouped with (the
// smallest chunk a full x-group gets); the control part at the start of the workspace is jobs_control_bytes() per call.
size_t jobs_partial_bytes(int64_t N, int32_t C, int32_t d_in, int32_t rank)
{
    if (N < 1 || N > kJbMaxTokens) return 0;
    int chunk = 0, count = 0;
    jb_balanced(d_in, jb_max_shrink_chunk(rank, 64 / rank), chunk, count);
    return align256((size_t)jb_max_tiles(N, C) * (size_t)count * kJbRows * rank * sizeof(unsigned long long));
}
size_t jobs_control_bytes() { return kJbCtlBytes; }

template <int R, bool GROUP>
static cudaError_t jobs_launch(const JobParams& prm, int64_t njobs_max, cudaStream_t s)
{
    using Cfg = JbCfg<R>;
    static int slots_dev[kMaxDevices] = {};        // resident CTAs per device: the most a cooperative launch may have
    int& slots = slots_dev[device_slot()];
    if (slots == 0) {
        cudaError_t e = cudaFuncSetAttribute(apply_jobs_kernel<R, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
        if (e != cudaSuccess) return e;
        int dev = 0, sms = 0, occ = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, apply_jobs_kernel<R, GROUP>, kJbThreads, Cfg::SMEM);
        slots = std::max(1, sms * occ);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::max<int64_t>(1, std::min<int64_t>(njobs_max, slots)));
    cfg.blockDim = dim3(kJbThreads);
    cfg.dynamicSmemBytes = Cfg::SMEM;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    const int64_t how = tune(kTuneJobsLaunch);     // 0: cooperative (default); 1: plain; 2: programmatic (measurements only)
    if (how == 2) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
    } else {
        attr[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident at once: a CTA may wait for another's shrink job
        attr[0].val.cooperative = 1;
    }
    cfg.attrs = attr;
    cfg.numAttrs = how == 1 ? 0 : 1;
    note_launch();
    return cudaLaunchKernelEx(&cfg, apply_jobs_kernel<R, GROUP>, prm);
}

// All projections share one rank (checked by the caller).  ctl: the control part of the workspace (jobs_control_bytes(),
// zero between calls); part: room for the partials of this launch.
static molora_status_t jobs_enqueue(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C, JobParams& prm, void* ctl,
                                    void* part, size_t part_bytes, bool group, cudaStream_t s)
{
    const int R = projs[0].rank;
    const int maxm = 64 / R;
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        prm.p[i] = i < P ? projs[i] : molora_proj_desc_t{};
        prm.gm[i] = prm.gch[i] = prm.pgroup[i] = prm.pslot[i] = prm.ech[i] = 0;
        prm.part_off[i] = 0;
        for (int j = 0; j < 4; ++j) prm.gmem[i][j] = 0;
    }
    prm.P = P;
    prm.C = C;
    prm.N = (int32_t)N;
    prm.Tmax = (int32_t)jb_max_tiles(N, C);
    // x-groups: projections that read the same activations, at most 64 / R of them per group
    prm.ng = 0;
    for (int i = 0; i < P; ++i) {
        int g = -1;
        for (int k = 0; k < prm.ng && g < 0; ++k) {
            const molora_proj_desc_t& h = projs[prm.gmem[k][0]];
            if (h.x == projs[i].x && h.ldx == projs[i].ldx && h.d_in == projs[i].d_in && prm.gm[k] < maxm) g = k;
        }
        if (g < 0) g = prm.ng++;
        prm.pgroup[i] = g;
        prm.pslot[i] = prm.gm[g];
        prm.gmem[g][prm.gm[g]++] = i;
    }
    size_t off = 0;
    prm.sstart[0] = 0;
    for (int g = 0; g < MOLORA_MAX_PROJECTIONS; ++g) {
        int chunk = 0, count = 0;
        if (g < prm.ng) {
            jb_balanced(projs[prm.gmem[g][0]].d_in, jb_max_shrink_chunk(R, prm.gm[g]), chunk, count);
            prm.gch[g] = chunk;
            prm.part_off[g] = (int64_t)(off / sizeof(unsigned long long));
            off += align256((size_t)prm.Tmax * count * prm.gm[g] * kJbRows * R * sizeof(unsigned long long));
        }
        prm.sstart[g + 1] = prm.sstart[g] + count;
    }
    prm.estart[0] = 0;
    for (int i = 0; i < MOLORA_MAX_PROJECTIONS; ++i) {
        int chunk = 0, count = 0;
        if (i < P) {
            jb_balanced(projs[i].d_out, jb_max_expand_chunk(R), chunk, count);
            prm.ech[i] = chunk;
        }
        prm.estart[i + 1] = prm.estart[i] + count;
    }
    if (ctl == nullptr || part == nullptr || part_bytes < off || !aligned16(ctl) || !aligned16(part)) return MOLORA_ERR_WORKSPACE;
    prm.ctl = static_cast<uint32_t*>(ctl);
    prm.partials = static_cast<unsigned long long*>(part);
    const int64_t njobs_max = (int64_t)prm.Tmax * (prm.sstart[prm.ng] + prm.estart[P]);
    cudaError_t e;
    if (group) e = R == 16 ? jobs_launch<16, true>(prm, njobs_max, s) : R == 32 ? jobs_launch<32, true>(prm, njobs_max, s) : jobs_launch<64, true>(prm, njobs_max, s);
    else e = R == 16 ? jobs_launch<16, false>(prm, njobs_max, s) : R == 32 ? jobs_launch<32, false>(prm, njobs_max, s) : jobs_launch<64, false>(prm, njobs_max, s);
    return cuda_ok(e);
}

molora_status_t launch_apply_jobs(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C, const int32_t* offsets,
                                  const int32_t* perm, void* ctl, void* part, size_t part_bytes, uint32_t* dev_status,
                                  cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    JobParams prm;
    prm.offsets = offsets;
    prm.perm = perm;
    prm.dev_status = dev_status;
    prm.r = nullptr;
    prm.counts_out = prm.offsets_out = prm.perm_out = nullptr;
    return jobs_enqueue(projs, P, N, C, prm, ctl, part, part_bytes, false, s);
}

molora_status_t launch_group_apply_jobs(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                        int32_t* counts, int32_t* offsets, int32_t* perm, void* ctl, void* part,
                                        size_t part_bytes, uint32_t* dev_status, cudaStream_t s)
{
    JobParams prm;
    prm.offsets = nullptr;
    prm.perm = nullptr;
    prm.dev_status = dev_status;
    prm.r = r;
    prm.counts_out = counts;
    prm.offsets_out = offsets;
    prm.perm_out = perm;
    return jobs_enqueue(projs, P, N, C, prm, ctl, part, part_bytes, true, s);
}

}  // namespace molora
