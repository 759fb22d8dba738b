// Grouped LoRA shrink -> expand for decode-sized calls (a few hundred tokens, segments of tens of rows), bf16.
//
// Here the bytes are dominated by y (read + write) and by the adapter stacks, every (segment, projection)
// pair is a small problem, and the whole layer must finish in a few microseconds, so the design goal is many
// small, fully independent CTAs that start streaming at once -- no TMEM, no mbarrier pipeline, no set-up phase:
//
//   tile     up to 32 positions of one segment (two 16-row MMA tiles), owned by a cluster of S <= 4 CTAs
//   shrink   CTA q takes the q-th slice of d_in; its 8 warps take interleaved 32-wide k blocks.  A fragments
//            come straight from global memory (16-byte loads; the k order inside a block is permuted, which a
//            dot product does not mind), the A_c rows of the block are copied by the warp itself into a private
//            shared-memory buffer in the same permuted order and read with ldmatrix.trans.  fp32 partial
//            t[32, R] per warp -> shared-memory sum -> partial per CTA.
//   exchange every CTA pushes its partial into a slot of each peer (distributed shared memory), one hardware
//            cluster barrier, local sum in rank order; t is scaled and split into a bf16 hi/lo A-fragment pair.
//   expand   a cluster covers S * 768 output columns (blockIdx.z selects the slice; wider projections use more
//            clusters and recompute the cheap shrink), CTA q a contiguous 768-column run, its warps interleaved
//            32-column groups, at most three each: B_c[R, 32] is copied
//            by the warp into its private buffer (ldmatrix.trans gives the B fragments), y is read in the
//            accumulator layout before the MMAs, updated in fp32, rounded once and stored at the original rows.
//
// Every request a warp will ever make (its x rows, A_c blocks, B_c groups and y pieces) is issued right at the start,
// so a tile costs about four memory round trips: perm, the loads, the exchange, the stores.
//
// mma.sync.m16n8k16 is the legacy tensor path on sm_100a; it is used here because a decode tile has 9-32 valid
// rows, far below the 128-row tcgen05 tile, and the flops (~0.3 GFLOP per layer) are irrelevant next to the
// bytes.  Everything a warp needs after the exchange is warp-private, so the only block-wide barriers are the
// two around the partial-t sum and the two cluster barriers around the exchange.
#include <stdlib.h>

#include <algorithm>

#include "common.cuh"
#include "sm100_ptx.cuh"

namespace molora {

using namespace ptx;

constexpr int kDecThreads = 256;
constexpr int kDecWarps = 8;
constexpr int kDecRows = 32;              // rows per tile
constexpr int kDecMaxSplit = 4;
constexpr int kDecPermCache = 1024;       // calls with at most this many tokens keep perm in shared memory

struct DecodeParams {
    molora_proj_desc_t p[MOLORA_MAX_PROJECTIONS];
    const int32_t* offsets;
    const int32_t* perm;
    int32_t N;
    int32_t passes;                       // expand passes per CTA: a cluster covers S * passes * (8 warps * GD * 32) columns
    int32_t P, C, max_rows;               // segments with at least max_rows rows belong to the tensor-core kernel
#ifdef MOLORA_TRACE
    long long* trace;                     // development builds only: clock64 stamps per CTA
#endif
};

#ifdef MOLORA_TRACE
#define DEC_TR(slot)                                                                                   \
    do {                                                                                               \
        if (prm.trace != nullptr && threadIdx.x == 0) {                                                \
            const int cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;            \
            if (cta < 2048) prm.trace[cta * 16 + (slot)] = (slot) == 0 ? (long long)clock64() : (long long)clock64(); \
        }                                                                                              \
    } while (0)
#define DEC_GT(slot)                                                                                   \
    do {                                                                                               \
        if (prm.trace != nullptr && threadIdx.x == 0) {                                                \
            const int cta = (blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x;            \
            long long t_;                                                                              \
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                                     \
            if (cta < 2048) prm.trace[cta * 16 + (slot)] = t_;                                         \
        }                                                                                              \
    } while (0)
#else
#define DEC_TR(slot) do { } while (0)
#define DEC_GT(slot) do { } while (0)
#endif

__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// Row of the warp's A_c buffer that holds memory row k (0..31 inside a block): the two k16 steps of a block use
// rows [0,16) and [16,32); inside a step the order matches the k slots of the A fragment built from a 16-byte load.
__device__ __forceinline__ int dec_krow(int k)
{
    const int q = k >> 3, s = (k >> 2) & 1, w = k & 3;
    return s * 16 + (w < 2 ? 2 * q + w : 8 + 2 * q + (w - 2));
}

// Work per warp that is in flight at once: KD k blocks of the shrink and GD 32-column groups of the expand
// (fewer for the larger ranks, whose blocks and groups are bigger: shared memory and registers)
template <int R>
struct DecCfg {
    static constexpr int KD = R == 16 ? 3 : R == 32 ? 2 : 1;
    static constexpr int GD = R == 16 ? 3 : 2;
    static constexpr int COLS_PER_CTA = kDecWarps * GD * 32;     // output columns per CTA (768 for rank 16)
    static constexpr int AROW = R * 2 + 16;                      // padded row pitch (bytes): conflict-free ldmatrix
    static constexpr int BROW = 32 * 2 + 16;
    static constexpr int ABUF = 32 * AROW;                       // one 32-row k block of A_c
    static constexpr int BBUF = R * BROW;                        // one 32-column group of B_c
    static constexpr int WBUF = KD * ABUF + GD * BBUF;           // per warp: separate areas, both phases overlap
    static constexpr int TBYTES = kDecRows * R * 4;              // one fp32 copy of t
    // [8 warp buffers][8 per-warp partial t][slots: one partial t per cluster rank][tfin]
    static constexpr int SMEM = kDecWarps * WBUF + (kDecWarps + kDecMaxSplit + 1) * TBYTES;
};

template <int R>
__global__ void __launch_bounds__(kDecThreads, 2) apply_decode_kernel(const __grid_constant__ DecodeParams prm)
{
    using Cfg = DecCfg<R>;
    constexpr int NT = R / 8;                      // n8 tiles of the shrink
    constexpr int KB = R / 16;                     // k16 blocks of the expand
    constexpr int kDecKD = Cfg::KD, kDecGD = Cfg::GD, kDecColsPerCta = Cfg::COLS_PER_CTA;

    DEC_TR(0);
    DEC_GT(14);
    const molora_proj_desc_t& pd = prm.p[blockIdx.y];
    if (pd.rank != R) return;
    const uint32_t S = cluster_nctarank(), crank = cluster_ctarank();
    // blockIdx.z selects the cluster's slice of d_out (S * 768 columns); projections with fewer slices leave early
    const int ngroups = pd.d_out / 32;
    const int G0 = (int)blockIdx.z * (int)S * prm.passes * (kDecColsPerCta / 32);
    if (G0 >= ngroups) return;
    // One memory round trip brings the segment table and (for small calls) the whole permutation on chip.
    __shared__ int32_t offs_s[MOLORA_MAX_ADAPTERS + 1];
    __shared__ int32_t perm_s[kDecPermCache];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int i = tid; i <= prm.C; i += kDecThreads) offs_s[i] = __ldg(prm.offsets + i);
    const bool perm_cached = prm.N <= kDecPermCache;
    if (perm_cached)
        for (int i = tid; i < prm.N; i += kDecThreads) perm_s[i] = __ldg(prm.perm + i);
    __syncthreads();
    int seg, row0, rows;
    if (!find_tile_smem(offs_s, prm.C, kDecRows, blockIdx.x / S, 1, prm.max_rows, seg, row0, rows)) return;
    DEC_TR(1);
    if (S > 1) cluster_arrive_relaxed();           // "I am running": peers wait for this before writing to my memory

    // dynamic shared memory: [8 warp buffers][8 per-warp partial t][slots: one partial t per cluster rank][tfin]
    extern __shared__ __align__(16) unsigned char dsm[];
    float* tparts = reinterpret_cast<float*>(dsm + kDecWarps * Cfg::WBUF);
    float* slots = tparts + kDecWarps * kDecRows * R;
    float* tfin = slots + kDecMaxSplit * kDecRows * R;

    const int g = lane >> 2, q = lane & 3;
    const bool two = rows > 16;                    // second 16-row MMA tile holds valid rows

    // token rows of this thread's fragment rows: (mt, half) -> tile row mt*16 + g + 8*half; padding repeats the last row
    int64_t tok[2][2];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = mt * 16 + g + 8 * h;
            const int pos = row0 + (r < rows ? r : rows - 1);
            tok[mt][h] = perm_cached ? perm_s[pos] : __ldg(prm.perm + pos);
        }

    const __nv_bfloat16* __restrict__ x = static_cast<const __nv_bfloat16*>(pd.x);
    __nv_bfloat16* __restrict__ y = static_cast<__nv_bfloat16*>(pd.y);
    const __nv_bfloat16* __restrict__ Ac = static_cast<const __nv_bfloat16*>(pd.A) + (int64_t)seg * pd.d_in * R;
    const __nv_bfloat16* __restrict__ Bc = static_cast<const __nv_bfloat16*>(pd.B) + (int64_t)seg * R * pd.d_out;
    const uint32_t wa = smem_u32(dsm + warp * Cfg::WBUF);           // A area of this warp
    const uint32_t wbB = wa + kDecKD * Cfg::ABUF;                   // B area of this warp
    float* tpart = tparts + warp * kDecRows * R;                   // this warp's partial t

    auto stage_A = [&](int slot, int b) {          // 32 rows of A_c (R*2 bytes each), permuted to the fragment order
        constexpr int PIECES = R * 2 / 16;
        for (int e = lane; e < 32 * PIECES; e += 32) {
            const int k = e / PIECES, pc = e - k * PIECES;
            cp_async_16(wa + slot * Cfg::ABUF + dec_krow(k) * Cfg::AROW + pc * 16, Ac + (int64_t)(b * 32 + k) * R + pc * 8);
        }
    };
    // R rows of 32 columns, copied as 16 column pairs per row.  Pair (8 q' + 2 j, +1) goes to position j*4 + q', so
    // that n8 tile j holds the columns {8 q' + 2 j, 8 q' + 2 j + 1}: a thread's accumulator columns over the four
    // tiles of a group are then 8 CONSECUTIVE columns of y (one 16-byte access per row instead of four 4-byte ones).
    auto stage_B = [&](int slot, int grp) {
        for (int e = lane; e < R * 16; e += 32) {
            const int k = e >> 4, pr = e & 15;                          // pr = 4 q' + j
            const int pos = (pr & 3) * 4 + (pr >> 2);
            cp_async_4(wbB + slot * Cfg::BBUF + k * Cfg::BROW + pos * 4, Bc + (int64_t)k * pd.d_out + grp * 32 + pr * 2);
        }
    };
    auto load_x = [&](uint4 (&v)[2][2], int b) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                v[mt][h] = (mt == 0 || two) ? ldg128_stream(x + tok[mt][h] * pd.ldx + b * 32 + q * 8) : make_uint4(0, 0, 0, 0);
    };
    // y for this thread's accumulator columns: [mt][half] = 8 bf16 at (row, grp*32 + 8q); word j belongs to n8 tile j
    auto load_y = [&](uint4 (&v)[2][2], int grp) {
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h)
                v[mt][h] = (mt == 0 || two) ? ld128_rw_stream(y + tok[mt][h] * pd.ldy + grp * 32 + 8 * q) : make_uint4(0, 0, 0, 0);
    };

    DEC_TR(2);
    // my output groups: CTA q owns a contiguous run of groups, its warps interleave inside it
    const int G1 = min(ngroups, G0 + (int)S * prm.passes * (kDecColsPerCta / 32));
    const int per_cta = (G1 - G0 + (int)S - 1) / (int)S;
    const int g_lo = G0 + (int)crank * per_cta, g_hi = min(G1, g_lo + per_cta);

    // ---------------------------------------------------------------- request everything: x, A_c, then B_c and y
    const int kblocks = pd.d_in / 32;
    const int kb0 = (int)(crank * kblocks / S), kb1 = (int)((crank + 1) * kblocks / S);
    uint4 xv[kDecKD][2][2];
    uint4 yv[kDecGD][2][2];
#pragma unroll
    for (int j = 0; j < kDecKD; ++j) {
        const int b = kb0 + warp + j * kDecWarps;
        if (b < kb1) {
            stage_A(j, b);
            load_x(xv[j], b);
        }
    }
    cp_async_commit();
#pragma unroll
    for (int j = 0; j < kDecGD; ++j) {
        const int grp = g_lo + warp + j * kDecWarps;
        if (grp < g_hi) {
            stage_B(j, grp);
            load_y(yv[j], grp);
        }
    }
    cp_async_commit();

    DEC_TR(3);
    // ---------------------------------------------------------------- shrink over my k blocks
    float acc[2][NT][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][n][i] = 0.f;

    auto shrink_block = [&](int slot, const uint4 (&xb)[2][2]) {
#pragma unroll
        for (int s = 0; s < 2; ++s) {                                   // two k16 steps per block
            uint32_t bf[NT / 2][4];
#pragma unroll
            for (int n16 = 0; n16 < NT / 2; ++n16) {
                const int m = lane >> 3;                                // matrix of the x4 load this lane addresses
                ldmatrix_x4_trans(bf[n16], wa + slot * Cfg::ABUF + (s * 16 + (m & 1) * 8 + (lane & 7)) * Cfg::AROW +
                                               (n16 * 16 + (m >> 1) * 8) * 2);
            }
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                if (mt == 0 || two) {
                    uint32_t a[4];
                    a[0] = s ? xb[mt][0].z : xb[mt][0].x;
                    a[2] = s ? xb[mt][0].w : xb[mt][0].y;
                    a[1] = s ? xb[mt][1].z : xb[mt][1].x;
                    a[3] = s ? xb[mt][1].w : xb[mt][1].y;
#pragma unroll
                    for (int n16 = 0; n16 < NT / 2; ++n16) {
                        mma16816(acc[mt][2 * n16], a, bf[n16][0], bf[n16][1]);
                        mma16816(acc[mt][2 * n16 + 1], a, bf[n16][2], bf[n16][3]);
                    }
                }
            }
        }
    };

    cp_async_wait<1>();                                                 // the A_c blocks have landed (B_c may still fly)
    __syncwarp();
    DEC_TR(4);
#pragma unroll
    for (int j = 0; j < kDecKD; ++j)
        if (kb0 + warp + j * kDecWarps < kb1) shrink_block(j, xv[j]);
    // long reductions (d_in / S beyond 24 blocks): further passes of kDecKD blocks, requested one pass at a time
    for (int b0 = kb0 + warp + kDecKD * kDecWarps; b0 < kb1; b0 += kDecKD * kDecWarps) {
        __syncwarp();
#pragma unroll
        for (int j = 0; j < kDecKD; ++j) {
            const int b = b0 + j * kDecWarps;
            if (b < kb1) {
                stage_A(j, b);
                load_x(xv[j], b);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
#pragma unroll
        for (int j = 0; j < kDecKD; ++j)
            if (b0 + j * kDecWarps < kb1) shrink_block(j, xv[j]);
    }
    __syncwarp();

    DEC_TR(5);
    // per-warp partial -> shared memory -> CTA partial -> pushed into every peer's slot of my rank
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            const int c = n * 8 + 2 * q;
            *reinterpret_cast<float2*>(&tpart[(mt * 16 + g) * R + c]) = make_float2(acc[mt][n][0], acc[mt][n][1]);
            *reinterpret_cast<float2*>(&tpart[(mt * 16 + g + 8) * R + c]) = make_float2(acc[mt][n][2], acc[mt][n][3]);
        }
    __syncthreads();
    DEC_TR(6);
    if (S > 1) cluster_wait();                                          // every peer is running
    DEC_TR(7);
    for (int e = tid; e < kDecRows * R; e += kDecThreads) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kDecWarps; ++w) s += tparts[w * kDecRows * R + e];
        if (S > 1) {
            const uint32_t mine = smem_u32(&slots[crank * kDecRows * R + e]);
            for (uint32_t c2 = 0; c2 < S; ++c2) st_cluster_f32(map_to_cta(mine, c2), s);
        } else {
            slots[e] = s;
        }
    }
    DEC_TR(8);
    if (S > 1) cluster_sync_all(); else __syncthreads();              // all partials have arrived in my slots
    DEC_TR(9);
    for (int e = tid; e < kDecRows * R; e += kDecThreads) {
        float s = 0.f;
        for (uint32_t c2 = 0; c2 < S; ++c2) s += slots[c2 * kDecRows * R + e];   // rank order: identical bits in every CTA
        tfin[e] = s * pd.scale;
    }
    __syncthreads();

    DEC_TR(10);
    // A fragments of t for the expand: bf16 hi and lo parts
    uint32_t thi[2][KB][4], tlo[2][KB][4];
#pragma unroll
    for (int mt = 0; mt < 2; ++mt)
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = mt * 16 + g + 8 * (i & 1);
                const int c = kb * 16 + 2 * q + 8 * (i >> 1);
                const float2 t = *reinterpret_cast<const float2*>(&tfin[r * R + c]);
                const float h0 = __bfloat162float(__float2bfloat16_rn(t.x)), h1 = __bfloat162float(__float2bfloat16_rn(t.y));
                thi[mt][kb][i] = f32x2_to_bf16x2(h0, h1);
                tlo[mt][kb][i] = f32x2_to_bf16x2(t.x - h0, t.y - h1);
            }

    // ---------------------------------------------------------------- expand over my 32-column groups
    auto expand_group = [&](int slot, int grp, const uint4 (&yg)[2][2]) {
        float d[2][4][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) d[mt][nt][i] = 0.f;
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            uint32_t bf[2][4];                                          // [n16 pair][b0,b1 of tile 2p, b0,b1 of tile 2p+1]
#pragma unroll
            for (int p2 = 0; p2 < 2; ++p2) {
                const int m = lane >> 3;
                ldmatrix_x4_trans(bf[p2], wbB + slot * Cfg::BBUF + (kb * 16 + (m & 1) * 8 + (lane & 7)) * Cfg::BROW +
                                              (p2 * 16 + (m >> 1) * 8) * 2);
            }
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
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = mt * 16 + g + 8 * h;
                if (r < rows) {
                    const uint32_t yw[4] = {yg[mt][h].x, yg[mt][h].y, yg[mt][h].z, yg[mt][h].w};
                    uint32_t o[4];
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt)
                        o[nt] = f32x2_to_bf16x2(bf16lo_to_f32(yw[nt]) + d[mt][nt][2 * h],
                                                bf16hi_to_f32(yw[nt]) + d[mt][nt][2 * h + 1]);
                    stg128(y + tok[mt][h] * pd.ldy + grp * 32 + 8 * q, make_uint4(o[0], o[1], o[2], o[3]));
                }
            }
    };

    DEC_TR(11);
    cp_async_wait<0>();                                                 // my B_c groups (requested before the shrink)
    __syncwarp();
    DEC_TR(12);
#pragma unroll
    for (int j = 0; j < kDecGD; ++j) {
        const int grp = g_lo + warp + j * kDecWarps;
        if (grp < g_hi) expand_group(j, grp, yv[j]);
    }
    // wide projections: further passes of GD groups per warp, one extra memory round trip each
    for (int gbase = g_lo + warp + kDecGD * kDecWarps; gbase < g_hi; gbase += kDecGD * kDecWarps) {
        __syncwarp();
#pragma unroll
        for (int j = 0; j < kDecGD; ++j) {
            const int grp = gbase + j * kDecWarps;
            if (grp < g_hi) {
                stage_B(j, grp);
                load_y(yv[j], grp);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
        __syncwarp();
#pragma unroll
        for (int j = 0; j < kDecGD; ++j) {
            const int grp = gbase + j * kDecWarps;
            if (grp < g_hi) expand_group(j, grp, yv[j]);
        }
    }
    DEC_TR(13);
    DEC_GT(15);
}

bool decode_eligible(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    return dt == MOLORA_BF16 && (p.rank == 16 || p.rank == 32 || p.rank == 64) && (p.d_in % 32) == 0 && (p.d_out % 32) == 0;
}

template <int R>
constexpr int decode_smem_bytes()
{
    return DecCfg<R>::SMEM;
}

template <int R>
static cudaError_t decode_launch(const DecodeParams& prm, int64_t N, int split, cudaStream_t s)
{
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(apply_decode_kernel<R>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             decode_smem_bytes<R>());
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int64_t cap_rows = prm.max_rows == INT32_MAX ? N : std::min<int64_t>(N, (int64_t)prm.C * prm.max_rows);
    const int64_t tiles = ceil_div64(cap_rows, kDecRows) + prm.C;
    cudaLaunchConfig_t cfg = {};
    int max_dout = 0;
    for (int i = 0; i < prm.P; ++i)
        if (prm.p[i].rank == R) max_dout = std::max(max_dout, prm.p[i].d_out);
    const int nslices = ceil_div(max_dout, split * prm.passes * DecCfg<R>::COLS_PER_CTA);   // clusters along d_out (grid.z)
    cfg.gridDim = dim3((unsigned)(tiles * split), (unsigned)prm.P, (unsigned)nslices);
    cfg.blockDim = dim3(kDecThreads, 1, 1);
    cfg.dynamicSmemBytes = decode_smem_bytes<R>();
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)split;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, apply_decode_kernel<R>, prm);
}

molora_status_t launch_apply_decode(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                    const int32_t* offsets, const int32_t* perm, int32_t max_rows, cudaStream_t s)
{
    if (N == 0 || P == 0) return MOLORA_OK;
    DecodeParams prm;
    bool has[3] = {false, false, false};
    int min_kb = INT32_MAX;
    for (int i = 0; i < P; ++i) {
        prm.p[i] = projs[i];
        has[projs[i].rank == 16 ? 0 : projs[i].rank == 32 ? 1 : 2] = true;
        min_kb = std::min(min_kb, projs[i].d_in / 32);
    }
    for (int i = P; i < MOLORA_MAX_PROJECTIONS; ++i) prm.p[i] = molora_proj_desc_t{};
    prm.offsets = offsets;
    prm.perm = perm;
    prm.P = P;
    prm.C = C;
    prm.max_rows = max_rows;
    prm.N = (int32_t)N;
#ifdef MOLORA_TRACE
    prm.trace = getenv("MOLORA_TRACE_PTR") ? (long long*)strtoull(getenv("MOLORA_TRACE_PTR"), nullptr, 0) : nullptr;
#endif
    // CTAs per tile along d_in: 3 (one wave of CTAs for a 256-token layer of 7 projections), fewer while a warp
    // would be left without a k block; wide projections take up to 3 expand passes per CTA instead of more CTAs.
    int split = 3;
    const char* env = getenv("MOLORA_DECODE_SPLIT");                  // tuning overrides
    if (env != nullptr) split = std::max(1, std::min(atoi(env), kDecMaxSplit));
    while (split > 1 && min_kb / split < kDecWarps) --split;
    const char* envp = getenv("MOLORA_DECODE_PASSES");
    prm.passes = envp != nullptr ? std::max(1, atoi(envp)) : 3;
    cudaError_t e = cudaSuccess;
    if (has[0] && e == cudaSuccess) e = decode_launch<16>(prm, N, split, s);
    if (has[1] && e == cudaSuccess) e = decode_launch<32>(prm, N, split, s);
    if (has[2] && e == cudaSuccess) e = decode_launch<64>(prm, N, split, s);
    return cuda_ok(e);
}

}  // namespace molora
