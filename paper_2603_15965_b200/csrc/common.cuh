// Shared device/host helpers of the sm_100a routed-LoRA kernels.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "molora.h"

namespace molora {

constexpr int kWarp = 32;

__host__ __device__ constexpr int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
__host__ __device__ constexpr int ceil_div(int a, int b) { return (a + b - 1) / b; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- 16-byte vectors of the two storage types -------------------------------------------------
// A Vec<T> is one 128-bit global/shared access: 4 fp32 or 8 bf16 elements.
template <typename T>
struct VecTraits;
template <>
struct VecTraits<float> {
    static constexpr int kElems = 4;
};
template <>
struct VecTraits<__nv_bfloat16> {
    static constexpr int kElems = 8;
};

__device__ __forceinline__ uint4 ldg128(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
// Streaming 128-bit load for data read exactly once (activations): do not keep it in L1.
__device__ __forceinline__ uint4 ldg128_stream(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// Streaming 128-bit load of memory this kernel also writes (y): coherent path, no L1 allocation.
__device__ __forceinline__ uint4 ld128_rw_stream(const void* p)
{
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p)
                 : "memory");
    return v;
}
__device__ __forceinline__ void stg128(void* p, uint4 v) { *reinterpret_cast<uint4*>(p) = v; }
// 256-bit store (sm_100): p is 32-byte aligned
__device__ __forceinline__ void stg256(void* p, uint4 a, uint4 b)
{
    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x),
                 "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
}

// bf16 pair packed in a 32-bit word -> two fp32 (exact: bf16 is the top half of an fp32).
__device__ __forceinline__ float bf16lo_to_f32(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
// two fp32 -> packed bf16 pair, round to nearest even (lo in the low half).
__device__ __forceinline__ uint32_t f32x2_to_bf16x2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Unpack one 16-byte vector into fp32 registers (kElems of them).
template <typename T>
__device__ __forceinline__ void unpack(const uint4& v, float* out);
template <>
__device__ __forceinline__ void unpack<float>(const uint4& v, float* out)
{
    out[0] = __uint_as_float(v.x);
    out[1] = __uint_as_float(v.y);
    out[2] = __uint_as_float(v.z);
    out[3] = __uint_as_float(v.w);
}
template <>
__device__ __forceinline__ void unpack<__nv_bfloat16>(const uint4& v, float* out)
{
    out[0] = bf16lo_to_f32(v.x);
    out[1] = bf16hi_to_f32(v.x);
    out[2] = bf16lo_to_f32(v.y);
    out[3] = bf16hi_to_f32(v.y);
    out[4] = bf16lo_to_f32(v.z);
    out[5] = bf16hi_to_f32(v.z);
    out[6] = bf16lo_to_f32(v.w);
    out[7] = bf16hi_to_f32(v.w);
}
// Pack kElems fp32 registers into one 16-byte vector of T (one RNE rounding for bf16).
template <typename T>
__device__ __forceinline__ uint4 pack(const float* in);
template <>
__device__ __forceinline__ uint4 pack<float>(const float* in)
{
    return make_uint4(__float_as_uint(in[0]), __float_as_uint(in[1]), __float_as_uint(in[2]), __float_as_uint(in[3]));
}
template <>
__device__ __forceinline__ uint4 pack<__nv_bfloat16>(const float* in)
{
    return make_uint4(f32x2_to_bf16x2(in[0], in[1]), f32x2_to_bf16x2(in[2], in[3]), f32x2_to_bf16x2(in[4], in[5]),
                      f32x2_to_bf16x2(in[6], in[7]));
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

// Segment lookup shared by the apply kernels: tile index -> (segment c, first row position, row count).
// Segment c owns positions [offsets[c], offsets[c+1]) of perm; only segments whose size n satisfies
// min_rows <= n < max_rows are cut into tiles of `tile_rows` rows and numbered (this is how a kernel path is
// chosen per segment, on the device, from the histogram).  Returns false when `tile` is past the last tile.
// C <= 256, so a serial scan by every thread is a few hundred cached loads at worst; all threads of a CTA
// get the same answer.
__device__ __forceinline__ bool find_tile(const int32_t* __restrict__ offsets, int C, int tile_rows, int tile,
                                          int min_rows, int max_rows, int& seg, int& row0, int& rows)
{
    int base = 0;
    int prev = __ldg(offsets);
    for (int c = 0; c < C; ++c) {
        const int next = __ldg(offsets + c + 1);
        const int n = next - prev;
        const int tiles = (n >= min_rows && n < max_rows) ? (n + tile_rows - 1) / tile_rows : 0;
        if (tile < base + tiles) {
            seg = c;
            row0 = prev + (tile - base) * tile_rows;
            rows = min(tile_rows, next - row0);
            return true;
        }
        base += tiles;
        prev = next;
    }
    return false;
}

// Same lookup on a copy of offsets[0..C] that already sits in shared memory (one memory round trip for the
// whole table instead of one per segment scanned).
__device__ __forceinline__ bool find_tile_smem(const int32_t* offs, int C, int tile_rows, int tile, int min_rows,
                                               int max_rows, int& seg, int& row0, int& rows)
{
    int base = 0;
    for (int c = 0; c < C; ++c) {
        const int prev = offs[c], next = offs[c + 1];
        const int n = next - prev;
        const int tiles = (n >= min_rows && n < max_rows) ? (n + tile_rows - 1) / tile_rows : 0;
        if (tile < base + tiles) {
            seg = c;
            row0 = prev + (tile - base) * tile_rows;
            rows = min(tile_rows, next - row0);
            return true;
        }
        base += tiles;
    }
    return false;
}

// Lanes that hold the same routed adapter as this lane (the value for unrouted lanes is never used); shared by the grouping kernels.
__device__ __forceinline__ unsigned peers_of(int v, bool routed, int C)
{
    if (C <= 8) {   // a few ballots are cheaper than a match
        unsigned mine = 0;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const unsigned m = __ballot_sync(0xFFFFFFFFu, routed && v == c);
            if (v == c) mine = m;
        }
        return mine;
    }
    return __match_any_sync(0xFFFFFFFFu, routed ? v : -1);
}

// Bisection form of the lookup for kernels that decode many items per CTA.  tile_starts() (one warp, after
// offs[0..C] is in shared memory; eight consecutive segments per lane) fills tstart[c] = number of tiles owned by
// the segments before c, tstart[C] = all tiles; find_tile_bisect() then costs log2(C) shared-memory reads.
__device__ __forceinline__ void tile_starts(const int32_t* offs, int C, int tile_rows, int min_rows, int max_rows,
                                            int32_t* tstart)
{
    const int lane = threadIdx.x & 31;
    int cnt[8], sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = lane * 8 + j;
        const int n = c < C ? offs[c + 1] - offs[c] : 0;
        cnt[j] = (n >= min_rows && n < max_rows) ? (n + tile_rows - 1) / tile_rows : 0;
        sum += cnt[j];
    }
    int incl = sum;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
        if (lane >= off) incl += up;
    }
    int run = incl - sum;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int c = lane * 8 + j;
        if (c <= C) tstart[c] = run;
        run += cnt[j];
    }
    if (lane == 31 && C == MOLORA_MAX_ADAPTERS) tstart[MOLORA_MAX_ADAPTERS] = run;
}
// requires 0 <= tile < tstart[C]
__device__ __forceinline__ void find_tile_bisect(const int32_t* offs, const int32_t* tstart, int C, int tile_rows,
                                                 int tile, int& seg, int& row0, int& rows)
{
    int lo = 0, hi = C;                    // invariant: tstart[lo] <= tile < tstart[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (tstart[mid] <= tile) lo = mid;
        else hi = mid;
    }
    // lo is the last segment whose first tile is <= tile; segments that own no tile share their successor's start
    seg = lo;
    row0 = offs[lo] + (tile - tstart[lo]) * tile_rows;
    rows = min(tile_rows, offs[lo + 1] - row0);
}

// Host launchers implemented in the .cu files (stream already unwrapped).
// adapter == nullptr: vocabulary routing; otherwise the compositional gate (r = adapter[i] * M + m)
molora_status_t launch_route_vocab(const int32_t* ids, int64_t N, const int32_t* breaks, int32_t M,
                                   const int32_t* adapter, int32_t n_adapters, int32_t* r_out, uint32_t* dev_status,
                                   cudaStream_t s, const int32_t* slot_of = nullptr, int32_t n_catalog = 0);
// tcgen05 gate (bf16 activations, C > 4, d a multiple of 64, at least 1024 tokens).
bool gate_umma_eligible(int64_t N, int32_t d, int32_t C);
size_t route_gate_umma_workspace_bytes(int32_t d, int32_t C);
// The routers that run on tensor cores first write a three-term bf16 split of their fp32 weights into the workspace.
// image: 0 = build it, then route (the launches are chained); 1 = build only (molora_route_*_prepare); 2 = route with an
// image built earlier (molora_route_*_prepared: the weights are static in serving, so the preparation launch is saved).
enum ImageMode : int { kImageBuildAndUse = 0, kImageBuildOnly = 1, kImageUseOnly = 2 };
molora_status_t launch_route_gate_umma(const void* x, int64_t N, int32_t d, int64_t ldx, const float* G,
                                       const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                       uint32_t* dev_status, cudaStream_t s, int image = kImageBuildAndUse);
size_t route_gate_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C);
molora_status_t launch_route_gate(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* G,
                                  const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                  uint32_t* dev_status, cudaStream_t s, int image = kImageBuildAndUse);
// workspace of the prepared form: both tensor-core gates' images side by side (which one runs depends on N)
size_t route_gate_prepared_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C);
// Tensor-core (mma.sync) gate for bf16 activations; the CUDA-core kernel above serves fp32 activations.
// Needs route_gate_mma_workspace_bytes(d, C) bytes of scratch for the split gate weights.
size_t route_gate_mma_workspace_bytes(int32_t d, int32_t C);
molora_status_t launch_route_gate_mma(const void* x, int64_t N, int32_t d, int64_t ldx, const float* G,
                                      const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                      cudaStream_t s, int image = kImageBuildAndUse);
// The paper's MLP router (Eq. 9).  The tensor-core path (bf16 x, d a multiple of 64, at least 128 tokens) needs
// route_mlp_workspace_bytes(...) bytes for the split first-layer weights.
size_t route_mlp_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t H);
molora_status_t launch_route_mlp(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* W1,
                                 const float* b1, int32_t H, const float* W2, const float* b2, int32_t C, int32_t* r_out,
                                 float* logits_out, void* ws, size_t ws_bytes, uint32_t* dev_status, cudaStream_t s,
                                 int image = kImageBuildAndUse);
// Top-k selection and softmax over router logits (Eq. 8); idx / w slot-major [k][N].
molora_status_t launch_topk_softmax(const float* logits, int64_t N, int32_t C, int32_t k, int32_t* idx_out, float* w_out,
                                    cudaStream_t s);
// Adapter sets of top-k routing (sorted adapters of a token spelled in base C) and the weights in the same order.
// Adapter sets of top-k routing are numbered densely: the k adapters of a token, sorted (repeats allowed), are the
// topk_set_count(C, k) = binom(C + k - 1, k) multisets in colexicographic order, rank = sum_j binom(a_j + j, j + 1).
__host__ __device__ inline int64_t binom_small(int64_t n64, int r)         // r <= 4, n < 1000: closed forms in 32 bits
{
    const int n = (int)n64;
    if (n < r) return 0;
    switch (r) {
        case 0: return 1;
        case 1: return n;
        case 2: return n * (n - 1) / 2;
        case 3: return n * (n - 1) / 2 * (n - 2) / 3;
        default: return n * (n - 1) / 2 * (n - 2) / 3 * (n - 3) / 4;
    }
}
__host__ __device__ inline int64_t topk_set_count(int C, int k) { return binom_small((int64_t)C + k - 1, k); }
constexpr int kTopkSetTableBytes = MOLORA_MAX_ADAPTERS * 4;               // set -> its (up to four) adapters, one byte each
molora_status_t launch_topk_sets(const int32_t* idx, const float* w, int64_t N, int32_t C, int32_t k, int32_t* set_out,
                                 float* w_out, uint8_t* table_out, cudaStream_t s);
size_t group_workspace_bytes(int64_t N, int32_t C);
molora_status_t launch_group(const int32_t* r, int64_t N, int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm,
                             void* ws, size_t ws_bytes, uint32_t* dev_status, cudaStream_t s);
// CUDA-core path for the segments with fewer than max_rows rows (INT32_MAX: every segment).
molora_status_t launch_apply_rowtile(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N,
                                     int32_t C, const int32_t* offsets, const int32_t* perm, int32_t max_rows,
                                     cudaStream_t s);
// tcgen05 path for the segments with at least min_rows rows (bf16, rank 16/32/64, d_in and d_out multiples of 64).
bool umma_eligible(const molora_proj_desc_t& p, molora_dtype_t dt);
// With r (routing decisions, at most 4096 tokens, one rank, min_rows 1) the kernel groups on chip: offsets / perm /
// counts_out are then OUTPUTS, bit-equal to launch_group's.
bool group_apply_umma_eligible(int64_t N, int32_t C);
molora_status_t launch_apply_umma(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                  const int32_t* offsets, const int32_t* perm, uint32_t* dev_status, int32_t min_rows,
                                  cudaStream_t s, const int32_t* r = nullptr, int32_t* counts_out = nullptr,
                                  int32_t parts = 1, int32_t n_adapters = 0, const uint8_t* set_table = nullptr);
// (parts > 1: top-k routing in one pass -- C counts adapter SETS of `parts` adapters out of `n_adapters`, set_table[4 * set +
// j] names them, the projections carry the stacked rank parts x r and row_scale = the weights [parts][N]; adapters' rank
// 16, 32 or 64)

// mma.sync path for decode-sized calls (bf16, rank 16/32/64, d_in and d_out multiples of 32): a shrink launch and
// an expand launch; takes the segments with fewer than max_rows rows.  The workspace holds the fp32 partial
// shrink results: the sum of decode_workspace_bytes over the projections.
bool decode_eligible(const molora_proj_desc_t& p, molora_dtype_t dt);
// Single-launch streaming kernel for calls below the tcgen05 crossover (bf16, ranks 16 / 32 / 64, no workspace).
molora_status_t launch_apply_stream(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                    const int32_t* offsets, const int32_t* perm, int32_t max_rows, uint32_t* dev_status,
                                    cudaStream_t s);
// The same kernel for top-k routing in one pass: segments are adapter sets (n_sets of them, set_table[4 * set + j] = the
// j-th adapter of the set), the projections carry the stacked rank parts x r and row_scale = weights [parts][N].
bool stream_eligible(const molora_proj_desc_t& p, molora_dtype_t dt);
molora_status_t launch_apply_stream_sets(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t n_sets, int32_t parts,
                                         const uint8_t* set_table, const int32_t* offsets, const int32_t* perm,
                                         uint32_t* dev_status, cudaStream_t s);
molora_status_t launch_group_apply_stream_sets(const int32_t* sets, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                               int32_t n_sets, int32_t parts, const uint8_t* set_table, int32_t* counts,
                                               int32_t* offsets, int32_t* perm, uint32_t* dev_status, cudaStream_t s);
// The same kernel started from the routing decisions r: grouping (counts, offsets, perm as molora_group writes them)
// and apply in one launch; all projections of one rank, at most 4096 tokens.
bool group_apply_stream_eligible(int64_t N);
molora_status_t launch_group_apply_stream(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                          int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm,
                                          uint32_t* dev_status, cudaStream_t s);
// The two-launch kernels started from r: both kernels group on chip, the first also writes counts / offsets / perm;
// one rank, at most 1024 tokens.  Saves the grouping launch.
bool group_apply_decode_eligible(int64_t N);
molora_status_t launch_group_apply_decode(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N,
                                          int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm, void* ws,
                                          size_t ws_bytes, uint32_t* dev_status, cudaStream_t s);
size_t decode_workspace_bytes(int64_t N, int32_t d_in, int32_t rank);
molora_status_t launch_apply_decode(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                    const int32_t* offsets, const int32_t* perm, int32_t max_rows, void* ws,
                                    size_t ws_bytes, uint32_t* dev_status, cudaStream_t s);

// Job-list kernel for decode-sized calls (bf16, one rank per launch, at most 1024 tokens): one cooperative launch whose
// CTAs share chunk-sized shrink and expand jobs; partial shrink results and per-tile counters live in the workspace.
// ctl: jobs_control_bytes() bytes, zero before the first call and left zero by every call; part: the sum of
// jobs_partial_bytes over the projections of the launch.
bool jobs_eligible(const molora_proj_desc_t& p, molora_dtype_t dt, int64_t N);
size_t jobs_control_bytes();
size_t jobs_partial_bytes(int64_t N, int32_t C, int32_t d_in, int32_t rank);
molora_status_t launch_apply_jobs(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C, const int32_t* offsets,
                                  const int32_t* perm, void* ctl, void* part, size_t part_bytes, uint32_t* dev_status,
                                  cudaStream_t s);
molora_status_t launch_group_apply_jobs(const int32_t* r, const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C,
                                        int32_t* counts, int32_t* offsets, int32_t* perm, void* ctl, void* part,
                                        size_t part_bytes, uint32_t* dev_status, cudaStream_t s);

molora_status_t launch_bounded_wait_selftest(uint32_t* dev_status, int64_t limit_cycles, int32_t* result, cudaStream_t s);

// Path selection: a segment goes to the tensor-core kernel when it has at least kUmmaMinRows rows and the call
// has at least kUmmaMinTokens tokens (known on the host); everything else runs on the CUDA-core kernel.
constexpr int32_t kUmmaMinRows = 32;
constexpr int64_t kUmmaMinTokens = 1024;     // below this no projection uses the tensor-core kernel
constexpr int32_t kUmmaAllSegmentsMaxC = 64;   // up to this many adapters the tensor-core kernel takes all segments

// Launch helper: a cluster of cluster_x CTAs along x when cluster_x > 1, and, when under_predecessor is set,
// programmatic stream serialization: the kernel may start while the previous kernel of the stream still runs and
// calls ptx::grid_dependency_wait() before it touches what that kernel writes.  Used only between the two
// launches of one call (weight split -> tcgen05 gate, decode shrink -> expand), where the predecessor is known;
// across calls the kernels run in plain stream order (chaining them was measured: no gain on any workload).
bool chained_launch_enabled();   // false when the "chained_launch_off" override is set (plain stream order everywhere)
// Tuning overrides, for measurements and for tests that target one kernel: process-wide integers, 0 = the library's own
// choice.  Their start values come from the environment (MOLORA_UMMA_MIN_TOKENS, MOLORA_SMALL_PATH=stream|twophase|jobs,
// MOLORA_STREAM_TILE, MOLORA_UMMA_SPLIT, MOLORA_UMMA_TILE_ROWS, MOLORA_GROUP_SPLIT, MOLORA_CHAINED_LAUNCH=0), read ONCE
// when the library is first used; afterwards only molora_debug_set changes them.
enum TuneKey {
    kTuneUmmaMinTokens = 0,   // tcgen05 apply from this many tokens
    kTuneSmallPath,           // kernel below the tcgen05 crossover: 1 streaming, 2 two-launch, 3 job-list decode kernel
    kTuneStreamTile,          // rank-16 streaming tile: 16 or 32 rows
    kTuneUmmaSplit,           // cluster size of the tcgen05 apply
    kTuneUmmaTileRows,        // rows per tile of the tcgen05 apply
    kTuneGroupSplit,          // cluster size of the grouping kernel
    kTuneChainedLaunchOff,    // 1: no programmatic dependent launches
    kTuneJobsLaunch,          // job-list kernel: 0 cooperative launch, 1 plain, 2 programmatic (measurements only)
    kTuneCount
};
int64_t tune(TuneKey key);
void note_launch();               // one more kernel enqueued by this library (molora_launch_count)
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                 unsigned cluster_x, bool under_predecessor, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (under_predecessor && chained_launch_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    note_launch();
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Launch attributes (opt-in shared memory sizes, occupancy-derived wave sizes) belong to a device: the launchers cache
// them in small arrays indexed by the ordinal of the current device.
constexpr int kMaxDevices = 64;
inline int device_slot()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) dev = 0;
    return dev % kMaxDevices;
}

inline int sm_count()
{
    static int sms_dev[kMaxDevices] = {};
    int& sms = sms_dev[device_slot()];
    if (sms == 0) {
        int dev = 0, n = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            return 148;                           // no device visible (host-only callers of the size queries): B200's count
        sms = n;
    }
    return sms;
}

inline molora_status_t cuda_ok(cudaError_t e) { return e == cudaSuccess ? MOLORA_OK : MOLORA_ERR_CUDA; }

}  // namespace molora
