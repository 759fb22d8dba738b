// C ABI: argument validation on the host, then enqueue.  Nothing here touches device memory from the host,
// allocates, or synchronises.
#include "common.cuh"

#include <algorithm>
#include <atomic>
#include <cstdlib>
#include <cstring>
#include <mutex>

using namespace molora;

namespace molora {
namespace {
std::atomic<int64_t> g_tune[kTuneCount];
std::atomic<uint64_t> g_launches{0};
std::once_flag g_tune_once;
const char* const kTuneNames[kTuneCount] = {"umma_min_tokens", "small_path", "stream_tile", "umma_split",
                                            "umma_tile_rows", "group_split", "chained_launch_off", "jobs_launch"};
void tune_from_environment()
{
    auto num = [](const char* name) {
        const char* e = std::getenv(name);
        return e != nullptr && e[0] != '\0' ? (int64_t)std::atoll(e) : (int64_t)0;
    };
    g_tune[kTuneUmmaMinTokens] = std::max<int64_t>(0, num("MOLORA_UMMA_MIN_TOKENS"));
    const char* sp = std::getenv("MOLORA_SMALL_PATH");
    g_tune[kTuneSmallPath] = sp == nullptr ? 0 : sp[0] == 's' ? 1 : sp[0] == 't' ? 2 : sp[0] == 'j' ? 3 : 0;
    g_tune[kTuneStreamTile] = num("MOLORA_STREAM_TILE");
    g_tune[kTuneUmmaSplit] = num("MOLORA_UMMA_SPLIT");
    g_tune[kTuneUmmaTileRows] = num("MOLORA_UMMA_TILE_ROWS");
    g_tune[kTuneGroupSplit] = num("MOLORA_GROUP_SPLIT");
    const char* ch = std::getenv("MOLORA_CHAINED_LAUNCH");
    g_tune[kTuneChainedLaunchOff] = ch != nullptr && std::strcmp(ch, "0") == 0 ? 1 : 0;
    g_tune[kTuneJobsLaunch] = num("MOLORA_JOBS_LAUNCH");
}
}  // namespace
int64_t tune(TuneKey key)
{
    std::call_once(g_tune_once, tune_from_environment);
    return g_tune[key].load(std::memory_order_relaxed);
}
bool chained_launch_enabled() { return tune(kTuneChainedLaunchOff) == 0; }
void note_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
}  // namespace molora

namespace {

// ---- path selection (bf16, ranks 16 / 32 / 64; everything else runs on the CUDA-core row-tile kernel)
// Three kernels cover the bf16 calls: the tcgen05 kernel (128-row tiles, clusters), the single-launch streaming
// kernel (32-row tiles, one CTA per item) and the two-launch small-tile kernels.  Measured on B200 (2048- and
// 4096-wide projections, 4-128 adapters, 1-7 projections per call):
//   rank 16  streaming wins until the projections of the call move ~150 MB (x once, y twice), tcgen05 above;
//   rank 32  streaming until ~60 MB, tcgen05 above (below 1024 tokens the two-launch pair ties for one projection
//            and loses by a third for a layer's worth of them);
//   rank 64  tcgen05 (tiles split over clusters of up to 8 CTAs) once the projections of the call move ~12 MB with at
//            least 256 tokens and segments of 32 rows on average (one 4096-wide projection: from 512 tokens, 21.0 us
//            against 24.3; two: 23.2 against 38.9 at 512 tokens; a layer of seven: 89.7 against 134.9), and from 1280
//            tokens in any case; below, the two-launch pair for one or two projections and the streaming kernel for
//            more (the streaming kernel has only two stages at this rank).
// The overrides "umma_min_tokens" (tcgen05 from n tokens) and "small_path" (the kernel used below it) of
// molora_debug_set force a choice, for measurements and for tests that target one kernel.
int64_t forced_umma_min_tokens() { return std::max<int64_t>(0, tune(kTuneUmmaMinTokens)); }
constexpr double kUmmaMinBytesR16 = 150e6, kUmmaMinBytesR32 = 60e6;
constexpr int64_t kUmmaMinTokensR64 = 1280, kUmmaMinTokensR64Wide = 256;
constexpr double kUmmaMinBytesR64 = 12e6;

double proj_bytes(int64_t N, int32_t d_in, int32_t d_out) { return (double)N * ((double)d_in + 2.0 * d_out) * 2.0; }

// group_bytes: bytes moved by all projections of this rank in the call
// rank 64: group_bytes may be a lower bound (one projection's own bytes when the others are not known)
bool use_umma_r64(int64_t N, int32_t C, double group_bytes)
{
    if (N >= kUmmaMinTokensR64) return true;
    return N >= kUmmaMinTokensR64Wide && N >= (int64_t)C * kUmmaMinRows && group_bytes >= kUmmaMinBytesR64;
}
bool use_umma(int32_t rank, int64_t N, int32_t C, double group_bytes)
{
    if (const int64_t forced = forced_umma_min_tokens()) return N >= forced;
    if (rank == 64) return use_umma_r64(N, C, group_bytes);
    if (N < kUmmaMinTokens) return false;
    if (rank == 16) return group_bytes >= kUmmaMinBytesR16;
    return group_bytes >= kUmmaMinBytesR32;
}
// the kernel for what the tcgen05 kernel does not take; same_rank: projections of this rank in the call (0: unknown)
bool small_path_is_stream(int32_t rank, int64_t N, int same_rank)
{
    if (const int64_t forced = tune(kTuneSmallPath)) {
        if (forced == 1) return true;
        if (forced == 2) return false;
    }
    (void)N;
    // rank 64: the two-launch pair for one or two projections (its split of the reduction over CTAs pays there);
    // with a layer's worth of them its items no longer fit a wave and the streaming kernel is faster
    return rank == 16 || rank == 32 || same_rank > 2;
}

// The job-list kernel shares chunk-sized jobs between all CTAs instead of giving every (tile, projection) pair to one CTA.
// Its jobs cost more than the streaming kernel's chunks (a partial exchange through L2 per shrink chunk), so it only pays
// where the streaming kernel's longest items dominate: measured on B200 (seven 2048 / 6144-wide rank-16 projections,
// 8 adapters, graph replay, us, streaming / job list): 32 tokens 10.4 / 11.7, 128: 12.0 / 13.9, 256: 14.9 / 16.6,
// 512: 26.4 / 21.7, 1024: 36.3 / 34.1; one projection, ranks 32 and 64: the streaming or the two-launch kernels win at
// every size.  Hence: rank 16, at least four projections of that rank in the call, more than 256 and at most 1024 tokens.
bool use_jobs(const molora_proj_desc_t& p, molora_dtype_t dt, int64_t N, int32_t C, int same_rank)
{
    (void)C;
    if (!jobs_eligible(p, dt, N)) return false;
    if (const int64_t forced = tune(kTuneSmallPath)) return forced == 3;
    return p.rank == 16 && same_rank >= 4 && N > 256;
}

bool rank_supported(int r) { return r == 8 || r == 16 || r == 32 || r == 64; }

molora_status_t check_proj(const molora_proj_desc_t& p, molora_dtype_t dt)
{
    if (p.x == nullptr || p.y == nullptr || p.A == nullptr || p.B == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (p.d_in <= 0 || p.d_out <= 0) return MOLORA_ERR_INVALID_ARG;
    if (!rank_supported(p.rank)) return MOLORA_ERR_UNSUPPORTED;
    if ((p.d_in % 8) != 0 || (p.d_out % 8) != 0 || (p.ldx % 8) != 0 || (p.ldy % 8) != 0) return MOLORA_ERR_UNSUPPORTED;
    if (p.ldx < p.d_in || p.ldy < p.d_out) return MOLORA_ERR_INVALID_ARG;
    if (!aligned16(p.x) || !aligned16(p.y) || !aligned16(p.A) || !aligned16(p.B)) return MOLORA_ERR_INVALID_ARG;
    (void)dt;
    return MOLORA_OK;
}

}  // namespace

extern "C" {

const char* molora_version(void) { return "molora-b200 0.2 (sm_100a)"; }

molora_status_t molora_debug_set(const char* name, int64_t value)
{
    if (name == nullptr) return MOLORA_ERR_INVALID_ARG;
    (void)tune(kTuneUmmaMinTokens);                 // the environment is read before the first override
    for (int k = 0; k < kTuneCount; ++k)
        if (std::strcmp(name, kTuneNames[k]) == 0) {
            g_tune[k].store(value, std::memory_order_relaxed);
            return MOLORA_OK;
        }
    return MOLORA_ERR_INVALID_ARG;
}

uint64_t molora_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* molora_status_string(molora_status_t status)
{
    switch (status) {
        case MOLORA_OK: return "ok";
        case MOLORA_ERR_INVALID_ARG: return "invalid argument";
        case MOLORA_ERR_UNSUPPORTED: return "unsupported shape, rank or dtype";
        case MOLORA_ERR_WORKSPACE: return "workspace missing or too small";
        case MOLORA_ERR_CUDA: return "CUDA runtime error";
        case MOLORA_ERR_BUSY: return "every hot-set slot is in use";
        case MOLORA_ERR_NOT_RESIDENT: return "adapter not resident in the hot set";
    }
    return "unknown status";
}

molora_status_t molora_route_vocab(const int32_t* ids, int64_t N, const int32_t* breaks, int32_t M, int32_t* r_out,
                                   uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX) return MOLORA_ERR_INVALID_ARG;
    if (M < 1) return MOLORA_ERR_INVALID_ARG;
    if (M > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (breaks == nullptr || (N > 0 && (ids == nullptr || r_out == nullptr))) return MOLORA_ERR_INVALID_ARG;
    return launch_route_vocab(ids, N, breaks, M, nullptr, 0, r_out, dev_status, static_cast<cudaStream_t>(stream));
}

molora_status_t molora_route_composite(const int32_t* ids, const int32_t* adapter, int64_t N, const int32_t* breaks,
                                       int32_t M, int32_t n_adapters, int32_t* r_out, uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX) return MOLORA_ERR_INVALID_ARG;
    if (M < 1 || n_adapters < 1) return MOLORA_ERR_INVALID_ARG;
    if ((int64_t)M * n_adapters > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (breaks == nullptr || (N > 0 && (ids == nullptr || adapter == nullptr || r_out == nullptr))) return MOLORA_ERR_INVALID_ARG;
    return launch_route_vocab(ids, N, breaks, M, adapter, n_adapters, r_out, dev_status, static_cast<cudaStream_t>(stream));
}

size_t molora_route_gate_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C)
{
    if (d <= 0 || C < 1 || C > 32) return 0;
    return route_gate_workspace_bytes(xdt, d, C);
}

molora_status_t molora_route_gate(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* G,
                                  const float* bias, int32_t C, int32_t* r_out, float* logits_out, void* ws,
                                  size_t ws_bytes, uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX || d <= 0 || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if (C > 32 || (d % 8) != 0 || (ldx % 8) != 0) return MOLORA_ERR_UNSUPPORTED;
    if (ldx < d || G == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && (x == nullptr || r_out == nullptr || !aligned16(x))) return MOLORA_ERR_INVALID_ARG;
    const size_t need = route_gate_workspace_bytes(xdt, d, C);
    if (need > 0 && (ws == nullptr || ws_bytes < need || !aligned16(ws))) return MOLORA_ERR_WORKSPACE;
    return launch_route_gate(x, xdt, N, d, ldx, G, bias, C, r_out, logits_out, ws, dev_status, static_cast<cudaStream_t>(stream));
}

// ---- the same routers with the weight images built once (static router weights)
size_t molora_route_gate_prepared_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C)
{
    if (d <= 0 || C < 1 || C > 32) return 0;
    return route_gate_prepared_workspace_bytes(xdt, d, C);
}

molora_status_t molora_route_gate_prepare(molora_dtype_t xdt, int32_t d, int32_t C, const float* G, void* ws, size_t ws_bytes,
                                          void* stream)
{
    if (d <= 0 || C < 1 || G == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if (C > 32 || (d % 8) != 0) return MOLORA_ERR_UNSUPPORTED;
    const size_t need = route_gate_prepared_workspace_bytes(xdt, d, C);
    if (need > 0 && (ws == nullptr || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) % 256) != 0)) return MOLORA_ERR_WORKSPACE;
    return launch_route_gate(nullptr, xdt, 0, d, 0, G, nullptr, C, nullptr, nullptr, ws, nullptr, static_cast<cudaStream_t>(stream),
                             kImageBuildOnly);
}

molora_status_t molora_route_gate_prepared(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* G,
                                           const float* bias, int32_t C, int32_t* r_out, float* logits_out, const void* ws,
                                           size_t ws_bytes, uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX || d <= 0 || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if (C > 32 || (d % 8) != 0 || (ldx % 8) != 0) return MOLORA_ERR_UNSUPPORTED;
    if (ldx < d || G == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && (x == nullptr || r_out == nullptr || !aligned16(x))) return MOLORA_ERR_INVALID_ARG;
    const size_t need = route_gate_prepared_workspace_bytes(xdt, d, C);
    if (need > 0 && (ws == nullptr || ws_bytes < need || (reinterpret_cast<uintptr_t>(ws) % 256) != 0)) return MOLORA_ERR_WORKSPACE;
    return launch_route_gate(x, xdt, N, d, ldx, G, bias, C, r_out, logits_out, const_cast<void*>(ws), dev_status,
                             static_cast<cudaStream_t>(stream), kImageUseOnly);
}

molora_status_t molora_route_mlp_prepare(molora_dtype_t xdt, int32_t d, int32_t H, int32_t C, const float* W1, void* ws,
                                         size_t ws_bytes, void* stream)
{
    if (d <= 0 || H < 1 || C < 1 || W1 == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if ((d % 8) != 0 || H > 128 || C > 32) return MOLORA_ERR_UNSUPPORTED;
    return launch_route_mlp(nullptr, xdt, 0, d, 0, W1, nullptr, H, nullptr, nullptr, C, nullptr, nullptr, ws, ws_bytes, nullptr,
                            static_cast<cudaStream_t>(stream), kImageBuildOnly);
}

molora_status_t molora_route_mlp_prepared(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* W1,
                                          const float* b1, int32_t H, const float* W2, const float* b2, int32_t C,
                                          int32_t* r_out, float* logits_out, const void* ws, size_t ws_bytes,
                                          uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX || d <= 0 || H < 1 || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if ((d % 8) != 0 || (ldx % 8) != 0 || H > 128 || C > 32) return MOLORA_ERR_UNSUPPORTED;
    if (ldx < d) return MOLORA_ERR_INVALID_ARG;
    if (W1 == nullptr || W2 == nullptr || (N > 0 && (x == nullptr || r_out == nullptr))) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && !aligned16(x)) return MOLORA_ERR_INVALID_ARG;
    return launch_route_mlp(x, xdt, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, const_cast<void*>(ws), ws_bytes, dev_status,
                            static_cast<cudaStream_t>(stream), kImageUseOnly);
}

size_t molora_route_mlp_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t H, int32_t C)
{
    if (d <= 0 || H < 1 || H > 128 || C < 1 || C > 32) return 0;
    return route_mlp_workspace_bytes(xdt, d, H);
}

molora_status_t molora_route_mlp(const void* x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float* W1,
                                 const float* b1, int32_t H, const float* W2, const float* b2, int32_t C, int32_t* r_out,
                                 float* logits_out, void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX || d <= 0 || H < 1 || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (xdt != MOLORA_F32 && xdt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if ((d % 8) != 0 || (ldx % 8) != 0 || H > 128 || C > 32) return MOLORA_ERR_UNSUPPORTED;
    if (ldx < d) return MOLORA_ERR_INVALID_ARG;
    if (W1 == nullptr || W2 == nullptr || (N > 0 && (x == nullptr || r_out == nullptr))) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && !aligned16(x)) return MOLORA_ERR_INVALID_ARG;
    return launch_route_mlp(x, xdt, N, d, ldx, W1, b1, H, W2, b2, C, r_out, logits_out, ws, ws_bytes, dev_status,
                            static_cast<cudaStream_t>(stream));
}

size_t molora_group_workspace_bytes(int64_t N, int32_t C) { return group_workspace_bytes(N, C); }

molora_status_t molora_group(const int32_t* r, int64_t N, int32_t C, int32_t* counts, int32_t* offsets, int32_t* perm,
                             void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream)
{
    if (N < 0 || N >= INT32_MAX || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (C > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (counts == nullptr || offsets == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && (r == nullptr || perm == nullptr)) return MOLORA_ERR_INVALID_ARG;
    const size_t need = group_workspace_bytes(N, C);
    if (need > 0 && (ws == nullptr || ws_bytes < need || !aligned16(ws))) return MOLORA_ERR_WORKSPACE;
    return launch_group(r, N, C, counts, offsets, perm, ws, ws_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

size_t molora_apply_workspace_bytes(int64_t N, int32_t C, int32_t d_in, int32_t d_out, int32_t rank)
{
    // Two kernels need scratch: the job-list kernel (control words + partial shrink results; decode-sized bf16 calls) and
    // the two-launch small-tile kernels (partial shrink results).  Which one runs depends on the other projections of
    // the call, which are not known here, so the figure covers both where both are possible; the element type is not
    // known either, so it assumes bf16 (fp32 calls need none).
    if (N <= 0 || C < 1 || d_in <= 0 || d_out <= 0 || (rank != 16 && rank != 32 && rank != 64)) return 0;
    if ((d_in % 32) != 0 || (d_out % 32) != 0) return 0;
    size_t need = 0;
    molora_proj_desc_t probe{};
    probe.d_in = d_in;
    probe.d_out = d_out;
    probe.rank = rank;
    const int64_t small = tune(kTuneSmallPath);
    // (by default the job-list kernel only takes rank 16 above 256 tokens, see use_jobs)
    if (jobs_eligible(probe, MOLORA_BF16, N) && (small == 3 || (small == 0 && rank == 16 && N > 256)))
        need += jobs_control_bytes() + jobs_partial_bytes(N, C, d_in, rank);
    if (small == 3 && need > 0) return need;
    if (small_path_is_stream(rank, N, 0)) return need;
    // two-launch kernels: needed unless the tcgen05 kernel is certain to take every segment (for ranks 16 and 32 that
    // depends on the other projections of the call, which are not known here)
    const int64_t forced = forced_umma_min_tokens();
    const bool umma_certain = forced > 0 ? N >= forced : (rank == 64 && use_umma_r64(N, C, proj_bytes(N, d_in, d_out)));
    if (umma_certain && C <= kUmmaAllSegmentsMaxC && (d_in % 64) == 0 && (d_out % 64) == 0) return need;
    return need + decode_workspace_bytes(N, d_in, rank);
}

namespace {
// The projections of a batched apply split by kernel.  With more than kUmmaAllSegmentsMaxC adapters the projections of
// the tcgen05 kernel are also handed to a small-tile kernel and each segment is taken by exactly one of the two,
// chosen on the device from its row count.
struct ApplyPlan {
    molora_proj_desc_t tc[MOLORA_MAX_PROJECTIONS], sc[MOLORA_MAX_PROJECTIONS], dc[MOLORA_MAX_PROJECTIONS], cc[MOLORA_MAX_PROJECTIONS];
    molora_proj_desc_t small_sc[MOLORA_MAX_PROJECTIONS], small_dc[MOLORA_MAX_PROJECTIONS], small_cc[MOLORA_MAX_PROJECTIONS];
    molora_proj_desc_t jc[3][MOLORA_MAX_PROJECTIONS];     // job-list kernel, by rank (16, 32, 64)
    int n_tc = 0, n_sc = 0, n_dc = 0, n_cc = 0, n_small_sc = 0, n_small_dc = 0, n_small_cc = 0, n_jc[3] = {0, 0, 0};
    int32_t min_rows = 1;          // segments with at least this many rows go to the tcgen05 kernel
    // workspace layout: [control part of the job-list kernel | its partials, by rank | scratch of the two-launch kernels]
    size_t jobs_ctl = 0, jobs_part_off[3] = {0, 0, 0}, jobs_part[3] = {0, 0, 0}, decode_off = 0;
    size_t ws_need = 0;
};

// Argument checks, kernel split and workspace check of molora_apply_batched: everything that can refuse the call,
// before anything is enqueued.
molora_status_t plan_apply(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
                           const int32_t* offsets, const int32_t* perm, bool tables_given, void* ws, size_t ws_bytes,
                           ApplyPlan& pl)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS) return MOLORA_ERR_INVALID_ARG;
    if (N < 0 || N >= INT32_MAX || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (C > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (dt != MOLORA_F32 && dt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    if (tables_given && (offsets == nullptr || (N > 0 && perm == nullptr))) return MOLORA_ERR_INVALID_ARG;
    for (int i = 0; i < P; ++i) {
        const molora_status_t st = check_proj(projs[i], dt);
        if (st != MOLORA_OK) return st;
    }
    double group_bytes[3] = {0.0, 0.0, 0.0};       // ranks 16, 32, 64
    auto group_of = [](int32_t rank) { return rank == 16 ? 0 : rank == 32 ? 1 : 2; };
    for (int i = 0; i < P; ++i)
        if (umma_eligible(projs[i], dt)) group_bytes[group_of(projs[i].rank)] += proj_bytes(N, projs[i].d_in, projs[i].d_out);
    int same_rank[3] = {0, 0, 0};                  // projections per rank that a small-tile kernel can take
    for (int i = 0; i < P; ++i)
        if (decode_eligible(projs[i], dt)) ++same_rank[group_of(projs[i].rank)];
    for (int i = 0; i < P; ++i) {
        const int32_t rank = projs[i].rank;
        if (umma_eligible(projs[i], dt) && use_umma(rank, N, C, group_bytes[group_of(rank)])) pl.tc[pl.n_tc++] = projs[i];
        else if (use_jobs(projs[i], dt, N, C, same_rank[group_of(rank)])) pl.jc[group_of(rank)][pl.n_jc[group_of(rank)]++] = projs[i];
        else if (decode_eligible(projs[i], dt)) {
            if (small_path_is_stream(rank, N, same_rank[group_of(rank)])) pl.sc[pl.n_sc++] = projs[i];
            else pl.dc[pl.n_dc++] = projs[i];
        } else pl.cc[pl.n_cc++] = projs[i];
    }
    // With few adapters an under-filled 128-row tile is cheap, so the tensor-core kernel takes every segment and the
    // second launch is saved; with many adapters (up to 256 composite targets) tiny segments are the norm and go to a
    // small-tile kernel instead.
    pl.min_rows = C <= kUmmaAllSegmentsMaxC ? 1 : kUmmaMinRows;
    if (pl.n_tc > 0 && pl.min_rows > 1)
        for (int i = 0; i < pl.n_tc; ++i) {
            if (!decode_eligible(pl.tc[i], dt)) pl.small_cc[pl.n_small_cc++] = pl.tc[i];
            else if (small_path_is_stream(pl.tc[i].rank, N, same_rank[group_of(pl.tc[i].rank)])) pl.small_sc[pl.n_small_sc++] = pl.tc[i];
            else pl.small_dc[pl.n_small_dc++] = pl.tc[i];
        }
    size_t need_dc = 0, need_small = 0;
    for (int i = 0; i < pl.n_dc; ++i) need_dc += decode_workspace_bytes(N, pl.dc[i].d_in, pl.dc[i].rank);
    for (int i = 0; i < pl.n_small_dc; ++i) need_small += decode_workspace_bytes(N, pl.small_dc[i].d_in, pl.small_dc[i].rank);
    size_t off = 0;
    if (N > 0 && pl.n_jc[0] + pl.n_jc[1] + pl.n_jc[2] > 0) {
        pl.jobs_ctl = jobs_control_bytes();
        off = pl.jobs_ctl;
        for (int k = 0; k < 3; ++k) {
            pl.jobs_part_off[k] = off;
            for (int i = 0; i < pl.n_jc[k]; ++i) pl.jobs_part[k] += jobs_partial_bytes(N, C, pl.jc[k][i].d_in, pl.jc[k][i].rank);
            off += pl.jobs_part[k];
        }
    }
    pl.decode_off = off;
    pl.ws_need = N > 0 ? off + std::max(need_dc, need_small) : 0;
    if (pl.ws_need > 0 && (ws == nullptr || ws_bytes < pl.ws_need || !aligned16(ws))) return MOLORA_ERR_WORKSPACE;
    return MOLORA_OK;
}

molora_status_t enqueue_apply(const ApplyPlan& pl, molora_dtype_t dt, int64_t N, int32_t C, const int32_t* offsets,
                              const int32_t* perm, void* ws, size_t ws_bytes, uint32_t* dev_status, cudaStream_t s)
{
    molora_status_t st = MOLORA_OK;
    char* base = static_cast<char*>(ws);
    void* dws = ws != nullptr ? base + pl.decode_off : nullptr;              // scratch of the two-launch kernels
    const size_t dws_bytes = ws != nullptr && ws_bytes > pl.decode_off ? ws_bytes - pl.decode_off : 0;
    for (int k = 0; k < 3 && st == MOLORA_OK; ++k)
        if (pl.n_jc[k] > 0)
            st = launch_apply_jobs(pl.jc[k], pl.n_jc[k], N, C, offsets, perm, base, base + pl.jobs_part_off[k], pl.jobs_part[k],
                                   dev_status, s);
    if (st == MOLORA_OK && pl.n_tc > 0) {
        st = launch_apply_umma(pl.tc, pl.n_tc, N, C, offsets, perm, dev_status, pl.min_rows, s);
        if (st == MOLORA_OK && pl.n_small_sc > 0) st = launch_apply_stream(pl.small_sc, pl.n_small_sc, N, C, offsets, perm, pl.min_rows, dev_status, s);
        if (st == MOLORA_OK && pl.n_small_dc > 0) st = launch_apply_decode(pl.small_dc, pl.n_small_dc, N, C, offsets, perm, pl.min_rows, dws, dws_bytes, dev_status, s);
        if (st == MOLORA_OK && pl.n_small_cc > 0) st = launch_apply_rowtile(pl.small_cc, pl.n_small_cc, dt, N, C, offsets, perm, pl.min_rows, s);
    }
    if (st == MOLORA_OK && pl.n_sc > 0) st = launch_apply_stream(pl.sc, pl.n_sc, N, C, offsets, perm, INT32_MAX, dev_status, s);
    if (st == MOLORA_OK && pl.n_dc > 0) st = launch_apply_decode(pl.dc, pl.n_dc, N, C, offsets, perm, INT32_MAX, dws, dws_bytes, dev_status, s);
    if (st == MOLORA_OK && pl.n_cc > 0) st = launch_apply_rowtile(pl.cc, pl.n_cc, dt, N, C, offsets, perm, INT32_MAX, s);
    return st;
}
}  // namespace

molora_status_t molora_apply_batched(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N,
                                     int32_t C, const int32_t* offsets, const int32_t* perm, void* ws, size_t ws_bytes,
                                     uint32_t* dev_status, void* stream)
{
    ApplyPlan pl;
    const molora_status_t st = plan_apply(projs, P, dt, N, C, offsets, perm, true, ws, ws_bytes, pl);
    if (st != MOLORA_OK) return st;
    return enqueue_apply(pl, dt, N, C, offsets, perm, ws, ws_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

// How molora_group_apply_batched runs: 1 = one launch of the streaming kernel (every projection on it, one rank, at
// most 4096 tokens), 3 = one launch of the job-list kernel (every projection on it, one rank), 2 = the two-launch kernels
// with the grouping inside (one rank, at most 1024 tokens), 4 = one launch of the tcgen05 kernel with the grouping inside
// (every projection on it, one rank, at most 4096 tokens, few enough adapters that it takes every segment), 0 = the
// grouping launch followed by the apply launches.
static int group_apply_mode(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C)
{
    if (dt != MOLORA_BF16 || N < 1) return 0;
    double bytes = 0.0;
    bool same = true, stream = true, twophase = true, jobs = true, umma = true;
    for (int i = 0; i < P; ++i) {
        same = same && projs[i].rank == projs[0].rank && decode_eligible(projs[i], dt);
        if (!same) return 0;
        const bool jb = use_jobs(projs[i], dt, N, C, P);
        const bool st = small_path_is_stream(projs[i].rank, N, P);
        jobs = jobs && jb;
        stream = stream && !jb && st;
        twophase = twophase && !jb && !st;
        umma = umma && umma_eligible(projs[i], dt);
        if (umma_eligible(projs[i], dt)) bytes += proj_bytes(N, projs[i].d_in, projs[i].d_out);
    }
    if (use_umma(projs[0].rank, N, C, bytes)) return umma && group_apply_umma_eligible(N, C) ? 4 : 0;
    if (jobs) return 3;
    if (stream && group_apply_stream_eligible(N)) return 1;
    if (twophase && group_apply_decode_eligible(N)) return 2;
    return 0;
}

int32_t molora_group_apply_is_one_launch(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS || N < 1 || C < 1) return 0;
    const int mode = group_apply_mode(projs, P, dt, N, C);
    return mode == 1 || mode == 3 || mode == 4 ? 1 : 0;
}

int32_t molora_group_apply_skips_group_launch(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS || N < 1 || C < 1) return 0;
    return group_apply_mode(projs, P, dt, N, C) != 0 ? 1 : 0;
}

molora_status_t molora_group_apply_batched(const int32_t* r, int64_t N, int32_t C, int32_t* counts, int32_t* offsets,
                                           int32_t* perm, const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt,
                                           void* ws, size_t ws_bytes, uint32_t* dev_status, void* stream)
{
    // argument checks of both halves first: nothing is enqueued if either would refuse
    if (N < 0 || N >= INT32_MAX || C < 1) return MOLORA_ERR_INVALID_ARG;
    if (C > MOLORA_MAX_ADAPTERS) return MOLORA_ERR_UNSUPPORTED;
    if (counts == nullptr || offsets == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && (r == nullptr || perm == nullptr)) return MOLORA_ERR_INVALID_ARG;
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS) return MOLORA_ERR_INVALID_ARG;
    if (dt != MOLORA_F32 && dt != MOLORA_BF16) return MOLORA_ERR_UNSUPPORTED;
    for (int i = 0; i < P; ++i) {
        const molora_status_t st = check_proj(projs[i], dt);
        if (st != MOLORA_OK) return st;
    }
    // When every projection of the call runs on the streaming kernel (or on the two-launch kernels) with one rank, the
    // CTAs of those kernels do the grouping themselves.  Otherwise the two calls, in stream order.  Whatever could
    // refuse the call (the workspace of the two-launch kernels included) is checked before the first launch.
    const int mode = group_apply_mode(projs, P, dt, N, C);
    if (mode == 1)
        return launch_group_apply_stream(r, projs, P, N, C, counts, offsets, perm, dev_status, static_cast<cudaStream_t>(stream));
    if (mode == 4)
        return launch_apply_umma(projs, P, N, C, offsets, perm, dev_status, 1, static_cast<cudaStream_t>(stream), r, counts);
    if (mode == 3) {
        size_t part = 0;
        for (int i = 0; i < P; ++i) part += jobs_partial_bytes(N, C, projs[i].d_in, projs[i].rank);
        const size_t ctl = jobs_control_bytes();
        if (ws == nullptr || ws_bytes < ctl + part || !aligned16(ws)) return MOLORA_ERR_WORKSPACE;
        return launch_group_apply_jobs(r, projs, P, N, C, counts, offsets, perm, ws, static_cast<char*>(ws) + ctl, part, dev_status,
                                       static_cast<cudaStream_t>(stream));
    }
    if (mode == 2) {
        size_t need = 0;
        for (int i = 0; i < P; ++i) need += decode_workspace_bytes(N, projs[i].d_in, projs[i].rank);
        if (need > 0 && (ws == nullptr || ws_bytes < need || !aligned16(ws))) return MOLORA_ERR_WORKSPACE;
        return launch_group_apply_decode(r, projs, P, N, C, counts, offsets, perm, ws, ws_bytes, dev_status,
                                         static_cast<cudaStream_t>(stream));
    }
    ApplyPlan pl;
    molora_status_t st = plan_apply(projs, P, dt, N, C, offsets, perm, false, ws, ws_bytes, pl);
    if (st != MOLORA_OK) return st;
    st = molora_group(r, N, C, counts, offsets, perm, nullptr, 0, dev_status, stream);
    if (st != MOLORA_OK) return st;
    return enqueue_apply(pl, dt, N, C, offsets, perm, ws, ws_bytes, dev_status, static_cast<cudaStream_t>(stream));
}

molora_status_t molora_apply(const void* x, int64_t ldx, void* y, int64_t ldy, molora_dtype_t dt, int64_t N,
                             int32_t d_in, int32_t d_out, int32_t rank, const void* A, const void* B, int32_t C,
                             const int32_t* offsets, const int32_t* perm, float scale, void* ws, size_t ws_bytes,
                             uint32_t* dev_status, void* stream)
{
    molora_proj_desc_t p;
    p.x = x;
    p.ldx = ldx;
    p.y = y;
    p.ldy = ldy;
    p.A = A;
    p.B = B;
    p.d_in = d_in;
    p.d_out = d_out;
    p.rank = rank;
    p.scale = scale;
    p.row_scale = nullptr;
    return molora_apply_batched(&p, 1, dt, N, C, offsets, perm, ws, ws_bytes, dev_status, stream);
}

molora_status_t molora_topk_softmax(const float* logits, int64_t N, int32_t C, int32_t k, int32_t* idx_out, float* w_out,
                                    void* stream)
{
    if (N < 0 || N >= INT32_MAX || C < 1 || k < 1 || k > C) return MOLORA_ERR_INVALID_ARG;
    if (C > 32) return MOLORA_ERR_UNSUPPORTED;
    if (N > 0 && (logits == nullptr || idx_out == nullptr || w_out == nullptr)) return MOLORA_ERR_INVALID_ARG;
    return launch_topk_softmax(logits, N, C, k, idx_out, w_out, static_cast<cudaStream_t>(stream));
}

namespace {
struct TopkPlan {
    size_t counts, offsets, perm, sets, wsorted, table, apply_ws, apply_ws_bytes, total;
};
constexpr int kTopkMaxParts = 4;
TopkPlan plan_topk(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C)
{
    auto a256 = [](size_t v) { return (v + 255) & ~(size_t)255; };
    TopkPlan pl;
    // the apply workspace comes first: its control words stay at the same place (and zero) whatever N and C are
    pl.apply_ws = 0;
    pl.apply_ws_bytes = 0;
    for (int i = 0; i < P; ++i)
        pl.apply_ws_bytes += molora_apply_workspace_bytes(N, C, projs[i].d_in, projs[i].d_out, projs[i].rank);
    size_t off = a256(pl.apply_ws_bytes);
    // grouping outputs sized for adapter SETS as well (the single-pass path groups by set: up to 256 of them)
    const size_t n1 = (size_t)(N > 0 ? N : 1);
    pl.counts = off;   off = a256(off + sizeof(int32_t) * (size_t)MOLORA_MAX_ADAPTERS);
    pl.offsets = off;  off = a256(off + sizeof(int32_t) * (size_t)(MOLORA_MAX_ADAPTERS + 1));
    pl.perm = off;     off = a256(off + sizeof(int32_t) * n1);
    pl.sets = off;     off = a256(off + sizeof(int32_t) * n1);
    pl.wsorted = off;  off = a256(off + sizeof(float) * n1 * kTopkMaxParts);
    pl.table = off;    off = a256(off + kTopkSetTableBytes);         // adapter set -> its adapters
    pl.total = off;
    return pl;
}

// Eq. 8 in ONE pass over x and y: tokens are grouped by their SET of kept adapters, a segment's shrink runs against the
// stacked A of its k adapters (rank k x r), the k slices of t are weighted per token, and one expand against the stacked
// B adds all k deltas before the single rounding.  Taken when every projection can run on the streaming kernel with the
// stacked rank (bf16, r x k in {16, 32, 64}, k in {2, 4}, at most 256 adapter sets = multisets of k out of C adapters:
// binom(C + k - 1, k)) and the call is not one the tcgen05 kernel would take pass by pass.
// Returns 0: k passes; 1: one pass on the streaming kernel; 2: one pass on the tcgen05 kernel (adapters of rank >= 16, at
// most 64 adapter sets, widths that are multiples of 64, and a call large enough for that kernel at the stacked rank).
int topk_single_pass(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C, int32_t k)
{
    if (dt != MOLORA_BF16 || (k != 2 && k != 4) || N < 1) return 0;
    const int64_t sets = topk_set_count(C, k);
    if (sets > MOLORA_MAX_ADAPTERS) return 0;
    double bytes = 0.0;
    bool umma_ok = sets <= kUmmaAllSegmentsMaxC && projs[0].rank >= 16;
    for (int i = 0; i < P; ++i) {
        const int stacked = projs[i].rank * k;
        if (!stream_eligible(projs[i], dt) || (stacked != 16 && stacked != 32 && stacked != 64)) return 0;
        if (projs[i].rank != projs[0].rank) return 0;
        umma_ok = umma_ok && umma_eligible(projs[i], dt);
        bytes += proj_bytes(N, projs[i].d_in, projs[i].d_out);
    }
    // (with many sets every 128-row tile is a partial one: 64 sets at 8192 tokens lost to two passes, 113 against 106 us)
    if (umma_ok && (sets <= 16 || N >= sets * 256) && use_umma(projs[0].rank * k, N, (int32_t)sets, bytes)) return 2;
    const int64_t small = tune(kTuneSmallPath);
    if (small != 0 && small != 1) return 0;                         // a test or a measurement asks for another kernel
    return use_umma(projs[0].rank, N, C, bytes) ? 0 : 1;
}
}  // namespace

size_t molora_apply_topk_workspace_bytes(const molora_proj_desc_t* projs, int32_t P, int64_t N, int32_t C)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS || N < 0 || C < 1) return 0;
    return plan_topk(projs, P, N, C).total;
}

molora_status_t molora_apply_topk(const molora_proj_desc_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
                                  int32_t k, const int32_t* idx, const float* w, void* ws, size_t ws_bytes,
                                  uint32_t* dev_status, void* stream)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS || N < 0 || C < 1 || k < 1 || k > C) return MOLORA_ERR_INVALID_ARG;
    if (N > 0 && (idx == nullptr || w == nullptr)) return MOLORA_ERR_INVALID_ARG;
    const TopkPlan pl = plan_topk(projs, P, N, C);
    if (ws == nullptr || ws_bytes < pl.total || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return MOLORA_ERR_WORKSPACE;
    char* base = static_cast<char*>(ws);
    int32_t* counts = reinterpret_cast<int32_t*>(base + pl.counts);
    int32_t* offsets = reinterpret_cast<int32_t*>(base + pl.offsets);
    int32_t* perm = reinterpret_cast<int32_t*>(base + pl.perm);
    molora_proj_desc_t pass[MOLORA_MAX_PROJECTIONS];
    if (const int one_pass = topk_single_pass(projs, P, dt, N, C, k)) {
        for (int i = 0; i < P; ++i) {
            const molora_status_t st = check_proj(projs[i], dt);
            if (st != MOLORA_OK) return st;
        }
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        int32_t* sets = reinterpret_cast<int32_t*>(base + pl.sets);
        float* wsorted = reinterpret_cast<float*>(base + pl.wsorted);
        const int32_t n_sets = (int32_t)topk_set_count(C, k);
        uint8_t* table = reinterpret_cast<uint8_t*>(base + pl.table);
        for (int i = 0; i < P; ++i) {
            pass[i] = projs[i];
            pass[i].rank = projs[i].rank * k;       // the stacked rank of a set
            pass[i].row_scale = wsorted;            // [k][N], in the order of the set's adapters
        }
        molora_status_t st = launch_topk_sets(idx, w, N, C, k, sets, wsorted, table, s);
        if (st != MOLORA_OK) return st;
        if (one_pass == 2) {                         // tcgen05 kernel: one MMA per part in the shrink, stacked B in the expand
            if (group_apply_umma_eligible(N, n_sets))
                return launch_apply_umma(pass, P, N, n_sets, offsets, perm, dev_status, 1, s, sets, counts, k, C, table);
            st = molora_group(sets, N, n_sets, counts, offsets, perm, nullptr, 0, dev_status, stream);
            if (st != MOLORA_OK) return st;
            return launch_apply_umma(pass, P, N, n_sets, offsets, perm, dev_status, 1, s, nullptr, nullptr, k, C, table);
        }
        if (group_apply_stream_eligible(N))         // the CTAs of the apply group the sets themselves
            return launch_group_apply_stream_sets(sets, pass, P, N, n_sets, k, table, counts, offsets, perm, dev_status, s);
        st = molora_group(sets, N, n_sets, counts, offsets, perm, nullptr, 0, dev_status, stream);
        if (st != MOLORA_OK) return st;
        return launch_apply_stream_sets(pass, P, N, n_sets, k, table, offsets, perm, dev_status, s);
    }
    for (int32_t j = 0; j < k; ++j) {               // one (group, apply) pass per kept adapter slot
        for (int i = 0; i < P; ++i) {
            pass[i] = projs[i];
            pass[i].row_scale = w + (int64_t)j * N;
        }
        const molora_status_t st = molora_group_apply_batched(idx + (int64_t)j * N, N, C, counts, offsets, perm, pass, P, dt,
                                                              pl.apply_ws_bytes > 0 ? base + pl.apply_ws : nullptr,
                                                              pl.apply_ws_bytes, dev_status, stream);
        if (st != MOLORA_OK) return st;
    }
    return MOLORA_OK;
}

molora_status_t molora_selftest_bounded_wait(uint32_t* dev_status, int64_t limit_cycles, int32_t* result, void* stream)
{
    if (dev_status == nullptr || result == nullptr || limit_cycles < 1 || limit_cycles > 2000000000LL)
        return MOLORA_ERR_INVALID_ARG;
    return launch_bounded_wait_selftest(dev_status, limit_cycles, result, static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------------- host-buffer path
namespace {

struct HostPlan {          // byte offsets into the arena
    size_t ids, r, counts, offsets, perm, gate_ws, apply_ws, apply_ws_bytes, x[MOLORA_MAX_PROJECTIONS], y[MOLORA_MAX_PROJECTIONS], total;
    int x_owner[MOLORA_MAX_PROJECTIONS];   // first projection with the same x_host (its staged copy is shared)
};

size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }

bool plan_host(const molora_host_proj_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
               molora_router_t router, int32_t gate_proj, HostPlan& pl)
{
    if (projs == nullptr || P < 1 || P > MOLORA_MAX_PROJECTIONS || N < 0 || C < 1 || C > MOLORA_MAX_ADAPTERS) return false;
    if (dt != MOLORA_F32 && dt != MOLORA_BF16) return false;
    const size_t e = dt == MOLORA_BF16 ? 2 : 4;
    // the apply workspace comes first: its control words stay at the same place (and zero) whatever the shapes are
    pl.apply_ws = 0;
    pl.apply_ws_bytes = 0;
    for (int i = 0; i < P; ++i)
        pl.apply_ws_bytes += molora_apply_workspace_bytes(N, C, projs[i].d_in, projs[i].d_out, projs[i].rank);
    size_t off = align256(pl.apply_ws_bytes);
    pl.ids = off;      off = align256(off + sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
    pl.r = off;        off = align256(off + sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
    pl.counts = off;   off = align256(off + sizeof(int32_t) * (size_t)C);
    pl.offsets = off;  off = align256(off + sizeof(int32_t) * (size_t)(C + 1));
    pl.perm = off;     off = align256(off + sizeof(int32_t) * (size_t)(N > 0 ? N : 1));
    pl.gate_ws = off;
    if (router == MOLORA_ROUTE_GATE) {
        if (gate_proj < 0 || gate_proj >= P) return false;
        off = align256(off + route_gate_workspace_bytes(dt, projs[gate_proj].d_in, C));
    }
    for (int i = 0; i < P; ++i) {
        pl.x_owner[i] = i;
        for (int j = 0; j < i; ++j)
            if (projs[j].x_host == projs[i].x_host && projs[j].d_in == projs[i].d_in) { pl.x_owner[i] = j; break; }
        if (pl.x_owner[i] == i) {
            pl.x[i] = off;
            off = align256(off + e * (size_t)N * (size_t)projs[i].d_in);
        } else {
            pl.x[i] = pl.x[pl.x_owner[i]];
        }
        pl.y[i] = off;
        off = align256(off + e * (size_t)N * (size_t)projs[i].d_out);
    }
    pl.total = off;
    return true;
}

}  // namespace

size_t molora_forward_host_arena_bytes(const molora_host_proj_t* projs, int32_t P, molora_dtype_t dt, int64_t N,
                                       int32_t C, molora_router_t router, int32_t gate_proj)
{
    HostPlan pl;
    return plan_host(projs, P, dt, N, C, router, gate_proj, pl) ? pl.total : 0;
}

molora_status_t molora_forward_host(molora_router_t router, const int32_t* route_src_host, const int32_t* breaks_dev,
                                    int32_t M, const float* G_dev, const float* bias_dev, int32_t gate_proj,
                                    const molora_host_proj_t* projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
                                    void* arena, size_t arena_bytes, uint32_t* dev_status, void* stream)
{
    HostPlan pl;
    if (N >= INT32_MAX || !plan_host(projs, P, dt, N, C, router, gate_proj, pl)) return MOLORA_ERR_INVALID_ARG;
    if (router != MOLORA_ROUTE_VOCAB && router != MOLORA_ROUTE_GATE && router != MOLORA_ROUTE_GIVEN)
        return MOLORA_ERR_INVALID_ARG;
    if (router != MOLORA_ROUTE_GATE && N > 0 && route_src_host == nullptr) return MOLORA_ERR_INVALID_ARG;
    if (router == MOLORA_ROUTE_VOCAB && (breaks_dev == nullptr || M < 1 || M > MOLORA_MAX_ADAPTERS)) return MOLORA_ERR_INVALID_ARG;
    if (router == MOLORA_ROUTE_GATE && (G_dev == nullptr || C > 32)) return G_dev == nullptr ? MOLORA_ERR_INVALID_ARG : MOLORA_ERR_UNSUPPORTED;
    if (arena == nullptr || arena_bytes < pl.total || (reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return MOLORA_ERR_WORKSPACE;
    char* base = static_cast<char*>(arena);
    molora_proj_desc_t dev[MOLORA_MAX_PROJECTIONS];
    for (int i = 0; i < P; ++i) {
        if (projs[i].x_host == nullptr || projs[i].y_host == nullptr) return MOLORA_ERR_INVALID_ARG;
        dev[i].x = base + pl.x[i];
        dev[i].ldx = projs[i].d_in;
        dev[i].y = base + pl.y[i];
        dev[i].ldy = projs[i].d_out;
        dev[i].A = projs[i].A;
        dev[i].B = projs[i].B;
        dev[i].d_in = projs[i].d_in;
        dev[i].d_out = projs[i].d_out;
        dev[i].rank = projs[i].rank;
        dev[i].scale = projs[i].scale;
        dev[i].row_scale = nullptr;
        const molora_status_t st = check_proj(dev[i], dt);
        if (st != MOLORA_OK) return st;
    }
    if (N == 0) return MOLORA_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t e = dt == MOLORA_BF16 ? 2 : 4;
    int32_t* r = reinterpret_cast<int32_t*>(base + pl.r);
    int32_t* ids = reinterpret_cast<int32_t*>(base + pl.ids);
    // 1. activations and routing source: host -> device
    if (router != MOLORA_ROUTE_GATE &&
        cudaMemcpyAsync(router == MOLORA_ROUTE_VOCAB ? ids : r, route_src_host, sizeof(int32_t) * (size_t)N,
                        cudaMemcpyHostToDevice, s) != cudaSuccess)
        return MOLORA_ERR_CUDA;
    for (int i = 0; i < P; ++i) {
        if (pl.x_owner[i] == i &&
            cudaMemcpyAsync(base + pl.x[i], projs[i].x_host, e * (size_t)N * projs[i].d_in, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return MOLORA_ERR_CUDA;
        if (cudaMemcpyAsync(base + pl.y[i], projs[i].y_host, e * (size_t)N * projs[i].d_out, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return MOLORA_ERR_CUDA;
    }
    // 2. route
    molora_status_t st = MOLORA_OK;
    if (router == MOLORA_ROUTE_VOCAB) {
        st = launch_route_vocab(ids, N, breaks_dev, M, nullptr, 0, r, dev_status, s);
    } else if (router == MOLORA_ROUTE_GATE) {
        const molora_proj_desc_t& gp = dev[gate_proj];
        if ((gp.d_in % 8) != 0) return MOLORA_ERR_UNSUPPORTED;
        st = launch_route_gate(gp.x, dt, N, gp.d_in, gp.ldx, G_dev, bias_dev, C, r, nullptr, base + pl.gate_ws, dev_status, s);
    }
    if (st != MOLORA_OK) return st;
    // 3. group, 4. apply
    int32_t* offsets = reinterpret_cast<int32_t*>(base + pl.offsets);
    int32_t* perm = reinterpret_cast<int32_t*>(base + pl.perm);
    st = molora_group_apply_batched(r, N, C, reinterpret_cast<int32_t*>(base + pl.counts), offsets, perm, dev, P, dt,
                                    pl.apply_ws_bytes > 0 ? base + pl.apply_ws : nullptr, pl.apply_ws_bytes, dev_status,
                                    stream);
    if (st != MOLORA_OK) return st;
    // 5. results: device -> host
    for (int i = 0; i < P; ++i)
        if (cudaMemcpyAsync(projs[i].y_host, base + pl.y[i], e * (size_t)N * projs[i].d_out, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return MOLORA_ERR_CUDA;
    return MOLORA_OK;
}

}  // extern "C"
