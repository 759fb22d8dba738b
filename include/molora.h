/*
 * molora.h -- C ABI of the B200 (sm_100a) routed-LoRA library.
 *
 * The library computes per-token routed LoRA (Eq. 2 of the MoLoRA paper)
 *
 *        h_i = x_i W + x_i A_{r(i)} B_{r(i)},      r : [N] -> [C]
 *
 * on a caller-provided base projection y = x W, in three steps that mirror the paper's dispatch
 * pipeline (Section 3.3, Figure 2 right, Algorithms 1 and 2):
 *
 *   molora_route_*   the router r (vocabulary ranges, Definition 3.1; or a linear gate with top-1
 *                    argmax, Eq. 8 with k = 1 and the gate of Theorem 3.4 / Table 10)
 *   molora_group     histogram of r, exclusive scan into segment offsets, stable permutation
 *   molora_apply     grouped shrink t_i = x_i A_c and expand h_i = y_i + scale * t_i B_c, in place in y
 *
 * Conventions (all entry points unless stated otherwise)
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, valid on the current device, and
 *     must stay valid until the work enqueued on `stream` has completed.  The library allocates no
 *     memory, never synchronises the host and never reads device memory from the host: each call only
 *     validates its scalar arguments and enqueues kernels on `stream`, so calls may be captured into a
 *     CUDA graph.  The only process-wide state is per-device launch attributes cached on first use, a
 *     counter of enqueued launches (molora_launch_count) and the debug overrides of molora_debug_set.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Matrices are row-major; `ld*` is the row pitch in ELEMENTS.
 *   - Return value: MOLORA_OK, or an error code detected on the host BEFORE anything is enqueued
 *     (the call is then a no-op).  Conditions that can only be seen on the device (ids outside every
 *     vocabulary range, routing values outside [-1, C)) never fault: the offending token is treated as
 *     unrouted and the event is recorded in the optional device status word (see MOLORA_DEV_*).
 *   - Routing value -1 means "unrouted": the token belongs to no segment and keeps h_i = y_i.
 *
 * Supported set: N in [0, 2^31 - 1), 1 <= C <= 256 (Example 3.3's 64 x 4 composite targets),
 * rank in {8, 16, 32, 64}, element type fp32 or bf16 (x, y, A, B share it; accumulation is fp32),
 * d_in / d_out / ld multiples of 8 elements and all tensor base pointers 16-byte aligned.
 */
#ifndef MOLORA_H_
#define MOLORA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MOLORA_OK = 0,
    MOLORA_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer, pitch too small      */
    MOLORA_ERR_UNSUPPORTED = 2, /* rank / dtype / C / dimension outside the supported set                */
    MOLORA_ERR_WORKSPACE = 3,   /* workspace missing or smaller than molora_*_workspace_bytes reports     */
    MOLORA_ERR_CUDA = 4,        /* the CUDA runtime refused a launch or a copy (cudaGetLastError for why)  */
    MOLORA_ERR_BUSY = 5,        /* hot-set: every slot is pinned or being filled; try again later          */
    MOLORA_ERR_NOT_RESIDENT = 6 /* hot-set: the adapter is not (yet) in a slot                             */
} molora_status_t;

typedef enum { MOLORA_F32 = 0, MOLORA_BF16 = 1 } molora_dtype_t;

/* Bits OR-ed by kernels into the optional device status word (uint32, zeroed by the caller). */
#define MOLORA_DEV_ID_OUT_OF_RANGE 0x1u /* some token id lies in no vocabulary range: routed to -1          */
#define MOLORA_DEV_BAD_ROUTE 0x2u       /* some routing value lies outside [-1, C): treated as unrouted       */
#define MOLORA_DEV_TIMEOUT 0x4u         /* a bounded device-side wait gave up (results of that call invalid)   */

#define MOLORA_MAX_ADAPTERS 256
#define MOLORA_MAX_PROJECTIONS 8

/* Library version string, e.g. "molora-b200 0.1 (sm_100a)".  Static storage. */
const char *molora_version(void);

/* Human-readable name of a status code.  Static storage. */
const char *molora_status_string(molora_status_t status);

/* Diagnostics (the paper has no counterpart).
 * molora_launch_count: kernels this library has enqueued in this process so far (all threads, all devices); callers
 *   that report launch counts take the difference around a call.
 * molora_debug_set: overrides one of the library's own choices, for measurements and for tests that target one
 *   kernel; value 0 restores the default.  Names: "umma_min_tokens" (tcgen05 apply from that many tokens),
 *   "small_path" (kernel below it: 1 streaming, 2 two-launch, 3 job-list decode kernel), "stream_tile" (16 | 32),
 *   "umma_split", "umma_tile_rows", "group_split" (cluster sizes / tile height), "chained_launch_off" (1: plain stream
 *   order), "jobs_launch" (job-list kernel: 0 cooperative, 1 plain, 2 programmatic launch).  The start values are read once from the environment variables MOLORA_<NAME>.  Unknown name:
 *   MOLORA_ERR_INVALID_ARG.  Not meant to be changed while calls are in flight on other threads. */
uint64_t molora_launch_count(void);
molora_status_t molora_debug_set(const char *name, int64_t value);

/* ---------------------------------------------------------------------------------------------
 * Router 1: vocabulary routing (Definition 3.1 / Eq. 3; Algorithm 1 "FindModality"), 0-based:
 *     r_out[i] = m   with   breaks[m] <= ids[i] < breaks[m+1],  m in [0, M);   -1 if no range holds ids[i].
 * ids      device int32[N]   token vocabulary indices
 * breaks   device int32[M+1] non-decreasing range boundaries b_0..b_M (an empty range is legal), 1 <= M <= 256
 * r_out    device int32[N]   routing decision per token
 * dev_status  device uint32 or NULL; MOLORA_DEV_ID_OUT_OF_RANGE is OR-ed in if any id is unrouted
 * Integer work, exact.  N == 0 is a no-op. */
molora_status_t molora_route_vocab(const int32_t *ids, int64_t N, const int32_t *breaks, int32_t M, int32_t *r_out,
                                   uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Router 1b: compositional routing (Definition 3.2; Algorithm 1 "Compositional Gating Kernel", lines 4-6): the
 * modality of a token comes from its vocabulary index as above, its adapter from the request metadata, and the
 * composite target indexes a weight stack of shape (n_adapters, M, d, r):
 *     r_out[i] = adapter[i] * M + m(ids[i]);   -1 if ids[i] lies in no range or adapter[i] is outside [0, n_adapters).
 * adapter  device int32[N]   adapter index of every token (constant inside a request); M * n_adapters <= 256
 * The result feeds molora_group / molora_apply with C = n_adapters * M (Example 3.3: 64 x 4 = 256 targets).
 * dev_status  MOLORA_DEV_ID_OUT_OF_RANGE is OR-ed in if any token is left unrouted.  Integer work, exact. */
molora_status_t molora_route_composite(const int32_t *ids, const int32_t *adapter, int64_t N, const int32_t *breaks,
                                       int32_t M, int32_t n_adapters, int32_t *r_out, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Router 2: learned linear gate with top-1 selection (Eq. 8 with k = 1; gate form softmax(W x + b) of
 * Theorem 3.4 / Table 10).  Softmax is monotone and the weight of a single kept logit is 1, so
 *     z[i][c] = sum_k x[i][k] * G[k][c] (+ bias[c]),    r_out[i] = argmax_c z[i][c]  (lowest c on ties).
 * x        device [N, d] of type xdt, row pitch ldx >= d elements; d a multiple of 8; never written
 * G        device fp32 [d, C] row-major (gate weights);  bias  device fp32 [C] or NULL;  1 <= C <= 32
 * r_out    device int32[N]
 * logits_out  device fp32 [N, C] or NULL (the logits as the kernel accumulated them, fp32)
 * ws, ws_bytes  device scratch of at least molora_route_gate_workspace_bytes(xdt, d, C) bytes, 16-byte aligned
 *               (NULL when that is 0).  For bf16 x and C > 4 the kernel runs on the tensor cores (tcgen05 when N >= 1024
 *               and d is a multiple of 64, mma.sync otherwise) and keeps there a three-term bf16 split of G
 *               (hi + mid + lo = 24 mantissa bits), rebuilt on every call.
 * dev_status  device status word or NULL.  Only the tcgen05 kernel waits on the device (bounded): if a wait runs out,
 *             MOLORA_DEV_TIMEOUT is OR-ed in and the tokens of that 128-token tile get r_out = -1 (unrouted).
 * Products are exact in fp32 for bf16 x; accumulation is fp32 in a fixed, token-independent order. */
size_t molora_route_gate_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C);
molora_status_t molora_route_gate(const void *x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float *G,
                                  const float *bias, int32_t C, int32_t *r_out, float *logits_out, void *ws,
                                  size_t ws_bytes, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Router 3: the paper's learned router (Eq. 9), a 2-layer MLP with GELU, followed by top-1 selection:
 *     g(x_i) = W2 GELU(W1 x_i + b1) + b2,    r_out[i] = argmax_c g(x_i)[c]  (lowest c on ties)
 * with the exact GELU(t) = t (1 + erf(t / sqrt 2)) / 2.
 * x        device [N, d] of type xdt, row pitch ldx >= d elements; d a multiple of 8; never written
 * W1       device fp32 [d, H] row-major (input-major);  b1  device fp32 [H] or NULL;  1 <= H <= 128 (the paper: 64, 128)
 * W2       device fp32 [H, C] row-major;                b2  device fp32 [C] or NULL;  1 <= C <= 32
 * r_out    device int32[N];  logits_out  device fp32 [N, C] or NULL
 * ws, ws_bytes  device scratch of at least molora_route_mlp_workspace_bytes(xdt, d, H, C) bytes, 16-byte aligned (NULL
 *               when that is 0): for bf16 x and d a multiple of 64 the first layer runs on the tensor cores with a
 *               three-term bf16 split of W1 kept there (rebuilt on every call); MOLORA_ERR_WORKSPACE if it is
 *               needed (at least 128 tokens) and missing.
 * dev_status  device status word or NULL; as for molora_route_gate (the tensor-core kernel's waits are bounded:
 *             MOLORA_DEV_TIMEOUT, and r_out = -1 for the tokens of the tile whose wait ran out).
 * Products of the first layer are exact in fp32 for bf16 x; accumulation, GELU and the second layer are fp32. */
size_t molora_route_mlp_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t H, int32_t C);
molora_status_t molora_route_mlp(const void *x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx, const float *W1,
                                 const float *b1, int32_t H, const float *W2, const float *b2, int32_t C, int32_t *r_out,
                                 float *logits_out, void *ws, size_t ws_bytes, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The same two routers with the weight images built ONCE.  Router weights are static while a model is served; the
 * tensor-core routers (bf16 x; the gate with C > 4, the MLP with d a multiple of 64) spend a preparation launch per call on
 * the three-term split of G / W1.  molora_route_*_prepare runs that launch alone and leaves the images in `ws`;
 * molora_route_*_prepared routes with them: same arguments, results and errors as molora_route_gate / molora_route_mlp,
 * bit-identical decisions and logits, one launch fewer.  The caller keeps `ws` unchanged between the two and calls
 * prepare again (on the same stream, or otherwise ordered) whenever G / W1 change; the library cannot tell.
 *   gate: ws of at least molora_route_gate_prepared_workspace_bytes(xdt, d, C) bytes, 256-byte aligned (it holds the
 *         images of both tensor-core gates, since the token count decides which one runs; 0: nothing to prepare)
 *   MLP:  ws as for molora_route_mlp (molora_route_mlp_workspace_bytes), 16-byte aligned */
size_t molora_route_gate_prepared_workspace_bytes(molora_dtype_t xdt, int32_t d, int32_t C);
molora_status_t molora_route_gate_prepare(molora_dtype_t xdt, int32_t d, int32_t C, const float *G, void *ws,
                                          size_t ws_bytes, void *stream);
molora_status_t molora_route_gate_prepared(const void *x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx,
                                           const float *G, const float *bias, int32_t C, int32_t *r_out,
                                           float *logits_out, const void *ws, size_t ws_bytes, uint32_t *dev_status,
                                           void *stream);
molora_status_t molora_route_mlp_prepare(molora_dtype_t xdt, int32_t d, int32_t H, int32_t C, const float *W1, void *ws,
                                         size_t ws_bytes, void *stream);
molora_status_t molora_route_mlp_prepared(const void *x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx,
                                          const float *W1, const float *b1, int32_t H, const float *W2, const float *b2,
                                          int32_t C, int32_t *r_out, float *logits_out, const void *ws, size_t ws_bytes,
                                          uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The same gate for callers that cannot provide a workspace.  (The paper has no counterpart: this entry point
 * exists for integration reasons only.)  Some hosts of this library may not allocate device memory at the
 * point where they route tokens -- code running between the capture and replay of a fixed-address serving
 * graph, plug-ins that are handed tensors but no allocator, allocation-free real-time loops -- and so cannot
 * supply molora_route_gate's `ws`.  This variant keeps the scratch inside the library instead: a fixed 2 MiB
 * device array that every GPU loading the library holds until the process exits.
 *   - Same arguments, results and errors as molora_route_gate, without ws / ws_bytes / dev_status (a wait that runs
 *     out still leaves r_out = -1 for its tile).
 *   - Limit: molora_route_gate_workspace_bytes(xdt, d, C) must not exceed 2 MiB (2 097 152 bytes); e.g.
 *     bf16 x with C <= 16 up to d = 19 328, with C <= 32 up to d = 8 704.  Larger gates are refused with
 *     MOLORA_ERR_WORKSPACE and nothing is enqueued.  Calls that need no scratch (fp32 x, or C <= 4) always fit.
 *   - It calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device looks up the array's device address (with that device current); make
 *     that first call outside any stream capture.
 *   - All calls on a device share the one array, which keeps whatever the previous call wrote.  The kernels
 *     rewrite every byte they later read, so nothing has to be cleared between calls -- but two calls that
 *     overlap on the GPU (different streams, or graph branches) race on it: serialise them.
 */
molora_status_t molora_route_gate_noalloc(const void *x, molora_dtype_t xdt, int64_t N, int32_t d, int64_t ldx,
                                          const float *G, const float *bias, int32_t C, int32_t *r_out,
                                          float *logits_out, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Grouping (Section 3.3 steps 1-3; Algorithm 2; Table 10 "histogram"):
 *     counts[c]    = |{ i : r[i] = c }|
 *     offsets[0]   = 0,  offsets[c+1] = offsets[c] + counts[c]
 *     perm[offsets[c] + k] = index of the k-th token (ascending i) with r[i] = c
 * The paper allocates positions with atomicAdd (order inside a group unspecified) and emits pointer
 * pairs xs/ys; this library emits the unique STABLE order as 32-bit token indices, from which
 * xs[c][k] = x + perm[offsets[c]+k]*ldx.  Results are exact and deterministic.
 * r        device int32[N]; values outside [0, C) are unrouted (values < -1 or >= C also set
 *          MOLORA_DEV_BAD_ROUTE in dev_status)
 * counts   device int32[C];  offsets  device int32[C+1];  perm  device int32[N] (first offsets[C] entries valid)
 * ws, ws_bytes  device scratch of at least molora_group_workspace_bytes(N, C) bytes, 16-byte aligned
 *               (may be NULL when that function returns 0).  Contents are undefined afterwards.
 * dev_status    device uint32 or NULL.
 * offsets/perm of one call may feed any number of molora_apply calls (one routing per layer). */
size_t molora_group_workspace_bytes(int64_t N, int32_t C);
molora_status_t molora_group(const int32_t *r, int64_t N, int32_t C, int32_t *counts, int32_t *offsets, int32_t *perm,
                             void *ws, size_t ws_bytes, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Grouped LoRA application (Eq. 2; Figure 2 "Grouped GEMM" + "Scatter to original positions";
 * weight shapes of Table 10): for every segment c and every token i = perm[j], offsets[c] <= j < offsets[c+1],
 *     t_i = x_i A_c            (shrink, d_in -> rank, fp32, kept on chip)
 *     y_i <- y_i + scale * t_i B_c   (expand, rank -> d_out; one rounding to the storage type)
 * Rows of y that belong to no segment are not touched.
 * x   device [N, d_in]  of type dt, pitch ldx;  never written
 * y   device [N, d_out] of type dt, pitch ldy;  in: base projection x W, out: h
 * A   device [C, d_in, rank] of type dt, dense;  B  device [C, rank, d_out] of type dt, dense
 * offsets, perm   device outputs of molora_group for the same N, C (read on the device only)
 * ws, ws_bytes    device scratch of at least molora_apply_workspace_bytes(...) bytes, 16-byte aligned (NULL if
 *                 that is 0).  Two kernels use it.  The job-list kernel (bf16, at most 1024 tokens, few tiles per SM:
 *                 decode-sized calls) keeps two control words and the fp32 partial shrink results there, the latter as
 *                 64-bit records {value, tag of the launch}: ALL of ws must be ZERO-FILLED before its first use (never
 *                 clear only a part of it later); after that the same ws can be passed to any number of calls, of any
 *                 shape, without clearing -- every launch counts itself in the control words and old records never
 *                 carry the current tag.  Calls that share one ws must not overlap on the GPU.  The
 *                 two-launch small-tile kernels (bf16 rank 64 below 1280 tokens with one or two rank-64 projections in
 *                 the call; with more than 64 adapters also the short segments of larger rank-64 calls) keep partial
 *                 shrink results [slice][N][rank] behind that.
 *                 MOLORA_ERR_WORKSPACE if ws is needed and NULL, misaligned or too small.
 * dev_status      device uint32 or NULL; MOLORA_DEV_TIMEOUT is OR-ed in if a bounded wait inside a kernel gave
 *                 up (the kernel then returns without hanging; y is incomplete)
 * The kernel variant is chosen per call on the host from rank, token count and bytes (tcgen05 tiles of 128 rows
 * for large calls, a single-launch streaming kernel with 32-row tiles below that, a job-list kernel with 16-row
 * tiles whose CTAs share chunk-sized shrink and expand jobs for decode-sized calls, CUDA cores for fp32 storage,
 * rank 8 and odd widths) and per segment on the device from the segment sizes; the paper picks its tile shape
 * from the histogram too (Eq. 12-13). */
size_t molora_apply_workspace_bytes(int64_t N, int32_t C, int32_t d_in, int32_t d_out, int32_t rank);
molora_status_t molora_apply(const void *x, int64_t ldx, void *y, int64_t ldy, molora_dtype_t dt, int64_t N,
                             int32_t d_in, int32_t d_out, int32_t rank, const void *A, const void *B, int32_t C,
                             const int32_t *offsets, const int32_t *perm, float scale, void *ws, size_t ws_bytes,
                             uint32_t *dev_status, void *stream);

/* Same operation for P projections that share N, C, offsets and perm (the projections of one layer),
 * enqueued as one launch per kernel variant.  `projs` is a HOST array of P descriptors (1 <= P <=
 * MOLORA_MAX_PROJECTIONS), copied at enqueue time; the pointers inside are device pointers with the meaning
 * given above.  ws needs the SUM of molora_apply_workspace_bytes(N, C, d_in, d_out, rank) over the projections. */
typedef struct {
    const void *x;
    int64_t ldx;
    void *y;
    int64_t ldy;
    const void *A;
    const void *B;
    int32_t d_in, d_out, rank;
    float scale;
    const float *row_scale; /* device fp32[N] or NULL: extra factor per TOKEN on its delta (the routing weight w_ij of
                               top-k routing, Eq. 8); NULL means 1 */
} molora_proj_desc_t;
molora_status_t molora_apply_batched(const molora_proj_desc_t *projs, int32_t P, molora_dtype_t dt, int64_t N,
                                     int32_t C, const int32_t *offsets, const int32_t *perm, void *ws, size_t ws_bytes,
                                     uint32_t *dev_status, void *stream);

/* Grouping and grouped application of one layer in one call (Section 3.3 steps 1-4, Algorithm 2): exactly
 * molora_group(r, ...) followed by molora_apply_batched(projs, ...) on its outputs, with the arguments, results
 * (counts, offsets and perm are written, bit-equal to molora_group's), status bits and error behaviour of those two
 * calls; ws / ws_bytes as for molora_apply_batched.  When every projection of the call runs on the single-launch
 * streaming kernel or on the job-list kernel with one rank (bf16, at most 4096 / 1024 tokens, below the tcgen05
 * crossover) the whole call is ONE launch: every CTA builds the grouping in its shared memory before its first copy
 * request, which saves the grouping launch; the two-launch small-tile kernels do the same for at most 1024 tokens;
 * otherwise the grouping launch and the apply launches are enqueued in stream order. */
molora_status_t molora_group_apply_batched(const int32_t *r, int64_t N, int32_t C, int32_t *counts, int32_t *offsets,
                                           int32_t *perm, const molora_proj_desc_t *projs, int32_t P,
                                           molora_dtype_t dt, void *ws, size_t ws_bytes, uint32_t *dev_status,
                                           void *stream);
/* 1 if that call is a single launch for these projections (host array, as above), this token count and this number
 * of adapters, else 0; pure host arithmetic, for callers that count launches. */
int32_t molora_group_apply_is_one_launch(const molora_proj_desc_t *projs, int32_t P, molora_dtype_t dt, int64_t N,
                                         int32_t C);
/* 1 if that call needs no separate grouping launch: the single launch above, or the two-launch small-tile kernels
 * grouping on chip (bf16, one rank, at most 1024 tokens; their launches are then the two of molora_apply_batched). */
int32_t molora_group_apply_skips_group_launch(const molora_proj_desc_t *projs, int32_t P, molora_dtype_t dt, int64_t N,
                                              int32_t C);

/* ---------------------------------------------------------------------------------------------
 * Top-k weighted routing (Eq. 8): w_i = softmax(TopK(z_i, k)), delta h_i = sum_j w_ij x_i A^(j) B^(j).
 * molora_topk_softmax turns router logits (logits_out of molora_route_gate / molora_route_mlp) into the k kept
 * adapters per token and their weights:
 *   logits   device fp32 [N, C], 1 <= k <= C <= 32
 *   idx_out  device int32 [k, N] slot-major: idx_out[j*N + i] = the j-th choice of token i (j = 0: largest logit;
 *            equal logits: lowest index first);  w_out  device fp32 [k, N], softmax over the k kept logits
 * molora_apply_topk applies the k choices.  Where the streaming kernel can take the call (bf16, k in {2, 4}, rank x k in
 * {16, 32, 64}, at most 256 adapter sets = binom(C + k - 1, k), below the tcgen05 crossover) or the tcgen05 kernel can (adapters of rank 16 or 32, rank x k in
 * {32, 64}, at most 64 adapter sets, widths multiples of 64) it does so in ONE pass over x and y: tokens are grouped by their
 * SET of kept adapters, a segment shrinks against the stacked A of its k adapters, the k slices of t are weighted per
 * token and one expand against the stacked B adds all k deltas before the single rounding.  Otherwise: k passes of
 * (group, apply) with the weights as per-token factors; within a pass every row of y is touched by one adapter only, so
 * there are no conflicting updates and the result is deterministic, but y is rounded to its storage type once per pass.
 *   projs    HOST array of P descriptors as for molora_apply_batched (their row_scale is ignored)
 *   ws       device scratch of at least molora_apply_topk_workspace_bytes(projs, P, N, C) bytes, 256-byte aligned,
 *            zero-filled before its first use (see molora_apply) */
molora_status_t molora_topk_softmax(const float *logits, int64_t N, int32_t C, int32_t k, int32_t *idx_out, float *w_out,
                                    void *stream);
size_t molora_apply_topk_workspace_bytes(const molora_proj_desc_t *projs, int32_t P, int64_t N, int32_t C);
molora_status_t molora_apply_topk(const molora_proj_desc_t *projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
                                  int32_t k, const int32_t *idx, const float *w, void *ws, size_t ws_bytes,
                                  uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Hot-set slot table (Definition 5.1, Eq. 10-11): S adapter slots of caller-owned, fixed-address stacks
 * A_hot[S, M, d, r] and B_hot[S, M, r, d] per projection, a slot table sigma : [S] -> adapter ids of a catalog of
 * n_catalog adapters, kept on the host, and its inverse on the device (table_dev: int32[n_catalog], adapter id -> slot,
 * -1 = not resident) that molora_route_hotset reads.  The table is maintained asynchronously: loads run on a
 * maintenance stream of the caller's, the compute streams never wait for them, and because every address is fixed the
 * forward pass can be replayed from a CUDA graph while slots are refilled.
 *
 * Life of a load:   molora_hotset_begin_load(adapter)  -> slot (a free one, else the least recently pinned slot that
 *                       nothing is using; the evicted adapter's table entry is cleared on the maintenance stream first);
 *                       if the adapter already has a slot, that slot with fresh = 0 and nothing else to do
 *                   molora_hotset_upload(slot, stack, weights) once per stack (A and B of every projection): copies
 *                       `bytes_per_slot` bytes from host memory to stack + slot * bytes_per_slot
 *                   molora_hotset_commit(slot): writes the table entry after the weights (stream order) and records an
 *                       event; the adapter counts as resident once that event has completed (polled, never waited for)
 * Life of a step:   molora_hotset_pin(adapter) for every adapter the step routes to (MOLORA_ERR_NOT_RESIDENT if it is not
 *                   there yet), enqueue the step, molora_hotset_unpin(slot) when the step has completed.  A pinned slot
 *                   is never chosen for eviction; MOLORA_ERR_BUSY if no slot can be had.
 * table_dev must hold -1 in every entry before the first load (the caller fills it).  S * M <= 256.  All functions are
 * thread-safe.  backend: NULL for the CUDA runtime (cudaMemcpyAsync from preferably pinned memory, cudaEvent*), or
 * replacements for the four calls (a fake stream for tests, another copy engine); `user` is passed through.
 * The manager allocates host memory for its own bookkeeping only, never device memory. */
typedef struct molora_hotset molora_hotset_t;
typedef struct {
    molora_status_t (*copy_h2d)(void *dst_dev, const void *src_host, size_t bytes, void *stream, void *user);
    molora_status_t (*event_record)(void **event /* in/out: created on first use */, void *stream, void *user);
    int32_t (*event_done)(void *event, void *user); /* 1 if everything before the record has completed (no waiting) */
    void (*event_destroy)(void *event, void *user);
    void *user;
} molora_hotset_backend_t;
molora_status_t molora_hotset_create(int32_t S, int32_t M, int32_t n_catalog, int32_t *table_dev,
                                     const molora_hotset_backend_t *backend, molora_hotset_t **out);
void molora_hotset_destroy(molora_hotset_t *h);
int32_t molora_hotset_slot_of(molora_hotset_t *h, int32_t adapter);  /* slot of a resident adapter, else -1 */
int32_t molora_hotset_adapter_in(molora_hotset_t *h, int32_t slot);  /* sigma(slot): adapter id, -1 if the slot is free */
molora_status_t molora_hotset_pin(molora_hotset_t *h, int32_t adapter, int32_t *slot_out);
molora_status_t molora_hotset_unpin(molora_hotset_t *h, int32_t slot);
molora_status_t molora_hotset_begin_load(molora_hotset_t *h, int32_t adapter, void *maintenance_stream, int32_t *slot_out,
                                         int32_t *fresh_out /* 1: upload + commit this slot; 0: already resident or on its way */,
                                         int32_t *evicted_out /* adapter that lost its slot, -1 if none; may be NULL */);
molora_status_t molora_hotset_upload(molora_hotset_t *h, int32_t slot, void *stack_dev, const void *weights_host,
                                     size_t bytes_per_slot, void *maintenance_stream);
molora_status_t molora_hotset_commit(molora_hotset_t *h, int32_t slot, void *maintenance_stream);
/* Compositional routing through the slot table (Definition 3.2 with the adapter axis indexed by slot):
 *     r_out[i] = slot_table_dev[adapter_id[i]] * M + m(ids[i]);  -1 if the id lies in no range, the adapter id is outside
 *     [0, n_catalog) or the adapter is not resident (MOLORA_DEV_ID_OUT_OF_RANGE is then OR-ed into dev_status).
 * The result indexes stacks of S * M targets: C = S * M in molora_group / molora_apply. */
molora_status_t molora_route_hotset(const int32_t *ids, const int32_t *adapter_id, int64_t N, const int32_t *breaks,
                                    int32_t M, const int32_t *slot_table_dev, int32_t n_catalog, int32_t S,
                                    int32_t *r_out, uint32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------------------------
 * Failure-detection self-test.  Every device-side wait of the tensor-core apply kernel (on an mbarrier that a
 * producer warp, the tensor core or a peer CTA of the cluster completes) is bounded: a waiter that gives up sets
 * MOLORA_DEV_TIMEOUT in the status word and an abort flag after which all waits of the CTA fall through, so the
 * kernel returns and the context stays usable.  This entry point exercises exactly that code on a barrier that
 * nothing ever completes, with a limit of `limit_cycles` SM cycles (1 .. 2e9): afterwards *dev_status has
 * MOLORA_DEV_TIMEOUT set, result[0] == 1 (abort flag raised) and result[1] == 1 (a second wait fell through).
 * dev_status: device uint32; result: device int32[2].  Nothing faults, traps or spins without bound. */
molora_status_t molora_selftest_bounded_wait(uint32_t *dev_status, int64_t limit_cycles, int32_t *result, void *stream);

/* ---------------------------------------------------------------------------------------------
 * The whole path on HOST activations (one layer: route -> group -> apply for P projections), for callers
 * whose activations live in host memory.  Everything is enqueued on `stream` in this order: host-to-device
 * copies of the routing source and of every distinct x and every y into `arena`, the router, the grouping,
 * one batched apply (Eq. 2), device-to-host copies of every y back into y_host.  The call returns without
 * waiting; x_host / y_host must stay valid (and should be pinned for the copies to be asynchronous) until the
 * stream has finished.  Adapter stacks, gate weights and vocabulary breaks are DEVICE pointers: weights stay
 * resident at fixed addresses (the hot-set idea of Definition 5.1), only activations travel.
 *
 * router       MOLORA_ROUTE_VOCAB: route_src_host = ids int32[N], breaks_dev int32[M+1]
 *              MOLORA_ROUTE_GATE:  the gate reads the staged x of projection `gate_proj`; G_dev fp32 [d_in, C],
 *                                  bias_dev fp32 [C] or NULL
 *              MOLORA_ROUTE_GIVEN: route_src_host = r int32[N]
 * projs        HOST array of P descriptors (1 <= P <= MOLORA_MAX_PROJECTIONS); projections whose x_host
 *              pointers are equal share one staged copy
 * arena        device scratch of at least molora_forward_host_arena_bytes(...) bytes, 256-byte aligned, zero-filled
 *              before its first use (it holds the apply workspace, see molora_apply)
 * dev_status   device uint32 or NULL (as for the individual calls)
 * Errors are detected before anything is enqueued, as for the individual calls. */
typedef enum { MOLORA_ROUTE_VOCAB = 0, MOLORA_ROUTE_GATE = 1, MOLORA_ROUTE_GIVEN = 2 } molora_router_t;
typedef struct {
    const void *x_host; /* [N, d_in]  dense (pitch d_in)                         */
    void *y_host;       /* [N, d_out] dense; in: base projection x W, out: h     */
    const void *A;      /* device [C, d_in, rank]                                */
    const void *B;      /* device [C, rank, d_out]                               */
    int32_t d_in, d_out, rank;
    float scale;
} molora_host_proj_t;
size_t molora_forward_host_arena_bytes(const molora_host_proj_t *projs, int32_t P, molora_dtype_t dt, int64_t N,
                                       int32_t C, molora_router_t router, int32_t gate_proj);
molora_status_t molora_forward_host(molora_router_t router, const int32_t *route_src_host, const int32_t *breaks_dev,
                                    int32_t M, const float *G_dev, const float *bias_dev, int32_t gate_proj,
                                    const molora_host_proj_t *projs, int32_t P, molora_dtype_t dt, int64_t N, int32_t C,
                                    void *arena, size_t arena_bytes, uint32_t *dev_status, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* MOLORA_H_ */
