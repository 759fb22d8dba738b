/*
 * CPU oracle for per-token routed LoRA.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct restatement of what the routed-LoRA path computes, written from
 * the paper's definitions.  Every floating-point sum is carried in fp64, in index order, one token
 * at a time in the ORIGINAL token order; the grouping (histogram / offsets / permutation) is never
 * used to compute the LoRA result, so comparing the CUDA path's output with oracle_apply() checks
 * routing, grouping and the grouped shrink/expand end to end.
 *
 * Nothing here is shared with the CUDA path (no headers, helpers, tables or constants), and only the
 * tests, the smoke check and the benchmark's cpu-baseline leg may call it.
 *
 * Inputs are float32 arrays; for bf16 workloads they hold bf16-representable values, so the
 * conversion to double below is exact for both storage types.
 *
 * The only parallelism is an OpenMP "for" over tokens (tokens are independent in Eq. 2); each
 * token's arithmetic is serial and in index order, so results do not depend on the thread count.
 *
 * Pinned by tests/test_oracle_pins.py (constant routing == dense LoRA by a library matmul, selector
 * closed forms, the grouping example of Figure 2, upper_bound for vocabulary routing, exhaustive
 * routings on integer data, permutation equivariance, the N vs K*N work count of Theorem 3.6).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Definition 3.1 / Eq. 3 (vocabulary routing), read 0-based: with breaks b_0 <= b_1 <= ... <= b_M,
 * R(v) = m  <=>  b_m <= v < b_{m+1},  m in [0, M).  An id that lies in no range is unrouted (-1).
 * Linear search over the M ranges, exactly as the definition reads. */
int oracle_route_vocab(const int32_t *ids, int64_t N, const int32_t *breaks, int32_t M, int32_t *r)
{
    if (N < 0 || M <= 0) return 1;
    for (int64_t i = 0; i < N; ++i) {
        int32_t found = -1;
        for (int32_t m = 0; m < M; ++m) {
            if (breaks[m] <= ids[i] && ids[i] < breaks[m + 1]) { found = m; break; }
        }
        r[i] = found;
    }
    return 0;
}

/* Compositional routing (Definition 3.2, Algorithm 1 lines 4-6): a <- adapter index of the token from the request
 * metadata, m <- FindModality(v, b), c <- a * |M| + m.  A token whose id lies in no range, or whose adapter index
 * is outside [0, n_adapters), is unrouted (-1). */
int oracle_route_composite(const int32_t *ids, const int32_t *adapter, int64_t N, const int32_t *breaks, int32_t M,
                           int32_t n_adapters, int32_t *r)
{
    if (N < 0 || M <= 0 || n_adapters <= 0) return 1;
    for (int64_t t = 0; t < N; ++t) {
        const int32_t a = adapter[t];
        int32_t m = -1;
        for (int32_t j = 0; j < M; ++j) {
            if (breaks[j] <= ids[t] && ids[t] < breaks[j + 1]) { m = j; break; }
        }
        r[t] = (m >= 0 && a >= 0 && a < n_adapters) ? a * M + m : -1;
    }
    return 0;
}

/* Linear gate with top-1 selection (Eq. 8 with k = 1; the gate of Theorem 3.4 / Table 10 is
 * softmax(W x + b)).  Softmax is monotone, so the winner is the argmax of the raw logits
 * z[i][c] = sum_k x[i][k] * G[k][c] (+ bias[c]); with a single kept logit the softmax weight is 1.
 * Ties go to the lowest index.  margin[i] = (largest logit) - (second largest logit); for C == 1 it
 * is +infinity-like (1e300). */
int oracle_route_gate(const float *x, int64_t N, int32_t d, int64_t ldx, const float *G, const float *bias,
                      int32_t C, int32_t *r, double *z_out, double *margin_out)
{
    if (N < 0 || d <= 0 || C <= 0 || ldx < d) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double best = 0.0, second = 0.0;
        int32_t arg = -1;
        for (int32_t c = 0; c < C; ++c) {
            double z = 0.0;
            for (int32_t k = 0; k < d; ++k) z += (double)x[i * ldx + k] * (double)G[(int64_t)k * C + c];
            if (bias) z += (double)bias[c];
            if (z_out) z_out[i * C + c] = z;
            if (arg < 0) { best = z; arg = c; second = -1e300; }
            else if (z > best) { second = best; best = z; arg = c; }
            else if (z > second) { second = z; }
        }
        r[i] = arg;
        if (margin_out) margin_out[i] = (C > 1) ? best - second : 1e300;
    }
    return 0;
}

/* The paper's router (Eq. 9): g(x) = W2 GELU(W1 x + b1) + b2, a 2-layer MLP with hidden width H (64 in Eq. 9, 128 in
 * the 2560 -> 128 -> 4 variant of the appendix), followed by top-1 selection as in oracle_route_gate.  GELU is the
 * exact form t * Phi(t) = t * (1 + erf(t / sqrt 2)) / 2.  Weights are stored input-major: W1[d][H], W2[H][C].
 * z_out (optional) receives the logits, h_out (optional) the hidden activations after GELU. */
int oracle_route_mlp(const float *x, int64_t N, int32_t d, int64_t ldx, const float *W1, const float *b1, int32_t H,
                     const float *W2, const float *b2, int32_t C, int32_t *r, double *z_out, double *margin_out,
                     double *h_out)
{
    if (N < 0 || d <= 0 || H <= 0 || C <= 0 || ldx < d) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double h[1024];
        if (H > 1024) continue;
        for (int32_t j = 0; j < H; ++j) {
            double t = b1 ? (double)b1[j] : 0.0;
            for (int32_t k = 0; k < d; ++k) t += (double)W1[(int64_t)k * H + j] * (double)x[i * ldx + k];
            h[j] = 0.5 * t * (1.0 + erf(t / sqrt(2.0)));
            if (h_out) h_out[i * H + j] = h[j];
        }
        double best = 0.0, second = 0.0;
        int32_t arg = -1;
        for (int32_t c = 0; c < C; ++c) {
            double z = b2 ? (double)b2[c] : 0.0;
            for (int32_t j = 0; j < H; ++j) z += (double)W2[(int64_t)j * C + c] * h[j];
            if (z_out) z_out[i * C + c] = z;
            if (arg < 0) { best = z; arg = c; second = -1e300; }
            else if (z > best) { second = best; best = z; arg = c; }
            else if (z > second) { second = z; }
        }
        r[i] = arg;
        if (margin_out) margin_out[i] = (C > 1) ? best - second : 1e300;
    }
    return 0;
}

/* Section 3.3 (unified dispatch), steps 1-3, with a deterministic order inside each group:
 *   counts[c]  = |{ i : r[i] = c }|                        (the histogram h)
 *   offsets[0] = 0, offsets[c+1] = offsets[c] + counts[c]   (position allocation)
 *   perm[offsets[c] + k] = the k-th token, in ascending token index, routed to c
 * Tokens with r[i] outside [0, C) belong to no group.  O(N*C) double loop: trivially stable. */
int oracle_group(const int32_t *r, int64_t N, int32_t C, int32_t *counts, int32_t *offsets, int32_t *perm)
{
    if (N < 0 || C <= 0) return 1;
    int64_t p = 0;
    offsets[0] = 0;
    for (int32_t c = 0; c < C; ++c) {
        int32_t n = 0;
        for (int64_t i = 0; i < N; ++i) {
            if (r[i] == c) { perm[p++] = (int32_t)i; ++n; }
        }
        counts[c] = n;
        offsets[c + 1] = offsets[c] + n;
    }
    return 0;
}

/* One token through one adapter: h = y + scale * (x A_c) B_c, A_c [d_in, rank], B_c [rank, d_out]. */
static void lora_row(const float *x, const float *y, const float *Ac, const float *Bc, int32_t d_in, int32_t d_out,
                     int32_t rank, double scale, double *t, double *h)
{
    for (int32_t k = 0; k < rank; ++k) {
        double s = 0.0;
        for (int32_t j = 0; j < d_in; ++j) s += (double)x[j] * (double)Ac[(int64_t)j * rank + k];
        t[k] = s;
    }
    for (int32_t o = 0; o < d_out; ++o) {
        double s = 0.0;
        for (int32_t k = 0; k < rank; ++k) s += t[k] * (double)Bc[(int64_t)k * d_out + o];
        h[o] = (double)y[o] + scale * s;
    }
}

/* Eq. 2 (per-token routing): h_i = y_i + scale * x_i A_{r(i)} B_{r(i)} with y_i = x_i W supplied by the
 * caller; tokens with r(i) outside [0, C) keep h_i = y_i.  Weight layout follows Table 10:
 * A is (C, d_in, rank), B is (C, rank, d_out), both row-major.  *products counts token-adapter
 * products (Theorem 3.6: N for per-token routing, counting routed tokens). */
int oracle_apply(const float *x, int64_t ldx, const float *y, int64_t ldy, const float *A, const float *B,
                 const int32_t *r, int64_t N, int32_t d_in, int32_t d_out, int32_t rank, int32_t C, double scale,
                 double *h, int64_t *products)
{
    if (N < 0 || d_in <= 0 || d_out <= 0 || rank <= 0 || C <= 0 || ldx < d_in || ldy < d_out) return 1;
    int64_t count = 0;
#pragma omp parallel for schedule(static) reduction(+ : count)
    for (int64_t i = 0; i < N; ++i) {
        int32_t c = r[i];
        double *hi = h + i * (int64_t)d_out;
        if (c < 0 || c >= C) {
            for (int32_t o = 0; o < d_out; ++o) hi[o] = (double)y[i * ldy + o];
            continue;
        }
        double *t = (double *)malloc(sizeof(double) * (size_t)rank);
        lora_row(x + i * ldx, y + i * ldy, A + (int64_t)c * d_in * rank, B + (int64_t)c * rank * d_out, d_in, d_out,
                 rank, scale, t, hi);
        free(t);
        ++count;
    }
    if (products) *products = count;
    return 0;
}

/* Top-k weighted routing (Eq. 8): from the logits z_i the k largest are kept (ties: lowest index first), and
 * w_i = softmax over the kept logits.  idx and w are slot-major: idx[j * N + i] is the j-th choice of token i
 * (j = 0 the largest logit).  k <= C. */
int oracle_topk_softmax(const double *z, int64_t N, int32_t C, int32_t k, int32_t *idx, double *w)
{
    if (N < 0 || C <= 0 || k <= 0 || k > C) return 1;
    for (int64_t i = 0; i < N; ++i) {
        const double *zi = z + i * (int64_t)C;
        for (int32_t j = 0; j < k; ++j) {
            int32_t best = -1;
            for (int32_t c = 0; c < C; ++c) {
                int taken = 0;
                for (int32_t q = 0; q < j; ++q) taken |= idx[(int64_t)q * N + i] == c;
                if (taken) continue;
                if (best < 0 || zi[c] > zi[best]) best = c;
            }
            idx[(int64_t)j * N + i] = best;
        }
        const double zmax = zi[idx[i]];
        double den = 0.0;
        for (int32_t j = 0; j < k; ++j) den += exp(zi[idx[(int64_t)j * N + i]] - zmax);
        for (int32_t j = 0; j < k; ++j) w[(int64_t)j * N + i] = exp(zi[idx[(int64_t)j * N + i]] - zmax) / den;
    }
    return 0;
}

/* Eq. 8, second half: h_i = y_i + scale * sum_j w_ij x_i A^(r_ij) B^(r_ij) over the k kept adapters of token i
 * (slot-major idx, w as above; an index outside [0, C) contributes nothing). */
int oracle_apply_topk(const float *x, int64_t ldx, const float *y, int64_t ldy, const float *A, const float *B,
                      const int32_t *idx, const double *w, int32_t k, int64_t N, int32_t d_in, int32_t d_out,
                      int32_t rank, int32_t C, double scale, double *h)
{
    if (N < 0 || d_in <= 0 || d_out <= 0 || rank <= 0 || C <= 0 || k <= 0 || ldx < d_in || ldy < d_out) return 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < N; ++i) {
        double *hi = h + i * (int64_t)d_out;
        for (int32_t o = 0; o < d_out; ++o) hi[o] = (double)y[i * ldy + o];
        for (int32_t j = 0; j < k; ++j) {
            const int32_t c = idx[(int64_t)j * N + i];
            if (c < 0 || c >= C) continue;
            const float *Ac = A + (int64_t)c * d_in * rank, *Bc = B + (int64_t)c * rank * d_out;
            for (int32_t q = 0; q < rank; ++q) {
                double t = 0.0;
                for (int32_t kk = 0; kk < d_in; ++kk) t += (double)x[i * ldx + kk] * (double)Ac[(int64_t)kk * rank + q];
                t *= scale * w[(int64_t)j * N + i];
                for (int32_t o = 0; o < d_out; ++o) hi[o] += t * (double)Bc[(int64_t)q * d_out + o];
            }
        }
    }
    return 0;
}

/* Per-sequence routing served as K passes (Eq. 1 applied once per adapter, Theorem 3.6): pass k runs
 * the dense single-adapter LoRA of adapter k over ALL N tokens, then only rows with r[i] == k are kept.
 * Work is K*N token-adapter products.  The result must equal oracle_apply() bit for bit. */
int oracle_apply_perseq_kpass(const float *x, int64_t ldx, const float *y, int64_t ldy, const float *A,
                              const float *B, const int32_t *r, int64_t N, int32_t d_in, int32_t d_out,
                              int32_t rank, int32_t K, double scale, double *h, int64_t *products)
{
    if (N < 0 || d_in <= 0 || d_out <= 0 || rank <= 0 || K <= 0 || ldx < d_in || ldy < d_out) return 1;
    int64_t count = 0;
    double *pass = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1) * (size_t)d_out);
    if (!pass) return 2;
    for (int64_t i = 0; i < N; ++i)
        for (int32_t o = 0; o < d_out; ++o) h[i * (int64_t)d_out + o] = (double)y[i * ldy + o];
    for (int32_t k = 0; k < K; ++k) {
        int64_t pass_count = 0;
#pragma omp parallel for schedule(static) reduction(+ : pass_count)
        for (int64_t i = 0; i < N; ++i) {
            double *t = (double *)malloc(sizeof(double) * (size_t)rank);
            lora_row(x + i * ldx, y + i * ldy, A + (int64_t)k * d_in * rank, B + (int64_t)k * rank * d_out, d_in,
                     d_out, rank, scale, t, pass + i * (int64_t)d_out);
            free(t);
            ++pass_count;
        }
        count += pass_count;
        for (int64_t i = 0; i < N; ++i)
            if (r[i] == k) memcpy(h + i * (int64_t)d_out, pass + i * (int64_t)d_out, sizeof(double) * (size_t)d_out);
    }
    free(pass);
    if (products) *products = count;
    return 0;
}
