/*
 * fp64 CPU oracle for the WKV-6 (Finch / RWKV-6) time-mix recurrence that the
 * Finch-C2 layers of GoldFinch run during linear-time pre-fill.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
 * check and the CPU-baseline leg of the benchmark may call it.  It shares no
 * code, header, table or helper with the CUDA library and is deliberately the
 * slow, literal definition:
 *
 *   per head (heads are independent: the Finch-C2 formulae are stated per head,
 *   "after splitting the hidden dimension into heads"), with S an N x N matrix,
 *   S[i][j], i = key channel, j = value channel:
 *
 *     w_t      = exp(-exp(x_t))                                  (decay, Finch-C2 block eq. for w_t)
 *     y_t[j]   = sum_i r_t[i] * ( S_{t-1}[i][j] + u[i] k_t[i] v_t[j] )
 *     S_t[i][j]= w_t[i] * S_{t-1}[i][j] + k_t[i] v_t[j]
 *
 *   S_{t-1} is the paper's wkv_t = sum_{i<t} diag(prod_{j=i+1}^{t-1} w_j) k_i^T v_i
 *   (the wkv_t equation of the Finch-C2 section): the newest term i = t-1 carries
 *   the empty product, so w_t first acts when S_t is formed, and the output uses
 *   the state *before* the update.  With u == 0 the output is the paper's
 *   r_t . wkv_t; the diag(u) "bonus" term is classic Finch's, which the paper
 *   names only in passing and the library's contract defines.
 *
 * Pins (tests/test_oracle_pins.py): brute-force expansion of the wkv_t sum at
 * T <= 8, w == 1 cumulative-sum closed form, w == 0 special case, constant
 * w = 1/2 geometric closed form, split-and-carry, linearity / k-v rescaling,
 * head independence, orientation probes, a hand-computed worked example.  The Finch-C2
 * form at the end of this file (k (1 - w) keys, second-value vector, no bonus) is pinned in
 * tests/test_oracle_pins_c2.py: brute-force expansion, reduction to the bonus-free recurrence on
 * premultiplied keys, w == 1 / w == 0 special cases, constant w = 1/2 closed form, split-and-carry.
 *
 * Inputs arrive as float (an exact carrier for both fp32 and bf16 data) and are
 * widened to double before any arithmetic; every sum runs in double in plain
 * index order.  Layouts: r,k,v,x,y are [B][T][H][N] (N fastest), u is [H][N],
 * states are [B][H][N][N] row-major with i (key channel) before j (value channel).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int wkv6_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One (sequence, head) unit.  Rows of r,k,v,x,y are `row_stride` elements apart.
 * If w_direct != NULL it holds the decay w itself (same indexing as x) and x is
 * ignored: this lets the invariants w == 1 and w == 0 be stated exactly. */
static void unit_recurrence(const float *r, const float *k, const float *v, const float *x,
                            const double *w_direct, const float *u, const float *s_in,
                            double *s_out, double *y, long T, long N, long row_stride)
{
    double *S = (double *)malloc((size_t)N * N * sizeof(double));
    double *w = (double *)malloc((size_t)N * sizeof(double));
    for (long i = 0; i < N * N; ++i) S[i] = s_in ? (double)s_in[i] : 0.0;

    for (long t = 0; t < T; ++t) {
        const float *rt = r + t * row_stride, *kt = k + t * row_stride, *vt = v + t * row_stride;
        double *yt = y + t * row_stride;
        for (long c = 0; c < N; ++c)
            w[c] = w_direct ? w_direct[t * row_stride + c] : exp(-exp((double)x[t * row_stride + c]));
        /* output from the state before the update */
        for (long j = 0; j < N; ++j) {
            double acc = 0.0;
            for (long i = 0; i < N; ++i)
                acc += (double)rt[i] * (S[i * N + j] + (double)u[i] * (double)kt[i] * (double)vt[j]);
            yt[j] = acc;
        }
        /* decay row i by w_t[i], then add the rank-1 term k_t^T v_t */
        for (long i = 0; i < N; ++i)
            for (long j = 0; j < N; ++j)
                S[i * N + j] = w[i] * S[i * N + j] + (double)kt[i] * (double)vt[j];
    }
    if (s_out) memcpy(s_out, S, (size_t)N * N * sizeof(double));
    free(S);
    free(w);
}

/* Dense batch: r,k,v,x (and w_direct if given) are [B][T][H][N]; y likewise (double).
 * state_in may be NULL (zero state); state_out may be NULL. */
void wkv6_oracle_prefill(const float *r, const float *k, const float *v, const float *x,
                         const double *w_direct, const float *u, const float *state_in,
                         double *state_out, double *y, long B, long T, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long b = 0; b < B; ++b)
        for (long h = 0; h < H; ++h) {
            const size_t off = (size_t)b * T * C + (size_t)h * N;
            const size_t soff = ((size_t)b * H + h) * N * N;
            unit_recurrence(r + off, k + off, v + off, x ? x + off : NULL,
                            w_direct ? w_direct + off : NULL, u + h * N,
                            state_in ? state_in + soff : NULL,
                            state_out ? state_out + soff : NULL, y + off, T, N, C);
        }
}

/* Packed variable-length batch: rows cu_seqlens[s] .. cu_seqlens[s+1]-1 of the
 * [total_T][H][N] tensors form sequence s; states are [S][H][N][N]. */
void wkv6_oracle_prefill_varlen(const float *r, const float *k, const float *v, const float *x,
                                const float *u, const float *state_in, double *state_out,
                                double *y, const int32_t *cu_seqlens, long S, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long s = 0; s < S; ++s)
        for (long h = 0; h < H; ++h) {
            const long t0 = cu_seqlens[s], len = cu_seqlens[s + 1] - cu_seqlens[s];
            const size_t off = (size_t)t0 * C + (size_t)h * N;
            const size_t soff = ((size_t)s * H + h) * N * N;
            unit_recurrence(r + off, k + off, v + off, x + off, NULL, u + h * N,
                            state_in ? state_in + soff : NULL,
                            state_out ? state_out + soff : NULL, y + off, len, N, C);
        }
}

/*
 * The Finch-C2 form of the same recurrence, as the paper's Finch-C2 block writes it: the key that
 * enters the state is the projected key times one minus the decay of its own token,
 *     k'_t = k_t * (1 - w_t)                       (Finch-C2 block, k_t equation)
 * there is no bonus term, and the per-head output is r_t . wkv_t + u'_t with wkv_t = S_{t-1} and
 * u'_t the "second value" vector of the token (o_t equation, before LayerNorm / W^O):
 *     y_t[j]    = sum_i r_t[i] S_{t-1}[i][j] + u2_t[j]
 *     S_t[i][j] = w_t[i] S_{t-1}[i][j] + k'_t[i] v_t[j]
 * u2 may be NULL (no added vector).  w_direct as in unit_recurrence.  Same layouts.
 */
static void unit_recurrence_c2(const float *r, const float *k, const float *v, const float *x,
                               const double *w_direct, const float *u2, const float *s_in,
                               double *s_out, double *y, long T, long N, long row_stride)
{
    double *S = (double *)malloc((size_t)N * N * sizeof(double));
    double *w = (double *)malloc((size_t)N * sizeof(double));
    for (long i = 0; i < N * N; ++i) S[i] = s_in ? (double)s_in[i] : 0.0;
    for (long t = 0; t < T; ++t) {
        const float *rt = r + t * row_stride, *kt = k + t * row_stride, *vt = v + t * row_stride;
        double *yt = y + t * row_stride;
        for (long c = 0; c < N; ++c)
            w[c] = w_direct ? w_direct[t * row_stride + c] : exp(-exp((double)x[t * row_stride + c]));
        for (long j = 0; j < N; ++j) {
            double acc = 0.0;
            for (long i = 0; i < N; ++i) acc += (double)rt[i] * S[i * N + j];
            yt[j] = acc + (u2 ? (double)u2[t * row_stride + j] : 0.0);
        }
        for (long i = 0; i < N; ++i) {
            const double kp = (double)kt[i] * (1.0 - w[i]);
            for (long j = 0; j < N; ++j) S[i * N + j] = w[i] * S[i * N + j] + kp * (double)vt[j];
        }
    }
    if (s_out) memcpy(s_out, S, (size_t)N * N * sizeof(double));
    free(S);
    free(w);
}

void wkv6_oracle_prefill_c2(const float *r, const float *k, const float *v, const float *x,
                            const double *w_direct, const float *u2, const float *state_in,
                            double *state_out, double *y, long B, long T, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long b = 0; b < B; ++b)
        for (long h = 0; h < H; ++h) {
            const size_t off = (size_t)b * T * C + (size_t)h * N;
            const size_t soff = ((size_t)b * H + h) * N * N;
            unit_recurrence_c2(r + off, k + off, v + off, x ? x + off : NULL,
                               w_direct ? w_direct + off : NULL, u2 ? u2 + off : NULL,
                               state_in ? state_in + soff : NULL,
                               state_out ? state_out + soff : NULL, y + off, T, N, C);
        }
}

/* ---------------------------------------------------------------------------------------------------
 * LayerNorm across all heads: the normalisation in the o_t equation of the Finch-C2 block,
 *     o_t = LayerNorm(concat_h(r_t . wkv_t + u'_t)) W^O,
 * i.e. one LayerNorm over the D = H*N concatenated channels of a token (the paper replaces Finch's
 * per-head GroupNorm by it), before the output projection.  The paper gives no formula for the
 * operator; this is its standard definition (Ba, Kiros, Hinton 2016) with the customary per-channel
 * affine pair and the eps inside the square root:
 *     mu = (1/D) sum_c y[c],   var = (1/D) sum_c (y[c] - mu)^2          (biased variance)
 *     out[c] = (y[c] - mu) / sqrt(var + eps) * gamma[c] + beta[c]
 * gamma / beta may be NULL (1 / 0).  y, out: [rows][D] double, every sum in index order.
 * Pins (tests/test_oracle_pins_ln.py): closed form on an arithmetic progression, the two-element row,
 * a constant row, the library LayerNorm in float64, mean / variance of the output, shift and scale laws,
 * the difference to a per-head norm, channel indexing of gamma and beta.
 */
void c2_oracle_layernorm(const double *y, const double *gamma, const double *beta, double eps,
                         double *out, long rows, long D)
{
#pragma omp parallel for schedule(static)
    for (long row = 0; row < rows; ++row) {
        const double *yr = y + (size_t)row * D;
        double *o = out + (size_t)row * D;
        double mu = 0.0, var = 0.0;
        for (long c = 0; c < D; ++c) mu += yr[c];
        mu /= (double)D;
        for (long c = 0; c < D; ++c) var += (yr[c] - mu) * (yr[c] - mu);
        var /= (double)D;
        const double rstd = 1.0 / sqrt(var + eps);
        for (long c = 0; c < D; ++c)
            o[c] = (yr[c] - mu) * rstd * (gamma ? gamma[c] : 1.0) + (beta ? beta[c] : 0.0);
    }
}

/* ---------------------------------------------------------------------------------------------------
 * GOLD key compression: the step that ends linear pre-fill in GoldFinch.  The output x_t of the Finch-C2
 * layers is multiplied by the learned matrix W^{KD} in R^{D x D/16} and the result stored as the token's
 * entry of the compressed key cache:
 *     c_t = x_t W^{KD}                                   (GOLD key compression equation)
 * x: [rows][D], w: [D][Dc] row-major (Dc = D/16 in the paper; any Dc here), c: [rows][Dc]; every sum in
 * double, in index order over the D input channels.
 * Pins (tests/test_oracle_pins_kc.py): brute-force loops on a tiny case, a selection matrix, the all-ones
 * matrix (row sums), a single non-zero weight (orientation), linearity, the library matrix product in fp64.
 */
void gold_oracle_key_compress(const double *x, const double *w, double *c, long rows, long D, long Dc)
{
#pragma omp parallel for schedule(static)
    for (long t = 0; t < rows; ++t)
        for (long n = 0; n < Dc; ++n) {
            double acc = 0.0;
            for (long k = 0; k < D; ++k) acc += x[(size_t)t * D + k] * w[(size_t)k * Dc + n];
            c[(size_t)t * Dc + n] = acc;
        }
}
