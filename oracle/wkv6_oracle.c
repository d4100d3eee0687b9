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
 * Further down: the LayerNorm across all heads (tests/test_oracle_pins_ln.py), the GOLD key compression
 * (tests/test_oracle_pins_kc.py), the decay logit d_t = lora_omega(ddlerp_d(x_t, x_{t-1})) of the Finch-C2 block
 * (tests/test_oracle_pins_dl.py: operator end points, an invertible outer lora that exposes the inner ddlerp, scalar
 * loops, library routines, a hand value, token-shift laws) and the gradient of the recurrence
 * (tests/test_oracle_pins_bwd.py: central differences of the forward pass, the one-token closed form, linearity,
 * split-and-carry of the adjoint) and of its Finch-C2 form (tests/test_oracle_pins_bwd_c2.py: central differences, the
 * reduction to the classic gradient on premultiplied keys with the chain rule written out, the one-token closed form).
 * No function here is unpinned.
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

/*
 * The decay logit of the Finch-C2 block, d_t = lora_omega( ddlerp_d( x_t, x_{t-1} ) ), with the three
 * operators the Finch-C2 section defines (all vectors have the D channels of the model dimension, the two
 * low-rank matrices of a lora are A [D][R] and B [R][D], row-major):
 *     lerp(a, b, t)   = a + (b - a) .* t
 *     lora(x)         = lambda + tanh(x A) B
 *     ddlerp(a, b)    = a + (b - a) .* lora( a + (b - a) .* mu_x )
 * Each operator is one function below, written as the formula reads, and the logit is their composition:
 * lora_d (rank Rd: A_d, B_d, lambda_d) inside ddlerp_d, lora_omega (rank Rw) outside.  x_{t-1} of a sequence's
 * first token is the row x_prev[b] (the token before the call; NULL: zeros).
 * x: [B][T][D] double, x_prev: [B][D] or NULL, d: [B][T][D] double.  Pinned in tests/test_oracle_pins_dl.py.
 */
static void op_lerp(const double *a, const double *b, const double *t, double *out, long D)
{
    for (long c = 0; c < D; ++c) out[c] = a[c] + (b[c] - a[c]) * t[c];
}

static void op_lora(const double *x, const double *A, const double *Bm, const double *lambda, long D, long R,
                    double *out)
{
    double *h = (double *)malloc((size_t)(R > 0 ? R : 1) * sizeof(double));
    for (long q = 0; q < R; ++q) {
        double acc = 0.0;
        for (long c = 0; c < D; ++c) acc += x[c] * A[c * R + q];          /* (x A)[q] */
        h[q] = tanh(acc);
    }
    for (long c = 0; c < D; ++c) {
        double acc = 0.0;
        for (long q = 0; q < R; ++q) acc += h[q] * Bm[q * D + c];         /* (tanh(x A) B)[c] */
        out[c] = lambda[c] + acc;
    }
    free(h);
}

static void op_ddlerp(const double *a, const double *b, const double *mu_x, const double *A, const double *Bm,
                      const double *lambda, long D, long R, double *out)
{
    double *inner = (double *)malloc((size_t)D * sizeof(double));
    double *mix = (double *)malloc((size_t)D * sizeof(double));
    op_lerp(a, b, mu_x, inner, D);                 /* a + (b - a) .* mu_x */
    op_lora(inner, A, Bm, lambda, D, R, mix);      /* lora( . ) */
    op_lerp(a, b, mix, out, D);                    /* a + (b - a) .* lora( . ) */
    free(inner);
    free(mix);
}

void c2_oracle_decay_logit(const double *x, const double *x_prev, const double *mu_x, const double *A_d,
                           const double *B_d, const double *lambda_d, long Rd, const double *A_w,
                           const double *B_w, const double *lambda_w, long Rw, double *d, long B, long T, long D)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (long b = 0; b < B; ++b)
        for (long t = 0; t < T; ++t) {
            double *shifted = (double *)malloc((size_t)D * sizeof(double));
            double *mixed = (double *)malloc((size_t)D * sizeof(double));
            const double *xt = x + ((size_t)b * T + t) * D;
            for (long c = 0; c < D; ++c)                                   /* x_{t-1} */
                shifted[c] = t > 0 ? xt[c - D] : (x_prev ? x_prev[(size_t)b * D + c] : 0.0);
            op_ddlerp(xt, shifted, mu_x, A_d, B_d, lambda_d, D, Rd, mixed);
            op_lora(mixed, A_w, B_w, lambda_w, D, Rw, d + ((size_t)b * T + t) * D);
            free(shifted);
            free(mixed);
        }
}

/*
 * Gradient of the recurrence at the top of this file (training runs it backwards; the paper trains its models
 * with it and fine-tunes with the recurrent part frozen).  For a scalar loss L with dy_t = dL/dy_t and
 * dS_T = dL/dS_T given, the adjoint G_t = dL/dS_t of the state is carried from t = T down to 1 through the two
 * places S_{t-1} enters (the output y_t and the update to S_t):
 *     G_{t-1}[i][j] = w_t[i] G_t[i][j] + r_t[i] dy_t[j]
 * and every input's gradient is read off the forward formulas
 *     y_t[j]    = sum_i r_t[i] ( S_{t-1}[i][j] + u[i] k_t[i] v_t[j] ),   S_t[i][j] = w_t[i] S_{t-1}[i][j] + k_t[i] v_t[j]:
 *     dr_t[i]  = sum_j dy_t[j] ( S_{t-1}[i][j] + u[i] k_t[i] v_t[j] )
 *     dk_t[i]  = r_t[i] u[i] sum_j dy_t[j] v_t[j]  +  sum_j G_t[i][j] v_t[j]
 *     dv_t[j]  = ( sum_i r_t[i] u[i] k_t[i] ) dy_t[j]  +  sum_i G_t[i][j] k_t[i]
 *     du[i]   += r_t[i] k_t[i] sum_j dy_t[j] v_t[j]                       (summed over t and over the batch)
 *     dw_t[i]  = sum_j G_t[i][j] S_{t-1}[i][j],     dx_t[i] = dw_t[i] * ( - w_t[i] exp(x_t[i]) )     (w = exp(-exp(x)))
 *     dS_0     = G_0.
 * The forward states S_0 .. S_{T-1} are recomputed first and kept (T N^2 doubles per unit): slow and plain.
 * Pinned in tests/test_oracle_pins_bwd.py by central finite differences of the forward oracle.
 * Layouts as in the forward pass; du is [B][H][N] per batch entry (the caller sums over b), all outputs double.
 */
static void unit_backward(const float *r, const float *k, const float *v, const float *x, const float *u,
                          const float *s_in, const double *dy, const double *ds_T, double *dr, double *dk,
                          double *dv, double *dx, double *du, double *ds_0, long T, long N, long row_stride)
{
    const size_t NN = (size_t)N * N;
    double *S_all = (double *)malloc((size_t)(T > 0 ? T : 1) * NN * sizeof(double));   /* S_{t-1} for t = 1..T */
    double *S = (double *)malloc(NN * sizeof(double));
    double *G = (double *)malloc(NN * sizeof(double));
    for (size_t i = 0; i < NN; ++i) S[i] = s_in ? (double)s_in[i] : 0.0;
    for (long t = 0; t < T; ++t) {
        memcpy(S_all + (size_t)t * NN, S, NN * sizeof(double));
        for (long i = 0; i < N; ++i) {
            const double w = exp(-exp((double)x[t * row_stride + i]));
            for (long j = 0; j < N; ++j)
                S[i * N + j] = w * S[i * N + j] + (double)k[t * row_stride + i] * (double)v[t * row_stride + j];
        }
    }
    for (size_t i = 0; i < NN; ++i) G[i] = ds_T ? ds_T[i] : 0.0;
    for (long i = 0; i < N; ++i) du[i] = 0.0;
    for (long t = T - 1; t >= 0; --t) {
        const float *rt = r + t * row_stride, *kt = k + t * row_stride, *vt = v + t * row_stride, *xt = x + t * row_stride;
        const double *dyt = dy + t * row_stride, *Sp = S_all + (size_t)t * NN;
        double dyv = 0.0, ruk = 0.0;
        for (long j = 0; j < N; ++j) dyv += dyt[j] * (double)vt[j];
        for (long i = 0; i < N; ++i) ruk += (double)rt[i] * (double)u[i] * (double)kt[i];
        for (long i = 0; i < N; ++i) {
            double a_r = 0.0, a_k = 0.0, a_w = 0.0;
            for (long j = 0; j < N; ++j) {
                a_r += dyt[j] * (Sp[i * N + j] + (double)u[i] * (double)kt[i] * (double)vt[j]);
                a_k += G[i * N + j] * (double)vt[j];
                a_w += G[i * N + j] * Sp[i * N + j];
            }
            const double w = exp(-exp((double)xt[i]));
            dr[t * row_stride + i] = a_r;
            dk[t * row_stride + i] = (double)rt[i] * (double)u[i] * dyv + a_k;
            dx[t * row_stride + i] = a_w * (-w * exp((double)xt[i]));
            du[i] += (double)rt[i] * (double)kt[i] * dyv;
        }
        for (long j = 0; j < N; ++j) {
            double a_v = 0.0;
            for (long i = 0; i < N; ++i) a_v += G[i * N + j] * (double)kt[i];
            dv[t * row_stride + j] = ruk * dyt[j] + a_v;
        }
        for (long i = 0; i < N; ++i) {
            const double w = exp(-exp((double)xt[i]));
            for (long j = 0; j < N; ++j) G[i * N + j] = w * G[i * N + j] + (double)rt[i] * dyt[j];
        }
    }
    if (ds_0) memcpy(ds_0, G, NN * sizeof(double));
    free(S_all);
    free(S);
    free(G);
}

/* Dense batch: r,k,v,x [B][T][H][N] float carriers, dy [B][T][H][N] double, ds_T [B][H][N][N] double or NULL
 * (zero); outputs dr,dk,dv,dx [B][T][H][N], du_b [B][H][N] (per batch entry), ds_0 [B][H][N][N] or NULL. */
void wkv6_oracle_backward(const float *r, const float *k, const float *v, const float *x, const float *u,
                          const float *state_in, const double *dy, const double *ds_T, double *dr, double *dk,
                          double *dv, double *dx, double *du_b, double *ds_0, long B, long T, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long b = 0; b < B; ++b)
        for (long h = 0; h < H; ++h) {
            const size_t off = (size_t)b * T * C + (size_t)h * N;
            const size_t soff = ((size_t)b * H + h) * N * N;
            unit_backward(r + off, k + off, v + off, x + off, u + h * N, state_in ? state_in + soff : NULL,
                          dy + off, ds_T ? ds_T + soff : NULL, dr + off, dk + off, dv + off, dx + off,
                          du_b + ((size_t)b * H + h) * N, ds_0 ? ds_0 + soff : NULL, T, N, C);
        }
}

/* ---------------------------------------------------------------------------------------------------
 * Gradient of the Finch-C2 form (unit_recurrence_c2 above: keys k' = k (1 - w), no bonus, second-value
 * vector added to the output), the layer the paper trains.  With G_t = dL/dS_t carried from t = T down
 * (G_T given), every input's gradient is read off the forward formulas
 *     y_t[j] = sum_i r_t[i] S_{t-1}[i][j] + u2_t[j],   S_t[i][j] = w_t[i] S_{t-1}[i][j] + k_t[i] (1 - w_t[i]) v_t[j]:
 *     dr_t[i]  = sum_j dy_t[j] S_{t-1}[i][j]
 *     dkp_t[i] = sum_j G_t[i][j] v_t[j]                      (gradient of the key that enters the state)
 *     dk_t[i]  = dkp_t[i] (1 - w_t[i])
 *     dv_t[j]  = sum_i G_t[i][j] k_t[i] (1 - w_t[i])
 *     dw_t[i]  = sum_j G_t[i][j] S_{t-1}[i][j] - dkp_t[i] k_t[i]        (w_t scales the old state and shrinks the key)
 *     dx_t[i]  = dw_t[i] * ( -w_t[i] exp(x_t[i]) )                       (w = exp(-exp(x)))
 *     du2_t    = dy_t                                                    (not returned: it is the argument)
 *     G_{t-1}[i][j] = w_t[i] G_t[i][j] + r_t[i] dy_t[j],   dS_0 = G_0.
 * Pins (tests/test_oracle_pins_bwd_c2.py): central differences of the pinned forward oracle of this form, the
 * reduction to the pinned gradient of the bonus-free recurrence on premultiplied keys plus the chain rule through
 * k (1 - w), the one-token closed form, linearity in (dy, dS_T), split-and-carry of the adjoint.
 */
static void unit_backward_c2(const float *r, const float *k, const float *v, const float *x, const float *s_in,
                             const double *dy, const double *ds_T, double *dr, double *dk, double *dv, double *dx,
                             double *ds_0, long T, long N, long row_stride)
{
    const size_t NN = (size_t)N * N;
    double *S_all = (double *)malloc((size_t)(T > 0 ? T : 1) * NN * sizeof(double));   /* S_{t-1} for t = 1..T */
    double *S = (double *)malloc(NN * sizeof(double));
    double *G = (double *)malloc(NN * sizeof(double));
    for (size_t i = 0; i < NN; ++i) S[i] = s_in ? (double)s_in[i] : 0.0;
    for (long t = 0; t < T; ++t) {
        memcpy(S_all + (size_t)t * NN, S, NN * sizeof(double));
        for (long i = 0; i < N; ++i) {
            const double w = exp(-exp((double)x[t * row_stride + i]));
            const double kp = (double)k[t * row_stride + i] * (1.0 - w);
            for (long j = 0; j < N; ++j) S[i * N + j] = w * S[i * N + j] + kp * (double)v[t * row_stride + j];
        }
    }
    for (size_t i = 0; i < NN; ++i) G[i] = ds_T ? ds_T[i] : 0.0;
    for (long t = T - 1; t >= 0; --t) {
        const float *rt = r + t * row_stride, *kt = k + t * row_stride, *vt = v + t * row_stride, *xt = x + t * row_stride;
        const double *dyt = dy + t * row_stride, *Sp = S_all + (size_t)t * NN;
        for (long i = 0; i < N; ++i) {
            double a_r = 0.0, a_kp = 0.0, a_gs = 0.0;
            for (long j = 0; j < N; ++j) {
                a_r += dyt[j] * Sp[i * N + j];
                a_kp += G[i * N + j] * (double)vt[j];
                a_gs += G[i * N + j] * Sp[i * N + j];
            }
            const double ex = exp((double)xt[i]), w = exp(-ex);
            dr[t * row_stride + i] = a_r;
            dk[t * row_stride + i] = a_kp * (1.0 - w);
            dx[t * row_stride + i] = (a_gs - a_kp * (double)kt[i]) * (-w * ex);
        }
        for (long j = 0; j < N; ++j) {
            double a_v = 0.0;
            for (long i = 0; i < N; ++i) {
                const double w = exp(-exp((double)xt[i]));
                a_v += G[i * N + j] * (double)kt[i] * (1.0 - w);
            }
            dv[t * row_stride + j] = a_v;
        }
        for (long i = 0; i < N; ++i) {
            const double w = exp(-exp((double)xt[i]));
            for (long j = 0; j < N; ++j) G[i * N + j] = w * G[i * N + j] + (double)rt[i] * dyt[j];
        }
    }
    if (ds_0) memcpy(ds_0, G, NN * sizeof(double));
    free(S_all);
    free(S);
    free(G);
}

/* Dense batch, layouts as wkv6_oracle_backward (no bonus, so no du). */
void wkv6_oracle_backward_c2(const float *r, const float *k, const float *v, const float *x, const float *state_in,
                             const double *dy, const double *ds_T, double *dr, double *dk, double *dv, double *dx,
                             double *ds_0, long B, long T, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long b = 0; b < B; ++b)
        for (long h = 0; h < H; ++h) {
            const size_t off = (size_t)b * T * C + (size_t)h * N;
            const size_t soff = ((size_t)b * H + h) * N * N;
            unit_backward_c2(r + off, k + off, v + off, x + off, state_in ? state_in + soff : NULL, dy + off,
                             ds_T ? ds_T + soff : NULL, dr + off, dk + off, dv + off, dx + off,
                             ds_0 ? ds_0 + soff : NULL, T, N, C);
        }
}

/* Packed variable-length batches of the two gradients: rows cu_seqlens[s] .. cu_seqlens[s+1]-1 of the
 * [total_T][H][N] tensors form sequence s (wkv6_oracle_prefill_varlen's layout), states and their gradients
 * are [S][H][N][N], du_s is [S][H][N] (per sequence; the caller sums over s).  Every (sequence, head) unit is
 * the dense unit gradient on its own rows: the recurrence never crosses a sequence boundary, so neither does
 * its adjoint.  A sequence without tokens hands its incoming state gradient through (dS_0 = dS_T).
 * Pinned in tests/test_oracle_pins_bwd_varlen.py. */
void wkv6_oracle_backward_varlen(const float *r, const float *k, const float *v, const float *x, const float *u,
                                 const float *state_in, const double *dy, const double *ds_T, double *dr, double *dk,
                                 double *dv, double *dx, double *du_s, double *ds_0, const int32_t *cu_seqlens,
                                 long S, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long s = 0; s < S; ++s)
        for (long h = 0; h < H; ++h) {
            const long t0 = cu_seqlens[s], len = cu_seqlens[s + 1] - cu_seqlens[s];
            const size_t off = (size_t)t0 * C + (size_t)h * N;
            const size_t soff = ((size_t)s * H + h) * N * N;
            unit_backward(r + off, k + off, v + off, x + off, u + h * N, state_in ? state_in + soff : NULL,
                          dy + off, ds_T ? ds_T + soff : NULL, dr + off, dk + off, dv + off, dx + off,
                          du_s + ((size_t)s * H + h) * N, ds_0 ? ds_0 + soff : NULL, len, N, C);
        }
}

void wkv6_oracle_backward_c2_varlen(const float *r, const float *k, const float *v, const float *x,
                                    const float *state_in, const double *dy, const double *ds_T, double *dr,
                                    double *dk, double *dv, double *dx, double *ds_0, const int32_t *cu_seqlens,
                                    long S, long H, long N)
{
    const long C = H * N;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (long s = 0; s < S; ++s)
        for (long h = 0; h < H; ++h) {
            const long t0 = cu_seqlens[s], len = cu_seqlens[s + 1] - cu_seqlens[s];
            const size_t off = (size_t)t0 * C + (size_t)h * N;
            const size_t soff = ((size_t)s * H + h) * N * N;
            unit_backward_c2(r + off, k + off, v + off, x + off, state_in ? state_in + soff : NULL, dy + off,
                             ds_T ? ds_T + soff : NULL, dr + off, dk + off, dv + off, dx + off,
                             ds_0 ? ds_0 + soff : NULL, len, N, C);
        }
}
