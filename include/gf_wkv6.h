/*
 * gf_wkv6 -- WKV-6 (Finch / RWKV-6) time-mix recurrence for GoldFinch-style linear
 * pre-fill on NVIDIA B200 (sm_100a).  Plain C ABI: pointers and sizes only.
 *
 * What is computed (per sequence b and head h independently; the Finch-C2 time-mixing
 * formulae are stated per head).  With N the head size, S an N x N fp32 state whose
 * row index i is the key channel and column index j the value channel:
 *
 *     w_t       = exp(-exp(x_t))                                (Finch-C2 decay equation)
 *     y_t[j]    = sum_i r_t[i] * ( S_{t-1}[i][j] + u[i] * k_t[i] * v_t[j] )
 *     S_t[i][j] = w_t[i] * S_{t-1}[i][j] + k_t[i] * v_t[j]
 *
 * S_{t-1} is the paper's wkv_t = sum_{i<t} diag(prod_{j=i+1..t-1} w_j) k_i^T v_i and
 * r_t . wkv_t its per-head output before LayerNorm (Finch-C2 wkv_t / o_t equations);
 * the diag(u) term is classic Finch's "bonus" (pass u = 0 for the Finch-C2 form).
 * x is the decay *logit* d_t, not w and not log w.  k arrives final (any k*(1-w)
 * factor is the caller's).  The output uses the state before the update.
 *
 * Conventions common to every compute call
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, unless the
 *     function name ends in _host.  The library never allocates, frees or keeps
 *     user memory; compute calls only enqueue work on `stream` and return without
 *     synchronising the host.
 *   - Layout: r,k,v,x,y are [B][T][H][N] contiguous with N fastest (packed calls:
 *     [total_T][H][N]); u is [H][N] fp32; states are [B][H][N][N] fp32 row-major
 *     ([i][j], i = key channel).  Base pointers must be 16-byte aligned.
 *   - dtype of r,k,v,x,y: bf16 for the un-suffixed names, fp32 for the _f32 twins.
 *     u and the states are always fp32.  All accumulation is fp32.
 *   - state_in == NULL means a zero initial state.  state_out == NULL skips the
 *     final-state write.  state_out may alias state_in (in-place update).  y must
 *     not overlap any input.
 *   - N must be 64 (GF_ERR_UNSUPPORTED otherwise).  B, T, S or a sequence length of
 *     zero is legal: no y rows are written for it and its state passes through.
 *   - x may be any finite value or -inf (w = 1); +inf gives w = 0.  NaN inputs give
 *     NaN outputs.
 *   - Errors: argument errors are detected on the host before anything is enqueued
 *     and returned at once; a failed launch returns GF_ERR_CUDA.  No exception
 *     crosses this boundary.  Results are run-to-run deterministic.
 */
#ifndef GF_WKV6_H
#define GF_WKV6_H

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define GF_API __attribute__((visibility("default")))
#else
#define GF_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GF_OK = 0,
    GF_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, negative size, bad cu_seqlens bound */
    GF_ERR_UNSUPPORTED = 2, /* head size other than 64, unknown kernel selector */
    GF_ERR_CUDA = 3,        /* a CUDA runtime / driver call failed */
    GF_ERR_WORKSPACE = 4,   /* caller-supplied workspace too small */
    GF_ERR_TIMEOUT = 5      /* a bounded device-side wait gave up (see gf_wkv6_last_device_status) */
} gf_status_t;

/* A CUDA stream handle (cudaStream_t); NULL is the legacy default stream. */
typedef struct CUstream_st *gf_stream_t;

/* Kernel selector for the bf16 prefill entry points. */
typedef enum {
    GF_KERNEL_AUTO = 0,    /* chunked tensor-core kernel, exact kernel where it does not apply */
    GF_KERNEL_EXACT = 1,   /* token-by-token fp32 recurrence on the ALUs */
    GF_KERNEL_CHUNKED = 2  /* chunked tensor-core formulation */
} gf_kernel_t;

/* Dense prefill, bf16 r,k,v,x,y.  Runs the recurrence above over t = 1..T for every
 * (b,h) (the linear-time pre-fill of the Finch-C2 layers: wkv_t / o_t equations) and
 * writes y [B][T][H][N] and, if state_out != NULL, S_T [B][H][N][N]. */
GF_API gf_status_t gf_wkv6_prefill(const void *r, const void *k, const void *v, const void *x,
                            const float *u, const float *state_in, float *state_out, void *y,
                            int B, int T, int H, int N, gf_stream_t stream);

/* Dense prefill in the Finch-C2 form, bf16 r,k,v,x,u2,y: the paper's Finch-C2 block as written.  k is the
 * projected key BEFORE the block's "(1 - w_t)" factor; the call applies it (k'_t = k_t (1 - w_t), the k_t
 * equation), uses no bonus, and adds the token's second-value vector to the per-head output (the o_t
 * equation before LayerNorm and W^O):
 *     y_t = r_t . wkv_t + u2_t,     wkv_t = S_{t-1},     S_t = diag(w_t) S_{t-1} + k'_t^T v_t.
 * u2 is [B][T][H][N] bf16 (the block's u'_t), or NULL for no added vector.  Everything else (layouts,
 * states, sequence split with the registered workspace, error behaviour) is as for gf_wkv6_prefill.  The
 * factor is formed from the key scales the kernel already has (2^{-a_t} - 2^{-a_{t-1}}), which costs no
 * extra exponential; its relative error is about 2^-22 / (1 - w_t), i.e. below bf16 rounding for
 * w_t <= 0.9999. */
GF_API gf_status_t gf_wkv6_prefill_c2(const void *r, const void *k, const void *v, const void *x,
                               const void *u2, const float *state_in, float *state_out, void *y,
                               int B, int T, int H, int N, gf_stream_t stream);

/* The Finch-C2 form of the packed variable-length prefill and of the decode step (bf16): arguments as for
 * gf_wkv6_prefill_varlen / gf_wkv6_step with u2 (packed [total_T][H][N], resp. [B][H][N], bf16, or NULL) in
 * place of u; semantics as for gf_wkv6_prefill_c2 (the k_t and o_t equations of the Finch-C2 block). */
GF_API gf_status_t gf_wkv6_prefill_varlen_c2(const void *r, const void *k, const void *v, const void *x,
                                      const void *u2, const float *state_in, float *state_out, void *y,
                                      const int32_t *cu_seqlens, int S, int total_T, int max_seqlen,
                                      int H, int N, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_step_c2(const void *r, const void *k, const void *v, const void *x, const void *u2,
                            const float *state_in, float *state_out, void *y, int B, int H, int N,
                            gf_stream_t stream);

/* Same with fp32 r,k,v,x,y (token-by-token fp32 recurrence). */
GF_API gf_status_t gf_wkv6_prefill_f32(const float *r, const float *k, const float *v, const float *x,
                                const float *u, const float *state_in, float *state_out, float *y,
                                int B, int T, int H, int N, gf_stream_t stream);

/* Gradient of gf_wkv6_prefill_f32 (training; the paper trains its models with this recurrence and fine-tunes
 * long contexts through it): the adjoint of the wkv_t sum and of the output r_t . wkv_t (Finch-C2 wkv_t / o_t
 * equations) with the bonus term of the recurrence at the top of this file.  Given dy = dL/dy [B][T][H][N] and
 * dstate_out = dL/dS_T [B][H][N][N] (NULL: zero), with G_t = dL/dS_t carried from t = T down,
 *     G_{t-1}[i][j] = w_t[i] G_t[i][j] + r_t[i] dy_t[j],
 * it writes
 *     dr_t[i] = sum_j dy_t[j] ( S_{t-1}[i][j] + u[i] k_t[i] v_t[j] )
 *     dk_t[i] = sum_j G_t[i][j] v_t[j] + r_t[i] u[i] (v_t . dy_t)
 *     dv_t[j] = sum_i G_t[i][j] k_t[i] + ( sum_i r_t[i] u[i] k_t[i] ) dy_t[j]
 *     dx_t[i] = ( sum_j G_t[i][j] S_{t-1}[i][j] ) * ( -w_t[i] exp(x_t[i]) )        (gradient w.r.t. the decay logit)
 *     du[i]   = sum over b and t of r_t[i] k_t[i] (v_t . dy_t)                     ([H][N], summed over the batch)
 *     dstate_in = G_0                                                              ([B][H][N][N]; NULL: not written)
 * All tensors fp32, layouts as in the forward call; r,k,v,x,u,state_in are the forward call's inputs (state_in
 * NULL: zero).  dr,dk,dv,dx must not alias r,k,v,x,dy.  Token by token on the ALUs; the states the gradients need are
 * recomputed from checkpoints kept every 64 tokens in `workspace`, a caller-owned DEVICE buffer of at least
 * gf_wkv6_backward_workspace_bytes(B,T,H,N) bytes, 16-byte aligned (GF_ERR_WORKSPACE if absent or too small).
 * Enqueues two kernels on `stream`, allocates nothing, does not synchronise; deterministic (no atomics). */
GF_API gf_status_t gf_wkv6_backward_f32(const float *r, const float *k, const float *v, const float *x,
                                 const float *u, const float *state_in, const float *dy,
                                 const float *dstate_out, float *dr, float *dk, float *dv, float *dx,
                                 float *du, float *dstate_in, int B, int T, int H, int N,
                                 void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API size_t gf_wkv6_backward_workspace_bytes(int B, int T, int H, int N);

/* The same gradient for bf16 tensors (the gradient of gf_wkv6_prefill): r,k,v,x,dy and dr,dk,dv,dx are
 * [B][T][H][N] bf16, u, du, state_in, dstate_out, dstate_in fp32 as above; every formula above holds, with the
 * results rounded to bf16 once at the end.  Chunked on the tensor cores: the sequence is walked backwards in chunks
 * of 64 tokens with the state adjoint G carried in fp32, nine 64x64x64 bf16 products (fp32 accumulate) per chunk
 * give the in-chunk parts of dr, dk, dv and of G, and the decay-logit gradient comes from suffix sums of
 * r*dr - k*dk over the chunk plus rowsum(G * S) at the chunk's end; the chunk-start states come from a state-only
 * checkpoint pass of the forward kernel.  A chunk in which some channel decays by more than 2^-96 is processed token
 * by token in fp32 instead, so any decay logit is accepted (x = +inf leaves dx undefined, as in the formula).
 * `workspace`: caller-owned DEVICE buffer of at least gf_wkv6_backward_bf16_workspace_bytes(B,T,H,N) bytes, 16-byte
 * aligned (one 64x64 bf16 state per chunk and unit, plus 2 MiB per SM for the token-by-token path);
 * GF_ERR_WORKSPACE if absent or too small.  GF_ERR_UNSUPPORTED for B*T >= 2^31 - 64 rows or N != 64.  dstate_in must
 * not be dstate_out (GF_ERR_INVALID_ARG).  Enqueues three
 * kernels on `stream` (five when B*H is less than half the SMs: the sequences are then cut into segments that run
 * side by side, as in the forward call), allocates nothing, does not synchronise; deterministic (no atomics).  A
 * device-side wait that runs out is reported by gf_wkv6_last_device_status as for the forward call. */
GF_API gf_status_t gf_wkv6_backward(const void *r, const void *k, const void *v, const void *x, const float *u,
                             const float *state_in, const void *dy, const float *dstate_out, void *dr,
                             void *dk, void *dv, void *dx, float *du, float *dstate_in, int B, int T, int H,
                             int N, void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API size_t gf_wkv6_backward_bf16_workspace_bytes(int B, int T, int H, int N);

/* Gradient of gf_wkv6_prefill_c2, the Finch-C2 form the paper trains (Finch-C2 block: k_t equation with the factor
 * (1 - w_t), o_t equation without the bonus): the same adjoint recursion with
 *     dr_t[i] = sum_j dy_t[j] S_{t-1}[i][j]            dkp_t[i] = sum_j G_t[i][j] v_t[j]       dk_t = dkp_t (1 - w_t)
 *     dv_t[j] = sum_i G_t[i][j] k_t[i] (1 - w_t[i])
 *     dx_t[i] = ( sum_j G_t[i][j] S_{t-1}[i][j] - dkp_t[i] k_t[i] ) * ( -w_t[i] exp(x_t[i]) )
 * (the decay logit also reaches the loss through the key factor).  The second-value vector u2 only adds to the
 * output: its gradient is dy itself, so neither appears here.  k is the key BEFORE the (1 - w) factor, as in the
 * forward call.  Everything else (dtypes, layouts, workspace, statuses, launches but for the bonus sum) as
 * gf_wkv6_backward. */
GF_API gf_status_t gf_wkv6_backward_c2(const void *r, const void *k, const void *v, const void *x,
                                const float *state_in, const void *dy, const float *dstate_out, void *dr,
                                void *dk, void *dv, void *dx, float *dstate_in, int B, int T, int H, int N,
                                void *workspace, size_t workspace_bytes, gf_stream_t stream);

/* A training step's pair.  gf_wkv6_prefill_train / gf_wkv6_prefill_c2_train are gf_wkv6_prefill / gf_wkv6_prefill_c2
 * (same results, dense; calls with few units split their sequences as usual) that also leave the state before every chunk of 64
 * tokens and after the last one at the start of `workspace`, the gradient's workspace
 * (gf_wkv6_backward_bf16_workspace_bytes(B,T,H,N) bytes).  gf_wkv6_backward_saved / gf_wkv6_backward_c2_saved are
 * gf_wkv6_backward / gf_wkv6_backward_c2 without their first launch: they take those states from the workspace, which
 * must still hold what the forward call of the SAME r,k,v,x,state_in wrote (the caller's responsibility; nothing
 * checks it). */
GF_API gf_status_t gf_wkv6_prefill_train(const void *r, const void *k, const void *v, const void *x, const float *u,
                                  const float *state_in, float *state_out, void *y, int B, int T, int H, int N,
                                  void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_prefill_c2_train(const void *r, const void *k, const void *v, const void *x,
                                     const void *u2, const float *state_in, float *state_out, void *y, int B,
                                     int T, int H, int N, void *workspace, size_t workspace_bytes,
                                     gf_stream_t stream);
GF_API gf_status_t gf_wkv6_backward_saved(const void *r, const void *k, const void *v, const void *x, const float *u,
                                   const float *state_in, const void *dy, const float *dstate_out, void *dr,
                                   void *dk, void *dv, void *dx, float *du, float *dstate_in, int B, int T,
                                   int H, int N, void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_backward_c2_saved(const void *r, const void *k, const void *v, const void *x,
                                      const float *state_in, const void *dy, const float *dstate_out, void *dr,
                                      void *dk, void *dv, void *dx, float *dstate_in, int B, int T, int H,
                                      int N, void *workspace, size_t workspace_bytes, gf_stream_t stream);

/* Gradients of the packed variable-length prefill (gf_wkv6_prefill_varlen / gf_wkv6_prefill_varlen_c2; bf16 tensors,
 * fp32 states): the adjoint recursion of gf_wkv6_backward / gf_wkv6_backward_c2 run per (sequence, head) over the
 * sequence's own rows (the wkv_t recurrence never crosses a sequence boundary, so neither does its adjoint).  r, k, v,
 * x, dy and the four gradients are packed [total_T][H][N] bf16; cu_seqlens is a DEVICE int32 array of S+1
 * non-decreasing entries with cu_seqlens[0] = 0 and cu_seqlens[S] = total_T (not read on the host); max_seqlen an
 * upper bound on any sequence length; state_in / dstate_out (NULL: zero) and dstate_in (NULL: not written) are
 * [S][H][N][N] fp32; du [H][N] fp32 is summed over the sequences in index order.  A sequence without tokens hands its
 * state gradient through.  `workspace`: caller-owned DEVICE buffer of at least
 * gf_wkv6_backward_varlen_workspace_bytes(S,total_T,H,N) bytes, 16-byte aligned (H * (total_T / 64 + 2 S) states of
 * 64x64 bf16, plus 2 MiB per SM, plus the segment summaries of the widest split when S*H is less than half the SMs);
 * GF_ERR_WORKSPACE if absent or too small.  One CTA per (sequence, head), the longest sequences first; with S*H less
 * than half the SMs every sequence is cut into segments by max_seqlen, as in the dense call (segments past a shorter
 * sequence's end do no work): four kernels on `stream` (three for the Finch-C2 form), six resp. five when split, nothing allocated, no synchronisation, deterministic.
 * Other statuses as gf_wkv6_backward (dstate_in must not be dstate_out; total_T >= 2^31 - 64 or N != 64 unsupported). */
GF_API gf_status_t gf_wkv6_backward_varlen(const void *r, const void *k, const void *v, const void *x, const float *u,
                                    const float *state_in, const void *dy, const float *dstate_out, void *dr,
                                    void *dk, void *dv, void *dx, float *du, float *dstate_in,
                                    const int32_t *cu_seqlens, int S, int total_T, int max_seqlen, int H, int N,
                                    void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_backward_varlen_c2(const void *r, const void *k, const void *v, const void *x,
                                       const float *state_in, const void *dy, const float *dstate_out, void *dr,
                                       void *dk, void *dv, void *dx, float *dstate_in, const int32_t *cu_seqlens,
                                       int S, int total_T, int max_seqlen, int H, int N, void *workspace,
                                       size_t workspace_bytes, gf_stream_t stream);
GF_API size_t gf_wkv6_backward_varlen_workspace_bytes(int S, int total_T, int H, int N);

/* The training pair for packed sequences, as gf_wkv6_prefill_train / gf_wkv6_backward_saved for dense ones:
 * gf_wkv6_prefill_varlen_train / gf_wkv6_prefill_varlen_c2_train are gf_wkv6_prefill_varlen / gf_wkv6_prefill_varlen_c2
 * (same results; one CTA per sequence and head, never split and never persistent) that also leave the state before every
 * chunk of 64 tokens of every sequence, and after its last token, in `workspace`, the packed gradient's workspace
 * (gf_wkv6_backward_varlen_workspace_bytes(S,total_T,H,N) bytes); gf_wkv6_backward_varlen_saved /
 * gf_wkv6_backward_varlen_c2_saved are the packed gradient calls without their checkpoint launch.  The workspace must
 * still hold what the forward call of the SAME r,k,v,x,state_in,cu_seqlens wrote (nothing checks it). */
GF_API gf_status_t gf_wkv6_prefill_varlen_train(const void *r, const void *k, const void *v, const void *x,
                                         const float *u, const float *state_in, float *state_out, void *y,
                                         const int32_t *cu_seqlens, int S, int total_T, int max_seqlen, int H,
                                         int N, void *workspace, size_t workspace_bytes, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_prefill_varlen_c2_train(const void *r, const void *k, const void *v, const void *x,
                                            const void *u2, const float *state_in, float *state_out, void *y,
                                            const int32_t *cu_seqlens, int S, int total_T, int max_seqlen,
                                            int H, int N, void *workspace, size_t workspace_bytes,
                                            gf_stream_t stream);
GF_API gf_status_t gf_wkv6_backward_varlen_saved(const void *r, const void *k, const void *v, const void *x,
                                          const float *u, const float *state_in, const void *dy,
                                          const float *dstate_out, void *dr, void *dk, void *dv, void *dx,
                                          float *du, float *dstate_in, const int32_t *cu_seqlens, int S,
                                          int total_T, int max_seqlen, int H, int N, void *workspace,
                                          size_t workspace_bytes, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_backward_varlen_c2_saved(const void *r, const void *k, const void *v, const void *x,
                                             const float *state_in, const void *dy, const float *dstate_out,
                                             void *dr, void *dk, void *dv, void *dx, float *dstate_in,
                                             const int32_t *cu_seqlens, int S, int total_T, int max_seqlen,
                                             int H, int N, void *workspace, size_t workspace_bytes,
                                             gf_stream_t stream);

/* Packed variable-length prefill (batched serving).  Sequence s occupies rows
 * cu_seqlens[s] .. cu_seqlens[s+1]-1 of the [total_T][H][N] tensors; chunking restarts
 * at every sequence start, so a sequence never sees another's tokens.  cu_seqlens is a
 * DEVICE int32 array of S+1 non-decreasing entries with cu_seqlens[0] = 0 and
 * cu_seqlens[S] = total_T (the caller guarantees this; it is not read on the host).
 * max_seqlen is an upper bound on any sequence length.  States are [S][H][N][N].
 * A bf16 call with few (sequence, head) units takes the sequence split described at
 * gf_wkv6_set_workspace, cut by max_seqlen: gf_wkv6_workspace_bytes(S, max_seqlen, H, N) is the
 * scratch it uses, and segments that lie past a sequence's end do no work. */
GF_API gf_status_t gf_wkv6_prefill_varlen(const void *r, const void *k, const void *v, const void *x,
                                   const float *u, const float *state_in, float *state_out,
                                   void *y, const int32_t *cu_seqlens, int S, int total_T,
                                   int max_seqlen, int H, int N, gf_stream_t stream);

GF_API gf_status_t gf_wkv6_prefill_varlen_f32(const float *r, const float *k, const float *v,
                                       const float *x, const float *u, const float *state_in,
                                       float *state_out, float *y, const int32_t *cu_seqlens,
                                       int S, int total_T, int max_seqlen, int H, int N,
                                       gf_stream_t stream);

/* Single-token decode step (new-token generation with the state pre-fill left behind):
 * identical to a prefill with T = 1.  r,k,v,x,y are [B][H][N]; states [B][H][N][N]. */
GF_API gf_status_t gf_wkv6_step(const void *r, const void *k, const void *v, const void *x,
                         const float *u, const float *state_in, float *state_out, void *y,
                         int B, int H, int N, gf_stream_t stream);

GF_API gf_status_t gf_wkv6_step_f32(const float *r, const float *k, const float *v, const float *x,
                             const float *u, const float *state_in, float *state_out, float *y,
                             int B, int H, int N, gf_stream_t stream);

/* End-to-end dense prefill from HOST buffers (bf16 r,k,v,x,y; fp32 u and states, all in
 * host memory, pinned for full copy speed).  Copies the inputs to `dev_ws`, runs
 * gf_wkv6_prefill there and copies y and state_out back, all on `stream`; returns
 * without synchronising, so the caller synchronises `stream` before reading y.
 * dev_ws is a caller-owned DEVICE buffer of at least gf_wkv6_host_workspace_bytes()
 * bytes, 256-byte aligned (GF_ERR_WORKSPACE if dev_ws_bytes is too small). */
GF_API gf_status_t gf_wkv6_prefill_host(const void *r, const void *k, const void *v, const void *x,
                                 const float *u, const float *state_in, float *state_out, void *y,
                                 int B, int T, int H, int N, void *dev_ws, size_t dev_ws_bytes,
                                 gf_stream_t stream);
GF_API size_t gf_wkv6_host_workspace_bytes(int B, int T, int H, int N);

/* Optional scratch for bf16 prefill calls (dense or packed) with few (sequence, head) units.  One CTA walks one
 * unit's sequence, so a call with fewer units than half the GPU's SMs (long-context prefill of one
 * sequence) would leave most SMs idle.  With a workspace registered such a call cuts every sequence
 * into up to 8 segments: a first launch carries the state over each segment from a zero start and
 * leaves per segment its decay product and state increment (the pair (D, dS) of the recurrence
 * S <- diag(D) S + dS, which composes associatively across segments of the wkv_t sum) in the workspace,
 * the second launch folds them into each segment's start state and computes y.  Results agree with the
 * unsplit call to rounding.  Calls with MORE units than SMs run one CTA per SM that walks a stream of units
 * (a unit's pipeline fill overlaps the drain of the one before); a packed call of that kind draws its units,
 * longest sequences first, from a counter in the workspace (a small kernel of the call itself, on `stream`,
 * zeroes the counter and ranks the sequences there) and falls back to one CTA per unit without a workspace; a
 * dense one needs none.  gf_wkv6_workspace_bytes returns what gf_wkv6_prefill(B,T,H,N) (packed: B = S,
 * T = max_seqlen) would use on the current device: the summaries and start-state copies of a split, 64 + 4*S
 * bytes (rounded up to 256) for more units than SMs, else 0.  gf_wkv6_set_workspace registers a caller-owned
 * DEVICE buffer (256-byte aligned; NULL unregisters) for all later calls of this process; the library
 * never frees it.  With a registered buffer that is too small the call splits into as many segments as fit
 * (or runs unsplit).  A split call with a start state keeps a copy of it in the workspace and reads only the
 * copy once its second launch runs, so state_out may be state_in there too.  Calls that use the workspace
 * and overlap on the GPU (different streams) race on it. */
GF_API size_t gf_wkv6_workspace_bytes(int B, int T, int H, int N);
GF_API gf_status_t gf_wkv6_set_workspace(void *dev_ptr, size_t bytes);
/* The split a bf16 prefill call of B*H units and T tokens (packed: S, max_seqlen) takes on a GPU of n_sm SMs with at
 * most scratch_cap bytes of scratch (0: unlimited): *nseg segments per sequence (1: no split) of *seg_chunks 64-token
 * chunks (the last takes the rest) and *scratch_bytes of scratch: per unit one 16 640-byte summary for every segment
 * but the last and a 16 384-byte copy of the start state.  Host arithmetic only (no device is touched): what
 * gf_wkv6_workspace_bytes and gf_wkv6_prefill_static decide with, exposed for planning and for tests. */
GF_API gf_status_t gf_wkv6_split_plan(int B, int T, int H, int N, int n_sm, size_t scratch_cap, int *nseg,
                               int *seg_chunks, size_t *scratch_bytes);

/* Dense bf16 prefill for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this is a packaging variant of gf_wkv6_prefill.)  Some hosts of this library own no allocator at the
 * point of the call: a plug-in inside an inference server whose device memory is planned and handed out
 * up front, or a latency-critical loop that must never reach cudaMalloc and the device-wide
 * synchronisation it implies.  Such a caller could not supply the workspace that the sequence split of
 * gf_wkv6_prefill wants for calls with few (sequence, head) units, and would run those calls at a
 * fraction of the GPU.  This entry point takes the split with scratch that is built into the library: a
 * fixed array of GF_WKV6_STATIC_SCRATCH_BYTES in the library's device image (every GPU that loads the
 * library holds it until the process exits).  It allocates and frees nothing and ignores the registered
 * workspace; inputs, outputs, layouts and results are those of gf_wkv6_prefill.
 *   - Limit: the split takes the largest segment count (at most the one gf_wkv6_prefill would take) whose
 *     scratch -- per (sequence, head) unit one 16 640-byte summary for every segment but the last and a
 *     16 384-byte copy of the start state -- fits the array.  The size is that of 32 units cut four ways (one
 *     long sequence of 32 heads on a 148-SM GPU); up to 64 units fit with two segments.  A call that would
 *     split but does not fit even with two segments (65 to 74 units on 148 SMs) returns GF_ERR_WORKSPACE
 *     and enqueues nothing.  Calls that do not split (more units than half the SMs, or fewer than 16 chunks
 *     of 64 tokens) need no scratch and always pass.
 *   - It always runs the chunked tensor-core kernel: gf_wkv6_set_kernel is not consulted.
 *   - The first call on each device looks up the array's device address (with that device current), so
 *     make that first call before any stream capture begins on that device.
 *   - All calls share the one array and it keeps the previous call's contents.  Nothing in it has to be
 *     cleared: the first launch of a call writes every entry its second launch reads.  Calls that overlap
 *     on the GPU (different streams, or different host threads) race on it: serialise them. */
#define GF_WKV6_STATIC_SCRATCH_BYTES 2121728u      /* 32 units x (3 summaries of (64 + 64*64) floats + 64*64 floats) */
GF_API gf_status_t gf_wkv6_prefill_static(const void *r, const void *k, const void *v, const void *x,
                                   const float *u, const float *state_in, float *state_out, void *y,
                                   int B, int T, int H, int N, gf_stream_t stream);

/* Building blocks for splitting ONE sequence over several calls or several GPUs (sequence parallelism).
 * Over a run of tokens the recurrence acts on the state as the affine map S -> diag(D) S + dS, D the
 * product of the run's decays per key channel and dS the state the run reaches from zero (the wkv_t sum
 * restricted to the run); these maps compose in sequence order.
 * gf_wkv6_sequence_summary writes that pair for every (b,h) of a dense bf16 [B][T][H][N] run:
 * summary is a DEVICE fp32 array [B][H][64 + 64*64], D first, then dS row-major ([i][j], i = key channel).
 * It reads k, v, x only (c2 != 0: keys are multiplied by one minus their decay, as in gf_wkv6_prefill_c2).
 * gf_wkv6_fold_summaries applies n_fold such summaries, laid out [n_fold][B][H][64 + 64*64] in sequence
 * order, to state_in (NULL: zero) and writes the resulting [B][H][N][N] state to state_out (may alias
 * state_in).  A rank that holds the p-th piece of a sequence gathers every rank's summary, folds the
 * first p of them over the sequence's initial state and runs gf_wkv6_prefill on its piece with that start
 * state; the last rank's state_out is the sequence's final state. */
GF_API gf_status_t gf_wkv6_sequence_summary(const void *k, const void *v, const void *x, float *summary,
                                     int B, int T, int H, int N, int c2, gf_stream_t stream);
GF_API gf_status_t gf_wkv6_fold_summaries(const float *state_in, const float *summaries, int n_fold,
                                   int B, int H, int N, float *state_out, gf_stream_t stream);

/* Forces the kernel used by the bf16 prefill calls of this process (default
 * GF_KERNEL_AUTO).  Process-wide, not thread-safe against concurrent compute calls. */
GF_API gf_status_t gf_wkv6_set_kernel(gf_kernel_t kernel);

/* Synchronises `stream`, then returns GF_ERR_TIMEOUT if any kernel launched by this
 * library since the last query gave up on a bounded wait (its outputs are then
 * undefined), GF_ERR_CUDA if the stream reports an error, else GF_OK.  Clears the flag. */
GF_API gf_status_t gf_wkv6_last_device_status(gf_stream_t stream);

/* Every device-side wait of the prefill kernels (on a copy, a tensor-core product, another warp) is bounded: when
 * it runs out the kernel raises the status flag that gf_wkv6_last_device_status reports and all its warps leave.
 * gf_wkv6_set_wait_limit sets the bound, in microseconds, for the launches of later calls of this process
 * (0 restores the default of 2 s; a healthy launch waits microseconds at a time, so the bound only matters when
 * something is wrong).
 * gf_wkv6_selftest_wait_timeout shows the mechanism at work without disturbing anything: it enqueues a one-warp
 * kernel that waits, with that same bounded wait, on a barrier nobody arrives on; after `microseconds` (1 .. 1 000 000)
 * the wait gives up, the flag is raised and the kernel ends, so the next gf_wkv6_last_device_status returns
 * GF_ERR_TIMEOUT once and GF_OK afterwards.  No other state of the library or the device is touched. */
GF_API gf_status_t gf_wkv6_set_wait_limit(unsigned int microseconds);
GF_API gf_status_t gf_wkv6_selftest_wait_timeout(unsigned int microseconds, gf_stream_t stream);

/* Number of kernels this library has launched in this process (for benchmarks). */
GF_API uint64_t gf_wkv6_launch_count(void);

GF_API const char *gf_status_string(gf_status_t status);
/* LayerNorm across all heads: the normalisation that follows the WKV output in the o_t equation of the
 * Finch-C2 block, o_t = LayerNorm(concat_h(r_t . wkv_t + u'_t)) W^O (the paper replaces Finch's per-head
 * GroupNorm by one LayerNorm over the D = H*N concatenated channels of a token).  For every row (token):
 *     mu = mean_c y[c],  var = mean_c (y[c] - mu)^2,  out[c] = (y[c] - mu) / sqrt(var + eps) * gamma[c] + beta[c].
 * The paper does not spell the operator out; eps inside the root and the per-channel affine pair are the
 * customary definition.  The output projection W^O is a plain GEMM and not part of this library.
 *   y, out    DEVICE [rows][H][N] (bf16, resp. fp32 for _f32), 16-byte aligned; out may be y (in place).
 *             Typically y is the output of a gf_wkv6_prefill* / gf_wkv6_step* call with rows = B*T tokens.
 *   gamma,beta DEVICE fp32 [H*N], or NULL for 1 resp. 0.     eps >= 0 (HOST value).
 * Arithmetic in fp32 (two passes: mean, then squared deviations), one rounding to the output type.
 * H*N must be a multiple of 8 and at most 8192 (GF_ERR_UNSUPPORTED otherwise); rows = 0 is a no-op.
 * Enqueues one kernel on `stream`, allocates nothing, does not synchronise. */
GF_API gf_status_t gf_c2_layernorm(const void *y, const float *gamma, const float *beta, float eps, void *out,
                            long long rows, int H, int N, gf_stream_t stream);
GF_API gf_status_t gf_c2_layernorm_f32(const float *y, const float *gamma, const float *beta, float eps,
                                float *out, long long rows, int H, int N, gf_stream_t stream);

/* The decay logit of the Finch-C2 block, the producer of the x argument of the prefill calls above:
 *     d_t = lora_omega( ddlerp_d( x_t, x_{t-1} ) )                                   (Finch-C2 block, d_t equation)
 * with the operators of the Finch-C2 section, lerp(a, b, t) = a + (b - a) t, lora(v) = lambda + tanh(v A) B and
 * ddlerp(a, b) = a + (b - a) lora( a + (b - a) mu_x ); the decay itself, w_t = exp(-exp(d_t)), is taken inside the
 * WKV kernels.  Written out: z = x_t + (x_{t-1} - x_t) mu_x; m = x_t + (x_{t-1} - x_t)(lambda_d + tanh(z A_d) B_d);
 * d_t = lambda_w + tanh(m A_w) B_w.
 *   x       DEVICE bf16 [B][T][D]   the block's input (D = heads * 64 channels of the model dimension)
 *   x_prev  DEVICE bf16 [B][D] or NULL: the token before each sequence's first one (NULL: zeros); x_{t-1} of any
 *           other token is the row above it
 *   mu_x, lambda_d, lambda_w   DEVICE fp32 [D]
 *   A_d [D][Rd], B_d [Rd][D]   DEVICE bf16 row-major: the lora inside ddlerp_d
 *   A_w [D][Rw], B_w [Rw][D]   DEVICE bf16 row-major: lora_omega
 *   d       DEVICE bf16 [B][T][D]   written; must not alias x
 * bf16 operands on the tensor cores with fp32 accumulation; z, m, the two tanh vectors and d are each rounded to
 * bf16 once; tanh is the hardware approximation (relative error about 2^-11).  D must be a multiple of 64; Rd and Rw
 * multiples of 16, at most 64 (GF_ERR_UNSUPPORTED otherwise; Finch uses 32 and 64); pointers 16-byte aligned.
 * Enqueues one kernel on `stream`, allocates nothing, does not synchronise. */
GF_API gf_status_t gf_c2_decay_logit(const void *x, const void *x_prev, const float *mu_x, const void *A_d,
                              const void *B_d, const float *lambda_d, const void *A_w, const void *B_w,
                              const float *lambda_w, void *d, int B, int T, int D, int Rd, int Rw,
                              gf_stream_t stream);

/* GOLD key compression, the product that ends linear pre-fill: c_t = x_t W^{KD} (GOLD key compression equation),
 * the token's entry of the compressed key cache, with W^{KD} the learned D x D/16 matrix.
 *   x     DEVICE bf16 [rows][D]   (the output of the Finch-C2 layers, one row per token)
 *   w_kd  DEVICE bf16 [D][Dc]     row-major (Dc = D/16 in the paper)
 *   c     DEVICE bf16 [rows][Dc]  written; must not alias x or w_kd
 * bf16 operands on the tensor cores, fp32 accumulation over D, one rounding to bf16.  D and Dc must be multiples
 * of 8 and Dc at most 256 (GF_ERR_UNSUPPORTED otherwise; D = 768 -> 48 and D = 2048 -> 128 are the paper's two
 * models); pointers 16-byte aligned; rows = 0 is a no-op.
 * Enqueues one kernel on `stream`, allocates nothing, does not synchronise. */
GF_API gf_status_t gf_gold_key_compress(const void *x, const void *w_kd, void *c, long long rows, int D, int Dc,
                                 gf_stream_t stream);

GF_API int gf_wkv6_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GF_WKV6_H */
