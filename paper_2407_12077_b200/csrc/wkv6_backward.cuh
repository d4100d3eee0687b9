// Gradient of the WKV-6 recurrence, token by token in fp32 on the ALUs (the counterpart of the exact
// forward kernel; training runs the recurrence backwards).
//
// Forward, per (sequence, head):  y_t[j] = sum_i r_t[i] (S_{t-1}[i][j] + u[i] k_t[i] v_t[j]),
//                                 S_t[i][j] = w_t[i] S_{t-1}[i][j] + k_t[i] v_t[j],  w = exp(-exp(x)).
// With G_t = dL/dS_t (G_T given) carried down from t = T:
//   dr_t[i] = sum_j dy_t[j] S_{t-1}[i][j] + u[i] k_t[i] (v_t . dy_t)
//   dk_t[i] = sum_j G_t[i][j] v_t[j]      + r_t[i] u[i] (v_t . dy_t)
//   dv_t[j] = sum_i G_t[i][j] k_t[i]      + (sum_i r_t[i] u[i] k_t[i]) dy_t[j]
//   dx_t[i] = (sum_j G_t[i][j] S_{t-1}[i][j]) (-w_t[i] exp(x_t[i]))
//   du[i]  += r_t[i] k_t[i] (v_t . dy_t)
//   G_{t-1}[i][j] = w_t[i] G_t[i][j] + r_t[i] dy_t[j],   dS_0 = G_0.
// The gradients need S_{t-1} while t runs downwards, so the states are recomputed from checkpoints: one
// CTA per unit first runs the recurrence forwards and keeps the state before every 64th token in the
// workspace; then, segment by segment from the last, it recomputes the 64 states of the segment into the
// workspace (they stay in L2) and walks the segment backwards.
// 128 threads: threads 0-63 own rows (thread i holds G[i][.] in registers and reads S_{t-1}[i][.]: the sums
// over j of dr, dk, dx are private), threads 64-127 own columns (thread j holds G[.][j], and S[.][j] while
// states are recomputed: the sum over i of dv is private).  Both copies of G take the same update.  The
// token's vectors are broadcast through shared memory.  No atomics: results are deterministic; du is
// left per unit and summed over the batch by a second, tiny kernel in a fixed order.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace gf {
namespace bw {

constexpr int N = 64;          // head size
constexpr int SEG = 64;        // tokens between state checkpoints
constexpr int THREADS = 128;

// floats of workspace per unit: checkpoints, the states of one segment, the unit's du
__host__ __device__ inline size_t unit_floats(int T)
{
    const size_t nseg = (size_t)(T + SEG - 1) / SEG;
    return nseg * N * N + (size_t)SEG * N * N + N;
}

__global__ void __launch_bounds__(THREADS)
wkv6_backward_kernel(const float* __restrict__ r, const float* __restrict__ k, const float* __restrict__ v,
                     const float* __restrict__ x, const float* __restrict__ u, const float* __restrict__ state_in,
                     const float* __restrict__ dy, const float* __restrict__ dstate_out, float* __restrict__ dr,
                     float* __restrict__ dk, float* __restrict__ dv, float* __restrict__ dx, float* dstate_in,
                     float* ws, int T, int H)
{
    __shared__ float sr[N], sk[N], sv[N], sw[N], sdy[N], sx[N], su[N];
    const int unit = blockIdx.x, b = unit / H, h = unit % H;
    const int tid = threadIdx.x, idx = tid & 63;
    const bool rows = tid < 64;                                  // row owner (i = idx) or column owner (j = idx)
    const size_t C = (size_t)H * N;
    const size_t tok0 = (size_t)b * T * C + (size_t)h * N;       // element offset of this unit's token 0
    const int nseg = (T + SEG - 1) / SEG;
    float* ckpt = ws + (size_t)unit * unit_floats(T);            // [nseg][N][N]
    float* segst = ckpt + (size_t)nseg * N * N;                  // [SEG][N][N]: S_{t-1} of the segment's tokens
    float* du_unit = segst + (size_t)SEG * N * N;                // [N]
    const size_t sbase = (size_t)unit * N * N;

    if (tid < N) su[tid] = u[h * N + tid];

    // ---- forward sweep: the state before every SEG-th token (column owners carry S[.][j])
    float S[N];
    if (!rows) {
#pragma unroll
        for (int i = 0; i < N; ++i) S[i] = state_in ? state_in[sbase + (size_t)i * N + idx] : 0.f;
    }
    for (int t = 0; t < T; ++t) {
        const size_t o = tok0 + (size_t)t * C;
        __syncthreads();
        if (rows) { sk[idx] = k[o + idx]; sw[idx] = expf(-expf(x[o + idx])); }
        else sv[idx] = v[o + idx];
        __syncthreads();
        if (!rows) {
            if (t % SEG == 0) {
                float* c = ckpt + (size_t)(t / SEG) * N * N;
#pragma unroll
                for (int i = 0; i < N; ++i) c[(size_t)i * N + idx] = S[i];
            }
            const float vj = sv[idx];
#pragma unroll
            for (int i = 0; i < N; ++i) S[i] = fmaf(sw[i], S[i], sk[i] * vj);
        }
    }

    // ---- the adjoint of the state: G[i][.] on the row owners, G[.][j] on the column owners
    float G[N];
#pragma unroll
    for (int q = 0; q < N; ++q) {
        const size_t e = rows ? sbase + (size_t)idx * N + q : sbase + (size_t)q * N + idx;
        G[q] = dstate_out ? dstate_out[e] : 0.f;
    }
    float du_acc = 0.f;

    for (int seg = nseg - 1; seg >= 0; --seg) {
        const int t0 = seg * SEG, len = min(SEG, T - t0);
        // ---- recompute S_{t-1} for the segment's tokens from its checkpoint
        if (!rows) {
            const float* c = ckpt + (size_t)seg * N * N;
#pragma unroll
            for (int i = 0; i < N; ++i) S[i] = c[(size_t)i * N + idx];
        }
        for (int tt = 0; tt < len; ++tt) {
            const size_t o = tok0 + (size_t)(t0 + tt) * C;
            __syncthreads();
            if (rows) { sk[idx] = k[o + idx]; sw[idx] = expf(-expf(x[o + idx])); }
            else sv[idx] = v[o + idx];
            __syncthreads();
            if (!rows) {
                float* d = segst + (size_t)tt * N * N;
                const float vj = sv[idx];
#pragma unroll
                for (int i = 0; i < N; ++i) {
                    d[(size_t)i * N + idx] = S[i];
                    S[i] = fmaf(sw[i], S[i], sk[i] * vj);
                }
            }
        }
        // ---- walk the segment backwards
        for (int tt = len - 1; tt >= 0; --tt) {
            const size_t o = tok0 + (size_t)(t0 + tt) * C;
            __syncthreads();                                      // (also orders the state stores above before the loads below)
            if (rows) {
                sr[idx] = r[o + idx]; sk[idx] = k[o + idx];
                const float xv = x[o + idx];
                sx[idx] = xv; sw[idx] = expf(-expf(xv));
            } else {
                sv[idx] = v[o + idx]; sdy[idx] = dy[o + idx];
            }
            __syncthreads();
            float dyv = 0.f, ruk = 0.f;                           // v_t . dy_t and sum_i r u k: every thread forms both
#pragma unroll
            for (int q = 0; q < N; ++q) {
                dyv = fmaf(sdy[q], sv[q], dyv);
                ruk = fmaf(sr[q] * su[q], sk[q], ruk);
            }
            if (rows) {
                const float4* Srow = reinterpret_cast<const float4*>(segst + (size_t)tt * N * N + (size_t)idx * N);
                const float ri = sr[idx], ki = sk[idx], wi = sw[idx], ui = su[idx];
                float a_r = 0.f, a_k = 0.f, a_w = 0.f;
#pragma unroll
                for (int q4 = 0; q4 < N / 4; ++q4) {
                    const float4 s4 = Srow[q4];
                    const float sv4[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int q = 4 * q4 + e;
                        a_r = fmaf(sdy[q], sv4[e], a_r);
                        a_k = fmaf(G[q], sv[q], a_k);
                        a_w = fmaf(G[q], sv4[e], a_w);
                        G[q] = fmaf(wi, G[q], ri * sdy[q]);
                    }
                }
                dr[o + idx] = fmaf(ui * ki, dyv, a_r);
                dk[o + idx] = fmaf(ri * ui, dyv, a_k);
                dx[o + idx] = a_w * (-wi * expf(sx[idx]));
                du_acc = fmaf(ri * ki, dyv, du_acc);
            } else {
                const float dyj = sdy[idx];
                float a_v = 0.f;
#pragma unroll
                for (int q = 0; q < N; ++q) {
                    a_v = fmaf(G[q], sk[q], a_v);
                    G[q] = fmaf(sw[q], G[q], sr[q] * dyj);
                }
                dv[o + idx] = fmaf(ruk, dyj, a_v);
            }
        }
    }
    if (rows) du_unit[idx] = du_acc;
    else if (dstate_in) {
#pragma unroll
        for (int i = 0; i < N; ++i) dstate_in[sbase + (size_t)i * N + idx] = G[i];
    }
}

// du[h][i] = sum over the batch of the units' partial sums, in batch order
__global__ void __launch_bounds__(N)
wkv6_backward_du_kernel(const float* ws, size_t unit_stride, size_t du_offset, int B, int H, float* __restrict__ du)
{
    const int h = blockIdx.x, i = threadIdx.x;
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc += ws[(size_t)(b * H + h) * unit_stride + du_offset + i];
    du[h * N + i] = acc;
}

}  // namespace bw
}  // namespace gf
