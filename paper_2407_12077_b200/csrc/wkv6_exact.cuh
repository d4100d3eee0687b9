// Token-by-token fp32 WKV-6 recurrence on the ALUs (the "exact" kernel).
//
// One CTA per (sequence, head).  256 threads: thread (g, j) with g = tid / 64 and
// j = tid % 64 keeps S[16g .. 16g+15][j] in registers, so the whole 64 x 64 state is
// register resident for the life of the sequence.  Tokens are staged through shared
// memory 16 at a time (coalesced loads, fetched one tile ahead into registers, widened to
// fp32, w = exp(-exp(x)) computed once per (token, channel)).  Per token every thread forms its partial of
//   y_t[j] = sum_i r_t[i] (S[i][j] + u[i] k_t[i] v_t[j])      (output before the update)
// and then applies S[i][j] = w_t[i] S[i][j] + k_t[i] v_t[j]; the four partials per j are
// summed after the tile.  No atomics: results are deterministic.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gf {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

constexpr int EX_N = 64;       // head size
constexpr int EX_TT = 16;      // tokens per shared-memory tile
constexpr int EX_THREADS = 256;

// Dense: cu_seqlens == nullptr, unit = b * H + h, rows b*T .. b*T+T-1.
// Packed: unit = s * H + h, rows cu_seqlens[s] .. cu_seqlens[s+1]-1.
template <typename IO>
__global__ void __launch_bounds__(EX_THREADS)
wkv6_exact_kernel(const IO* __restrict__ r, const IO* __restrict__ k, const IO* __restrict__ v,
                  const IO* __restrict__ x, const float* __restrict__ u,
                  const float* state_in, float* state_out, IO* __restrict__ y,
                  const int32_t* __restrict__ cu_seqlens, int T, int H)
{
    __shared__ __align__(16) float rs[EX_TT][EX_N], ks[EX_TT][EX_N], vs[EX_TT][EX_N], ws[EX_TT][EX_N];
    __shared__ __align__(16) float ypart[4][EX_TT][EX_N];
    __shared__ float coef[EX_TT];

    const int unit = blockIdx.x;
    const int seq = unit / H, h = unit % H;
    const int tid = threadIdx.x, g = tid >> 6, j = tid & 63;
    long long row0;
    int len;
    if (cu_seqlens) {
        row0 = cu_seqlens[seq];
        len = cu_seqlens[seq + 1] - cu_seqlens[seq];
    } else {
        row0 = (long long)seq * T;
        len = T;
    }
    const long long C = (long long)H * EX_N;
    const size_t sbase = (size_t)unit * EX_N * EX_N;

    float S[16];
#pragma unroll
    for (int ii = 0; ii < 16; ++ii)
        S[ii] = state_in ? state_in[sbase + (size_t)(16 * g + ii) * EX_N + j] : 0.f;

    const float u_c = u[h * EX_N + j];   // used in the load phase, where thread -> channel j

    // this thread's 4 (token, channel) pairs of a tile as they come from global memory; the next tile is
    // fetched into these registers while the current one runs through the recurrence
    IO rg[EX_TT / 4], kg[EX_TT / 4], vg[EX_TT / 4], xg[EX_TT / 4];
    auto fetch_tile = [&](int t0) {
        const int nt = min(EX_TT, len - t0);
#pragma unroll
        for (int p = 0; p < EX_TT / 4; ++p) {
            const int t = p * 4 + g;
            if (t < nt) {
                const size_t off = (size_t)(row0 + t0 + t) * C + (size_t)h * EX_N + j;
                rg[p] = r[off]; kg[p] = k[off]; vg[p] = v[off]; xg[p] = x[off];
            }
        }
    };
    if (len > 0) fetch_tile(0);

    for (int t0 = 0; t0 < len; t0 += EX_TT) {
        const int nt = min(EX_TT, len - t0);
        // ---- stage the tile: 16 tokens x 64 channels, 4 (token, channel) pairs per thread
#pragma unroll
        for (int p = 0; p < EX_TT / 4; ++p) {
            const int t = p * 4 + g;
            float rr = 0.f, kk = 0.f, vv = 0.f, ww = 1.f;
            if (t < nt) {
                rr = to_f32(rg[p]);
                kk = to_f32(kg[p]);
                vv = to_f32(vg[p]);
                ww = expf(-expf(to_f32(xg[p])));
            }
            rs[t][j] = rr; ks[t][j] = kk; vs[t][j] = vv; ws[t][j] = ww;
            // bonus coefficient sum_i r[i] u[i] k[i] of this token: reduce over the 64 channels
            float c = rr * u_c * kk;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            if ((j & 31) == 0) ypart[0][t][j >> 5] = c;      // two half sums per token, parked in ypart
        }
        __syncthreads();
        if (tid < EX_TT) coef[tid] = ypart[0][tid][0] + ypart[0][tid][1];
        __syncthreads();
        if (t0 + EX_TT < len) fetch_tile(t0 + EX_TT);
        // ---- recurrence over the tile (four independent partial sums per output)
        for (int t = 0; t < nt; ++t) {
            const float vv = vs[t][j];
            float acc[4] = {(g == 0) ? coef[t] * vv : 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 r4 = *reinterpret_cast<const float4*>(&rs[t][16 * g + 4 * q]);
                const float4 k4 = *reinterpret_cast<const float4*>(&ks[t][16 * g + 4 * q]);
                const float4 w4 = *reinterpret_cast<const float4*>(&ws[t][16 * g + 4 * q]);
                acc[0] = fmaf(r4.x, S[4 * q + 0], acc[0]); S[4 * q + 0] = fmaf(w4.x, S[4 * q + 0], k4.x * vv);
                acc[1] = fmaf(r4.y, S[4 * q + 1], acc[1]); S[4 * q + 1] = fmaf(w4.y, S[4 * q + 1], k4.y * vv);
                acc[2] = fmaf(r4.z, S[4 * q + 2], acc[2]); S[4 * q + 2] = fmaf(w4.z, S[4 * q + 2], k4.z * vv);
                acc[3] = fmaf(r4.w, S[4 * q + 3], acc[3]); S[4 * q + 3] = fmaf(w4.w, S[4 * q + 3], k4.w * vv);
            }
            ypart[g][t][j] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
        }
        __syncthreads();
        // ---- sum the four partials and store y (coalesced over j)
#pragma unroll
        for (int p = 0; p < EX_TT / 4; ++p) {
            const int t = p * 4 + g;
            if (t < nt) {
                const float s = (ypart[0][t][j] + ypart[1][t][j]) + (ypart[2][t][j] + ypart[3][t][j]);
                y[(size_t)(row0 + t0 + t) * C + (size_t)h * EX_N + j] = from_f32<IO>(s);
            }
        }
        __syncthreads();
    }
    if (state_out) {
#pragma unroll
        for (int ii = 0; ii < 16; ++ii) state_out[sbase + (size_t)(16 * g + ii) * EX_N + j] = S[ii];
    }
}

}  // namespace gf
