// LayerNorm across all heads: the normalisation of the o_t equation of the Finch-C2 block,
//     o_t = LayerNorm(concat_h(r_t . wkv_t + u'_t)) W^O,
// applied to the [rows][D = H*N] output of the WKV kernels (one LayerNorm over the D concatenated
// channels of a token, with per-channel gamma / beta and eps inside the square root).
//
// The operator is bound by HBM (D elements in, D out per token), so the kernel is built around two
// budgets: bytes in flight and instructions per element.
//  - A team of W warps (W = 1 up to 2048 channels, 2 up to 4096, 4 up to 8192) owns whole rows: lane l
//    of the team holds the 8-channel slices l + 32*W*j, j < VPL, of a row in registers.  Mean and
//    variance are a register pass plus one shuffle reduction each (two true passes: the mean first, then
//    the squared deviations), ten shuffles per row rather than per slice.
//  - Rows narrower than eight slices per lane are taken several at a time (up to 160 bytes per lane and
//    group, and the prefetch keeps a second group in flight); one CTA of twelve warps per SM walks the
//    rows (eight for fp32).  Measured: two CTAs per SM, sixteen warps (both spill) or twice the group
//    size lose; twelve warps beat eight by 2-7 %.
//  - The next group's slices are prefetched in their raw form (no instruction touches them until the
//    group is consumed) while the current group is reduced, normalised and stored.
//  - gamma and beta sit in shared memory, laid out so that every 16-byte read is contiguous across lanes.
//  - Teams of several warps exchange per-warp (mean, squared deviations) pairs through shared memory with
//    one named barrier per row group and merge them by the pairwise update formula (Chan, Golub,
//    LeVeque), which keeps the accuracy of the two-pass variance.
//  - Arithmetic on packed fp32 pairs; (y - mean) is formed before the scaling, so a constant row gives
//    exactly beta.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "device_info.cuh"
#include "gf_wkv6.h"

namespace gf {
namespace ln {

// Threads per CTA: the most warps that keep the widest variant free of register spills (12 for bf16, 8 for
// fp32, whose raw prefetch set is twice as large); divisible by the team widths 1, 2 and 4.
template <typename IO> constexpr int cta_threads() { return sizeof(IO) == 2 ? 384 : 256; }
constexpr int MAX_WARPS = 12;
constexpr int MAX_D = 8 * 32 * 4 * 8;               // lanes x team width x slices per lane, 8 channels each

// Eight consecutive elements as they come from memory; unpacked to fp32 only where they are consumed, so
// that a prefetched slice costs no instruction that would wait for its load.
template <typename IO> struct Raw;
template <> struct Raw<__nv_bfloat16> { uint4 u; };
template <> struct Raw<float> { float4 a, b; };

__device__ __forceinline__ void load_raw(const __nv_bfloat16* p, Raw<__nv_bfloat16>& r) { r.u = __ldcs(reinterpret_cast<const uint4*>(p)); }
__device__ __forceinline__ void load_raw(const float* p, Raw<float>& r)
{
    r.a = __ldcs(reinterpret_cast<const float4*>(p));
    r.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
}
__device__ __forceinline__ void zero_raw(Raw<__nv_bfloat16>& r) { r.u = make_uint4(0u, 0u, 0u, 0u); }
__device__ __forceinline__ void zero_raw(Raw<float>& r) { r.a = r.b = make_float4(0.f, 0.f, 0.f, 0.f); }
__device__ __forceinline__ void unpack(const Raw<__nv_bfloat16>& r, float2 (&f)[4])
{
    const uint32_t w[4] = {r.u.x, r.u.y, r.u.z, r.u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
}
__device__ __forceinline__ void unpack(const Raw<float>& r, float2 (&f)[4])
{
    f[0] = make_float2(r.a.x, r.a.y); f[1] = make_float2(r.a.z, r.a.w);
    f[2] = make_float2(r.b.x, r.b.y); f[3] = make_float2(r.b.z, r.b.w);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float2 (&f)[4])
{
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(f[i].x, f[i].y);
        w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
}
__device__ __forceinline__ void store8(float* p, const float2 (&f)[4])
{
    __stcs(reinterpret_cast<float4*>(p), make_float4(f[0].x, f[0].y, f[1].x, f[1].y));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(f[2].x, f[2].y, f[3].x, f[3].y));
}

// packed fp32 pair arithmetic (one instruction per pair)
__device__ __forceinline__ float2 add2(float2 a, float2 b)
{
    uint64_t ra = *reinterpret_cast<uint64_t*>(&a), rb = *reinterpret_cast<uint64_t*>(&b), rd;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    return *reinterpret_cast<float2*>(&rd);
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b)
{
    uint64_t ra = *reinterpret_cast<uint64_t*>(&a), rb = *reinterpret_cast<uint64_t*>(&b), rd;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(rd) : "l"(ra), "l"(rb));
    return *reinterpret_cast<float2*>(&rd);
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    uint64_t ra = *reinterpret_cast<uint64_t*>(&a), rb = *reinterpret_cast<uint64_t*>(&b), rc = *reinterpret_cast<uint64_t*>(&c), rd;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(rd) : "l"(ra), "l"(rb), "l"(rc));
    return *reinterpret_cast<float2*>(&rd);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// rows a team takes at a time: as many as keep at most 160 bytes per lane in one group (10 bf16 slices, 5 fp32
// slices: what the registers hold without spilling), between one and four
constexpr int rows_per_group(int VPL, int esize)
{
    const int r = (20 / esize) / VPL;
    return r < 1 ? 1 : (r > 4 ? 4 : r);
}
constexpr int smem_bytes(int VPL, int W) { return 2 * VPL * 2 * 32 * W * 16; }      // gamma and beta as float4 [VPL][2][32 W]

// y, out: [rows][D] (out may be y); gamma, beta: [D] fp32 or nullptr.  32 * W * VPL * 8 >= D; blockDim.x = cta_threads<IO>().
template <typename IO, int VPL, int W>
__global__ void __launch_bounds__(cta_threads<IO>(), 1)
layernorm_heads_kernel(const IO* __restrict__ y, const float* __restrict__ gamma, const float* __restrict__ beta,
                       float eps, IO* __restrict__ out, long long rows, int D)
{
    constexpr int R = rows_per_group(VPL, sizeof(IO));
    constexpr int THREADS = cta_threads<IO>();
    constexpr int TEAMS = THREADS / 32 / W;         // teams per CTA
    constexpr int TL = 32 * W;                      // lanes of a team
    extern __shared__ float4 gb[];                  // gamma [VPL][2][TL], then beta in the same layout
    __shared__ float2 part[TEAMS][2][R][W];         // per-warp (mean, squared deviations) by group parity
    __shared__ float cnt[MAX_WARPS];                // channels that each warp holds
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int team = warp / W, wt = warp % W, tl = wt * 32 + lane;

    for (int idx = tid; idx < VPL * 2 * TL; idx += THREADS) {
        const int j = idx / (2 * TL), half = (idx / TL) & 1, l = idx % TL;
        const int c = 8 * (l + TL * j) + 4 * half;
        float4 gv = make_float4(0.f, 0.f, 0.f, 0.f), bv = gv;
        if (c < D) {                                  // D is a multiple of 8: the four channels are all inside
            gv = gamma ? *reinterpret_cast<const float4*>(gamma + c) : make_float4(1.f, 1.f, 1.f, 1.f);
            if (beta) bv = *reinterpret_cast<const float4*>(beta + c);
        }
        gb[idx] = gv;
        gb[VPL * 2 * TL + idx] = bv;
    }
    int col[VPL];
    bool on[VPL];
    float mine = 0.f;
#pragma unroll
    for (int j = 0; j < VPL; ++j) {
        col[j] = 8 * (tl + TL * j);
        on[j] = col[j] < D;
        mine += on[j] ? 8.f : 0.f;
    }
    const float n_w = warp_sum(mine), inv_nw = 1.f / n_w;   // every warp holds at least one slice (host picks W, VPL)
    if (lane == 0) cnt[warp] = n_w;
    __syncthreads();
    const float inv_d = 1.f / (float)D;

    auto load_group = [&](Raw<IO> (&raw)[R][VPL], long long r0) {
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int j = 0; j < VPL; ++j) {
                if (on[j] && r0 + i < rows) load_raw(y + (size_t)(r0 + i) * D + col[j], raw[i][j]);
                else zero_raw(raw[i][j]);
            }
    };

    const long long stride = (long long)gridDim.x * TEAMS * R;
    long long r0 = ((long long)blockIdx.x * TEAMS + team) * R;
    Raw<IO> next[R][VPL];
    if (r0 < rows) load_group(next, r0);
    int par = 0;
    for (; r0 < rows; r0 += stride, par ^= 1) {
        float2 x[R][VPL][4];
#pragma unroll
        for (int i = 0; i < R; ++i)
#pragma unroll
            for (int j = 0; j < VPL; ++j) unpack(next[i][j], x[i][j]);
        if (r0 + stride < rows) load_group(next, r0 + stride);    // in flight during this group's arithmetic

        float2 scale[R], shift[R];                  // out = (x + shift) * scale * gamma + beta, shift = -mean (exact zero on a constant row)
        float mu[R], m2[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            // ---- mean of this warp's channels, then their squared deviations from it
            float2 s2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < VPL; ++j)
#pragma unroll
                for (int e = 0; e < 4; ++e) s2 = add2(s2, x[i][j][e]);
            mu[i] = warp_sum(s2.x + s2.y) * inv_nw;
            const float2 neg_m = make_float2(-mu[i], -mu[i]);
            float2 q2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int j = 0; j < VPL; ++j)
                if (on[j]) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 dv = add2(x[i][j][e], neg_m);
                        q2 = fma2(dv, dv, q2);
                    }
                }
            m2[i] = warp_sum(q2.x + q2.y);
        }
        if (W > 1) {
            // ---- merge the team's per-warp pairs
            if (lane == 0) {
#pragma unroll
                for (int i = 0; i < R; ++i) part[team][par][i][wt] = make_float2(mu[i], m2[i]);
            }
            asm volatile("bar.sync %0, %1;" ::"r"(1 + team), "r"(TL) : "memory");
#pragma unroll
            for (int i = 0; i < R; ++i) {
                float m = 0.f;
#pragma unroll
                for (int w = 0; w < W; ++w) m = fmaf(cnt[team * W + w], part[team][par][i][w].x, m);
                m *= inv_d;
                float q = 0.f;
#pragma unroll
                for (int w = 0; w < W; ++w) {
                    const float2 pw = part[team][par][i][w];
                    const float dm = pw.x - m;
                    q += fmaf(cnt[team * W + w] * dm, dm, pw.y);
                }
                mu[i] = m;
                m2[i] = q;
            }
            // part[team][par] is next written two groups on, after the barrier of the group between
        }
#pragma unroll
        for (int i = 0; i < R; ++i) {
            const float rstd = rsqrtf(fmaf(m2[i], inv_d, eps));
            scale[i] = make_float2(rstd, rstd);
            shift[i] = make_float2(-mu[i], -mu[i]);
        }
        // ---- normalise and store
#pragma unroll
        for (int j = 0; j < VPL; ++j)
            if (on[j]) {
                const float4 g0 = gb[(2 * j) * TL + tl], g1 = gb[(2 * j + 1) * TL + tl];
                const float4 b0 = gb[VPL * 2 * TL + (2 * j) * TL + tl], b1 = gb[VPL * 2 * TL + (2 * j + 1) * TL + tl];
                const float2 g[4] = {make_float2(g0.x, g0.y), make_float2(g0.z, g0.w), make_float2(g1.x, g1.y), make_float2(g1.z, g1.w)};
                const float2 b[4] = {make_float2(b0.x, b0.y), make_float2(b0.z, b0.w), make_float2(b1.x, b1.y), make_float2(b1.z, b1.w)};
#pragma unroll
                for (int i = 0; i < R; ++i)
                    if (r0 + i < rows) {
                        float2 o[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) o[e] = fma2(mul2(add2(x[i][j][e], shift[i]), scale[i]), g[e], b[e]);
                        store8(out + (size_t)(r0 + i) * D + col[j], o);
                    }
            }
    }
}

template <typename IO, int VPL, int W>
inline cudaError_t launch(const IO* y, const float* gamma, const float* beta, float eps, IO* out, long long rows, int D,
                          int n_sm, cudaStream_t st)
{
    constexpr int R = rows_per_group(VPL, sizeof(IO)), TEAMS = cta_threads<IO>() / 32 / W, SMEM = smem_bytes(VPL, W);
    if (SMEM + 1024 > 48 * 1024) {                  // dynamic plus the few static bytes would pass the default limit
        static PerDeviceFlag attr_set;              // opt in to the larger shared-memory size once per device
        const int dev = current_device();
        if (dev < 0) return cudaErrorInvalidDevice;
        if (!attr_set.is_set(dev)) {
            const cudaError_t e = cudaFuncSetAttribute(layernorm_heads_kernel<IO, VPL, W>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM);
            if (e != cudaSuccess) return e;
            attr_set.set(dev);
        }
    }
    const long long groups = (rows + (long long)R * TEAMS - 1) / ((long long)R * TEAMS);
    const unsigned grid = (unsigned)(groups < n_sm ? groups : n_sm);      // one resident CTA per SM walks the rows
    layernorm_heads_kernel<IO, VPL, W><<<grid, cta_threads<IO>(), SMEM, st>>>(y, gamma, beta, eps, out, rows, D);
    return cudaGetLastError();
}

}  // namespace ln

// Host side: picks the team width W and the slices per lane VPL from D (a multiple of 8, at most ln::MAX_D).
template <typename IO>
inline gf_status_t layernorm_heads(const IO* y, const float* gamma, const float* beta, float eps, IO* out, long long rows,
                                   int D, int n_sm, cudaStream_t st, std::atomic<uint64_t>* launches)
{
    if (D <= 0 || (D & 7) || D > ln::MAX_D || rows <= 0 || n_sm <= 0) return GF_ERR_INVALID_ARG;
    const int nvec = D / 8;
    const int w = nvec <= 256 ? 1 : (nvec <= 512 ? 2 : 4);
    const int vpl = (nvec + 32 * w - 1) / (32 * w);                       // 1..8; 5..8 for teams of several warps
    cudaError_t e = cudaErrorInvalidValue;
#define GF_LN_CASE(V, W_) \
    case V: e = ln::launch<IO, V, W_>(y, gamma, beta, eps, out, rows, D, n_sm, st); break;
    if (w == 1) {
        switch (vpl) { GF_LN_CASE(1, 1) GF_LN_CASE(2, 1) GF_LN_CASE(3, 1) GF_LN_CASE(4, 1)
                       GF_LN_CASE(5, 1) GF_LN_CASE(6, 1) GF_LN_CASE(7, 1) GF_LN_CASE(8, 1) }
    } else if (w == 2) {
        switch (vpl) { GF_LN_CASE(5, 2) GF_LN_CASE(6, 2) GF_LN_CASE(7, 2) GF_LN_CASE(8, 2) }
    } else {
        switch (vpl) { GF_LN_CASE(5, 4) GF_LN_CASE(6, 4) GF_LN_CASE(7, 4) GF_LN_CASE(8, 4) }
    }
#undef GF_LN_CASE
    launches->fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
