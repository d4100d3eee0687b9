// Single-token WKV-6 decode step: y = r (S + diag(u) k^T v), then S = diag(w) S + k^T v.
//
// The step streams the 16 KB fp32 state of every (sequence, head) once in and once out,
// so it is bound by state traffic.  One CTA per (sequence, head), 256 threads; thread
// (ig, jq) = (tid / 16, tid % 16) handles rows ig, ig+16, ig+32, ig+48 and the four
// columns 4*jq .. 4*jq+3 with 128-bit loads/stores (a warp covers two full 256-byte rows).
// Column sums over the 16 row groups go through shared memory in a fixed order
// (deterministic).  state_out may alias state_in: every element is read and written by
// the same thread.  C2 = true is the Finch-C2 form: the key is multiplied by one minus its decay,
// there is no bonus, and u2 (the token's second-value vector, may be NULL) is added to the output.
#pragma once
#include "wkv6_exact.cuh"

namespace gf {

constexpr int ST_THREADS = 256;

template <typename IO, bool C2 = false>
__global__ void __launch_bounds__(ST_THREADS)
wkv6_step_kernel(const IO* __restrict__ r, const IO* __restrict__ k, const IO* __restrict__ v,
                 const IO* __restrict__ x, const float* __restrict__ u,
                 const float* state_in, float* state_out, IO* __restrict__ y, int H,
                 const IO* __restrict__ u2 = nullptr)
{
    __shared__ __align__(16) float rs[64], ks[64], vs[64], ws[64];
    __shared__ float ruk[2];
    __shared__ __align__(16) float part[16][64];
    // Launched with programmatic stream serialisation: the next step kernel of the stream may be scheduled while
    // this one drains (it holds at its own wait below), and this one touches no global memory before the kernels
    // ahead of it have completed and flushed.  Without that launch attribute both instructions do nothing.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int unit = blockIdx.x, h = unit % H;
    const int tid = threadIdx.x;
    const size_t voff = (size_t)unit * 64;
    const size_t sbase = (size_t)unit * 64 * 64;

    asm volatile("griddepcontrol.wait;" ::: "memory");
    // issue the state loads first so they overlap the vector staging
    const int ig = tid >> 4, jq = tid & 15;
    float4 S[4];
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const int i = ig + 16 * p;
        S[p] = state_in ? *reinterpret_cast<const float4*>(state_in + sbase + (size_t)i * 64 + 4 * jq)
                        : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (tid < 64) {
        const float rr = to_f32(r[voff + tid]);
        const float ww = expf(-expf(to_f32(x[voff + tid])));
        const float kk = C2 ? to_f32(k[voff + tid]) * (1.f - ww) : to_f32(k[voff + tid]);
        rs[tid] = rr; ks[tid] = kk; vs[tid] = to_f32(v[voff + tid]);
        ws[tid] = ww;
        float c = C2 ? 0.f : rr * u[h * 64 + tid] * kk;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if ((tid & 31) == 0) ruk[tid >> 5] = c;
    }
    __syncthreads();
    const float4 v4 = *reinterpret_cast<const float4*>(&vs[4 * jq]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const int i = ig + 16 * p;
        const float rr = rs[i], kk = ks[i], ww = ws[i];
        acc.x = fmaf(rr, S[p].x, acc.x); acc.y = fmaf(rr, S[p].y, acc.y);
        acc.z = fmaf(rr, S[p].z, acc.z); acc.w = fmaf(rr, S[p].w, acc.w);
        S[p].x = fmaf(ww, S[p].x, kk * v4.x); S[p].y = fmaf(ww, S[p].y, kk * v4.y);
        S[p].z = fmaf(ww, S[p].z, kk * v4.z); S[p].w = fmaf(ww, S[p].w, kk * v4.w);
        if (state_out)
            *reinterpret_cast<float4*>(state_out + sbase + (size_t)i * 64 + 4 * jq) = S[p];
    }
    *reinterpret_cast<float4*>(&part[ig][4 * jq]) = acc;
    __syncthreads();
    if (tid < 64) {
        float s = (ruk[0] + ruk[1]) * vs[tid];
#pragma unroll
        for (int q = 0; q < 16; ++q) s += part[q][tid];
        if (C2 && u2) s += to_f32(u2[voff + tid]);
        y[voff + tid] = from_f32<IO>(s);
    }
}

// Launch with programmatic stream serialisation (see the kernel): back-to-back decode steps lose the launch gap.
template <typename IO, bool C2>
inline cudaError_t launch_step(unsigned grid, cudaStream_t st, const IO* r, const IO* k, const IO* v, const IO* x, const float* u,
                               const float* state_in, float* state_out, IO* y, int H, const IO* u2)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(ST_THREADS);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, wkv6_step_kernel<IO, C2>, r, k, v, x, u, state_in, state_out, y, H, u2);
}

}  // namespace gf
