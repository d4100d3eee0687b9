// C ABI of the gf_wkv6 library: argument validation, kernel selection and launches.
// Every entry point is declared and documented in include/gf_wkv6.h.
#include "gf_wkv6.h"

#include <atomic>
#include <mutex>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "decay_logit.cuh"
#include "key_compress.cuh"
#include "ln_heads.cuh"
#include "wkv6_backward.cuh"
#include "wkv6_backward_chunked.cuh"
#include "wkv6_chunked.cuh"
#include "wkv6_exact.cuh"
#include "wkv6_step.cuh"

namespace {

std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_kernel{GF_KERNEL_AUTO};
// caller-owned scratch registered with gf_wkv6_set_workspace (NULL: none)
std::atomic<float*> g_ws{nullptr};
std::atomic<size_t> g_ws_bytes{0};

// Scratch of gf_wkv6_prefill_static: lives in the library image on every GPU that loads it.  Its name is
// only a host-side handle here; the device address comes from cudaGetSymbolAddress (static_scratch()).
static __device__ __align__(256) float g_static_scratch[GF_WKV6_STATIC_SCRATCH_BYTES / sizeof(float)];

// Device address of g_static_scratch on the current device, looked up once per device.
float* static_scratch()
{
    static std::mutex mu;
    static float* addr[gf::MAX_DEVICES] = {};
    const int dev = gf::current_device();
    if (dev < 0) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        float* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess) return nullptr;
        addr[dev] = ptr;
    }
    return addr[dev];
}

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Pointer checks shared by all compute calls; `need_state_in` is false where NULL means zero.
gf_status_t check_ptrs(const void* r, const void* k, const void* v, const void* x, const float* u,
                       const float* state_in, const float* state_out, const void* y)
{
    if (!r || !k || !v || !x || !u || !y) return GF_ERR_INVALID_ARG;
    if (misaligned(r) || misaligned(k) || misaligned(v) || misaligned(x) || misaligned(u) ||
        misaligned(y) || misaligned(state_in) || misaligned(state_out))
        return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x) return GF_ERR_INVALID_ARG;
    return GF_OK;
}

inline gf_status_t launch_result()
{
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

// state_out <- state_in (or zero) for calls that have no tokens to process.
gf_status_t pass_state(const float* state_in, float* state_out, size_t n_units, cudaStream_t st)
{
    if (!state_out || n_units == 0) return GF_OK;
    const size_t bytes = n_units * 64 * 64 * sizeof(float);
    cudaError_t e = cudaSuccess;
    if (!state_in) e = cudaMemsetAsync(state_out, 0, bytes, st);
    else if (state_in != state_out) e = cudaMemcpyAsync(state_out, state_in, bytes, cudaMemcpyDeviceToDevice, st);
    return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

template <typename IO>
gf_status_t run_exact(const IO* r, const IO* k, const IO* v, const IO* x, const float* u,
                      const float* state_in, float* state_out, IO* y, const int32_t* cu,
                      int n_seq, int T, int H, cudaStream_t st)
{
    const long long units = (long long)n_seq * H;
    if (units > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    gf::wkv6_exact_kernel<IO><<<(unsigned)units, gf::EX_THREADS, 0, st>>>(r, k, v, x, u, state_in, state_out, y, cu, T, H);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_result();
}

template <typename IO>
gf_status_t prefill_dense(const IO* r, const IO* k, const IO* v, const IO* x, const float* u,
                          const float* state_in, float* state_out, IO* y, int B, int T, int H, int N,
                          cudaStream_t st, bool allow_chunked)
{
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if ((long long)B * T >= (1LL << 31)) return GF_ERR_INVALID_ARG;
    if (B == 0 || H == 0) return GF_OK;
    if (T == 0) return pass_state(state_in, state_out, (size_t)B * H, st);
    gf_status_t s = check_ptrs(r, k, v, x, u, state_in, state_out, y);
    if (s != GF_OK) return s;
    const int sel = g_kernel.load(std::memory_order_relaxed);
    if (allow_chunked && sel != GF_KERNEL_EXACT) {
        s = gf::chunked_prefill(reinterpret_cast<const __nv_bfloat16*>(r), reinterpret_cast<const __nv_bfloat16*>(k),
                                reinterpret_cast<const __nv_bfloat16*>(v), reinterpret_cast<const __nv_bfloat16*>(x),
                                u, state_in, state_out, reinterpret_cast<__nv_bfloat16*>(y), nullptr,
                                B, T, (long long)B * T, H, st, &g_launches, g_ws.load(std::memory_order_relaxed),
                                g_ws_bytes.load(std::memory_order_relaxed));
        if (s != GF_ERR_UNSUPPORTED || sel == GF_KERNEL_CHUNKED) return s;
    }
    return run_exact<IO>(r, k, v, x, u, state_in, state_out, y, nullptr, B, T, H, st);
}

template <typename IO>
gf_status_t prefill_varlen(const IO* r, const IO* k, const IO* v, const IO* x, const float* u,
                           const float* state_in, float* state_out, IO* y, const int32_t* cu, int S,
                           int total_T, int max_seqlen, int H, int N, cudaStream_t st, bool allow_chunked)
{
    if (S < 0 || total_T < 0 || max_seqlen < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (max_seqlen > total_T) max_seqlen = total_T;
    if (S == 0 || H == 0) return GF_OK;
    if (!cu || (reinterpret_cast<uintptr_t>(cu) & 3u)) return GF_ERR_INVALID_ARG;
    if (total_T == 0) return pass_state(state_in, state_out, (size_t)S * H, st);
    gf_status_t s = check_ptrs(r, k, v, x, u, state_in, state_out, y);
    if (s != GF_OK) return s;
    const int sel = g_kernel.load(std::memory_order_relaxed);
    if (allow_chunked && sel != GF_KERNEL_EXACT) {
        s = gf::chunked_prefill(reinterpret_cast<const __nv_bfloat16*>(r), reinterpret_cast<const __nv_bfloat16*>(k),
                                reinterpret_cast<const __nv_bfloat16*>(v), reinterpret_cast<const __nv_bfloat16*>(x),
                                u, state_in, state_out, reinterpret_cast<__nv_bfloat16*>(y), cu,
                                S, max_seqlen, (long long)total_T, H, st, &g_launches,
                                g_ws.load(std::memory_order_relaxed), g_ws_bytes.load(std::memory_order_relaxed));
        if (s != GF_ERR_UNSUPPORTED || sel == GF_KERNEL_CHUNKED) return s;
    }
    return run_exact<IO>(r, k, v, x, u, state_in, state_out, y, cu, S, max_seqlen, H, st);
}

template <typename IO>
gf_status_t step_impl(const IO* r, const IO* k, const IO* v, const IO* x, const float* u,
                      const float* state_in, float* state_out, IO* y, int B, int H, int N, cudaStream_t st)
{
    if (B < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    gf_status_t s = check_ptrs(r, k, v, x, u, state_in, state_out, y);
    if (s != GF_OK) return s;
    const long long units = (long long)B * H;
    if (units > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    const cudaError_t e = gf::launch_step<IO, false>((unsigned)units, st, r, k, v, x, u, state_in, state_out, y, H, nullptr);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace

namespace {
template <typename IO>
gf_status_t layernorm_call(const IO* y, const float* gamma, const float* beta, float eps, IO* out, long long rows,
                           int H, int N, gf_stream_t stream)
{
    if (rows < 0 || H < 0 || N < 0 || !(eps >= 0.f) || eps > 3.0e38f) return GF_ERR_INVALID_ARG;
    const long long D = (long long)H * N;
    if (rows == 0 || D == 0) return GF_OK;
    if ((D & 7) || D > gf::ln::MAX_D) return GF_ERR_UNSUPPORTED;
    if (rows > (1LL << 62) / D) return GF_ERR_INVALID_ARG;
    if (!y || !out || misaligned(y) || misaligned(out) || misaligned(gamma) || misaligned(beta)) return GF_ERR_INVALID_ARG;
    return gf::layernorm_heads<IO>(y, gamma, beta, eps, out, rows, (int)D, gf::sm_count(), (cudaStream_t)stream, &g_launches);
}
}  // namespace

extern "C" {

gf_status_t gf_wkv6_prefill(const void* r, const void* k, const void* v, const void* x, const float* u,
                            const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                            gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    return prefill_dense<bf>((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out,
                             (bf*)y, B, T, H, N, (cudaStream_t)stream, true);
}

gf_status_t gf_wkv6_prefill_static(const void* r, const void* k, const void* v, const void* x, const float* u,
                                   const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                                   gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if ((long long)B * T >= (1LL << 31)) return GF_ERR_INVALID_ARG;
    if (B == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (T == 0) return pass_state(state_in, state_out, (size_t)B * H, st);
    gf_status_t s = check_ptrs(r, k, v, x, u, state_in, state_out, y);
    if (s != GF_OK) return s;
    // The split takes as many segments as the built-in array holds; a call that would split but does not fit
    // even with two segments is refused rather than run at a fraction of the GPU.
    int seg_chunks = 0;
    size_t need = 0;
    const int n_sm = gf::sm_count();
    if (gf::choose_split((long long)B * H, T, n_sm, &seg_chunks, &need) > 1 &&
        gf::choose_split((long long)B * H, T, n_sm, &seg_chunks, &need, GF_WKV6_STATIC_SCRATCH_BYTES) == 1)
        return GF_ERR_WORKSPACE;                                          // beyond the built-in scratch
    float* scratch = static_scratch();
    if (!scratch) return GF_ERR_CUDA;
    return gf::chunked_prefill((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out, (bf*)y,
                               nullptr, B, T, (long long)B * T, H, st, &g_launches, scratch,
                               GF_WKV6_STATIC_SCRATCH_BYTES);
}

gf_status_t gf_wkv6_prefill_c2(const void* r, const void* k, const void* v, const void* x, const void* u2,
                               const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                               gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if ((long long)B * T >= (1LL << 31)) return GF_ERR_INVALID_ARG;
    if (B == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (T == 0) return pass_state(state_in, state_out, (size_t)B * H, st);
    if (!r || !k || !v || !x || !y) return GF_ERR_INVALID_ARG;
    if (misaligned(r) || misaligned(k) || misaligned(v) || misaligned(x) || misaligned(u2) || misaligned(y) ||
        misaligned(state_in) || misaligned(state_out))
        return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x || y == u2) return GF_ERR_INVALID_ARG;
    return gf::chunked_prefill((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, nullptr, state_in, state_out,
                               (bf*)y, nullptr, B, T, (long long)B * T, H, st, &g_launches,
                               g_ws.load(std::memory_order_relaxed), g_ws_bytes.load(std::memory_order_relaxed),
                               (const bf*)u2, 1);
}

gf_status_t gf_wkv6_prefill_varlen_c2(const void* r, const void* k, const void* v, const void* x, const void* u2,
                                      const float* state_in, float* state_out, void* y, const int32_t* cu_seqlens,
                                      int S, int total_T, int max_seqlen, int H, int N, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (S < 0 || total_T < 0 || max_seqlen < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (max_seqlen > total_T) max_seqlen = total_T;
    if (S == 0 || H == 0) return GF_OK;
    if (!cu_seqlens || (reinterpret_cast<uintptr_t>(cu_seqlens) & 3u)) return GF_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (total_T == 0) return pass_state(state_in, state_out, (size_t)S * H, st);
    if (!r || !k || !v || !x || !y) return GF_ERR_INVALID_ARG;
    if (misaligned(r) || misaligned(k) || misaligned(v) || misaligned(x) || misaligned(u2) || misaligned(y) ||
        misaligned(state_in) || misaligned(state_out))
        return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x || y == u2) return GF_ERR_INVALID_ARG;
    return gf::chunked_prefill((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, nullptr, state_in, state_out,
                               (bf*)y, cu_seqlens, S, max_seqlen, (long long)total_T, H, st, &g_launches,
                               g_ws.load(std::memory_order_relaxed), g_ws_bytes.load(std::memory_order_relaxed),
                               (const bf*)u2, 1);
}

gf_status_t gf_wkv6_step_c2(const void* r, const void* k, const void* v, const void* x, const void* u2,
                            const float* state_in, float* state_out, void* y, int B, int H, int N, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (B < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    if (!r || !k || !v || !x || !y) return GF_ERR_INVALID_ARG;
    if (misaligned(r) || misaligned(k) || misaligned(v) || misaligned(x) || misaligned(u2) || misaligned(y) ||
        misaligned(state_in) || misaligned(state_out))
        return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x || y == u2) return GF_ERR_INVALID_ARG;
    const long long units = (long long)B * H;
    if (units > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    const cudaError_t e = gf::launch_step<bf, true>((unsigned)units, (cudaStream_t)stream, (const bf*)r, (const bf*)k, (const bf*)v,
                                                   (const bf*)x, nullptr, state_in, state_out, (bf*)y, H, (const bf*)u2);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

gf_status_t gf_wkv6_sequence_summary(const void* k, const void* v, const void* x, float* summary, int B, int T, int H,
                                     int N, int c2, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    if (T == 0 || (long long)B * T >= (1LL << 31)) return GF_ERR_INVALID_ARG;
    if (!k || !v || !x || !summary || misaligned(k) || misaligned(v) || misaligned(x) || misaligned(summary))
        return GF_ERR_INVALID_ARG;
    return gf::chunked_summary((const bf*)k, (const bf*)v, (const bf*)x, summary, B, T, H, c2 != 0, (cudaStream_t)stream,
                               &g_launches);
}

gf_status_t gf_wkv6_fold_summaries(const float* state_in, const float* summaries, int n_fold, int B, int H, int N,
                                   float* state_out, gf_stream_t stream)
{
    if (B < 0 || H < 0 || N < 0 || n_fold < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    if (!state_out || (n_fold > 0 && !summaries) || misaligned(state_in) || misaligned(state_out) || misaligned(summaries))
        return GF_ERR_INVALID_ARG;
    const long long units = (long long)B * H;
    if (units > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    gf::wkv6_fold_kernel<<<(unsigned)units, 256, 0, (cudaStream_t)stream>>>(state_in, summaries, n_fold, units, state_out);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_result();
}

gf_status_t gf_wkv6_prefill_f32(const float* r, const float* k, const float* v, const float* x, const float* u,
                                const float* state_in, float* state_out, float* y, int B, int T, int H, int N,
                                gf_stream_t stream)
{
    return prefill_dense<float>(r, k, v, x, u, state_in, state_out, y, B, T, H, N, (cudaStream_t)stream, false);
}

gf_status_t gf_wkv6_prefill_varlen(const void* r, const void* k, const void* v, const void* x, const float* u,
                                   const float* state_in, float* state_out, void* y, const int32_t* cu_seqlens,
                                   int S, int total_T, int max_seqlen, int H, int N, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    return prefill_varlen<bf>((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out,
                              (bf*)y, cu_seqlens, S, total_T, max_seqlen, H, N, (cudaStream_t)stream, true);
}

gf_status_t gf_wkv6_prefill_varlen_f32(const float* r, const float* k, const float* v, const float* x,
                                       const float* u, const float* state_in, float* state_out, float* y,
                                       const int32_t* cu_seqlens, int S, int total_T, int max_seqlen, int H,
                                       int N, gf_stream_t stream)
{
    return prefill_varlen<float>(r, k, v, x, u, state_in, state_out, y, cu_seqlens, S, total_T, max_seqlen, H, N,
                                 (cudaStream_t)stream, false);
}

gf_status_t gf_wkv6_step(const void* r, const void* k, const void* v, const void* x, const float* u,
                         const float* state_in, float* state_out, void* y, int B, int H, int N, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    return step_impl<bf>((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out, (bf*)y,
                         B, H, N, (cudaStream_t)stream);
}

gf_status_t gf_wkv6_step_f32(const float* r, const float* k, const float* v, const float* x, const float* u,
                             const float* state_in, float* state_out, float* y, int B, int H, int N,
                             gf_stream_t stream)
{
    return step_impl<float>(r, k, v, x, u, state_in, state_out, y, B, H, N, (cudaStream_t)stream);
}

size_t gf_wkv6_backward_workspace_bytes(int B, int T, int H, int N)
{
    if (B <= 0 || T <= 0 || H <= 0 || N != 64) return 0;
    return (size_t)B * H * gf::bw::unit_floats(T) * sizeof(float);
}

gf_status_t gf_wkv6_backward_f32(const float* r, const float* k, const float* v, const float* x, const float* u,
                                 const float* state_in, const float* dy, const float* dstate_out, float* dr,
                                 float* dk, float* dv, float* dx, float* du, float* dstate_in, int B, int T, int H,
                                 int N, void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if ((long long)B * T >= (1LL << 31)) return GF_ERR_INVALID_ARG;
    if (B == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t sbytes = (size_t)B * H * 64 * 64 * sizeof(float);
    if (T == 0) {
        // no token: the state adjoint passes through and the bonus gets no gradient
        if (misaligned(dstate_out) || misaligned(dstate_in) || misaligned(du)) return GF_ERR_INVALID_ARG;
        cudaError_t e = cudaSuccess;
        if (dstate_in && !dstate_out) e = cudaMemsetAsync(dstate_in, 0, sbytes, st);
        else if (dstate_in && dstate_in != dstate_out) e = cudaMemcpyAsync(dstate_in, dstate_out, sbytes, cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && du) e = cudaMemsetAsync(du, 0, (size_t)H * 64 * sizeof(float), st);
        return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
    }
    if (!r || !k || !v || !x || !u || !dy || !dr || !dk || !dv || !dx || !du) return GF_ERR_INVALID_ARG;
    const void* ptrs[] = {r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, workspace};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    const void* ins[] = {r, k, v, x, dy};
    const void* outs[] = {dr, dk, dv, dx};
    for (const void* o : outs)
        for (const void* in : ins)
            if (o == in) return GF_ERR_INVALID_ARG;
    const long long units = (long long)B * H;
    if (units > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < gf_wkv6_backward_workspace_bytes(B, T, H, N)) return GF_ERR_WORKSPACE;
    float* ws = static_cast<float*>(workspace);
    gf::bw::wkv6_backward_kernel<<<(unsigned)units, gf::bw::THREADS, 0, st>>>(r, k, v, x, u, state_in, dy, dstate_out, dr, dk,
                                                                            dv, dx, dstate_in, ws, T, H);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return GF_ERR_CUDA;
    const size_t stride = gf::bw::unit_floats(T);
    gf::bw::wkv6_backward_du_kernel<<<(unsigned)H, gf::bw::N, 0, st>>>(ws, stride, stride - gf::bw::N, B, H, du);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_result();
}

size_t gf_wkv6_backward_bf16_workspace_bytes(int B, int T, int H, int N)
{
    if (B <= 0 || T <= 0 || H <= 0 || N != 64) return 0;
    const int n_sm = gf::sm_count();
    if (n_sm <= 0) return 0;
    return gf::chunked_backward_workspace_bytes((long long)B * H, T, n_sm);
}

namespace {
// bf16 gradient, classic (u, du given) or Finch-C2 form (c2: no bonus)
gf_status_t backward_bf16(const void* r, const void* k, const void* v, const void* x, const float* u,
                          const float* state_in, const void* dy, const float* dstate_out, void* dr, void* dk, void* dv,
                          void* dx, float* du, float* dstate_in, int B, int T, int H, int N, void* workspace,
                          size_t workspace_bytes, gf_stream_t stream, bool c2, bool saved = false)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t sbytes = (size_t)B * H * 64 * 64 * sizeof(float);
    if (T == 0) {
        // no token: the state adjoint passes through and the bonus gets no gradient
        if (misaligned(dstate_out) || misaligned(dstate_in) || misaligned(du)) return GF_ERR_INVALID_ARG;
        cudaError_t e = cudaSuccess;
        if (dstate_in && !dstate_out) e = cudaMemsetAsync(dstate_in, 0, sbytes, st);
        else if (dstate_in && dstate_in != dstate_out) e = cudaMemcpyAsync(dstate_in, dstate_out, sbytes, cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && du) e = cudaMemsetAsync(du, 0, (size_t)H * 64 * sizeof(float), st);
        return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
    }
    if (!r || !k || !v || !x || !dy || !dr || !dk || !dv || !dx || (!c2 && (!u || !du))) return GF_ERR_INVALID_ARG;
    const void* ptrs[] = {r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, workspace};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    const void* ins[] = {r, k, v, x, dy};
    const void* outs[] = {dr, dk, dv, dx};
    for (const void* o : outs)
        for (const void* in : ins)
            if (o == in) return GF_ERR_INVALID_ARG;
    // (a split call reads dstate_out in every segment's CTA and writes dstate_in from the first segment's: not in place)
    if (dstate_in && dstate_in == dstate_out) return GF_ERR_INVALID_ARG;
    if ((long long)B * H > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    if ((long long)B * T >= (1LL << 31) - 64) return GF_ERR_UNSUPPORTED;
    const size_t need = gf_wkv6_backward_bf16_workspace_bytes(B, T, H, N);
    if (need == 0) return GF_ERR_CUDA;
    if (!workspace || workspace_bytes < need) return GF_ERR_WORKSPACE;
    const gf_status_t s = gf::chunked_backward((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, (const bf*)dy,
                                               dstate_out, (bf*)dr, (bf*)dk, (bf*)dv, (bf*)dx, du, dstate_in, B, T, H,
                                               static_cast<float*>(workspace), st, &g_launches, c2, saved);
    if (s != GF_OK) return s;
    return launch_result();
}
}  // namespace

gf_status_t gf_wkv6_backward(const void* r, const void* k, const void* v, const void* x, const float* u,
                             const float* state_in, const void* dy, const float* dstate_out, void* dr, void* dk,
                             void* dv, void* dx, float* du, float* dstate_in, int B, int T, int H, int N,
                             void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return backward_bf16(r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, B, T, H, N, workspace,
                         workspace_bytes, stream, false);
}

gf_status_t gf_wkv6_backward_c2(const void* r, const void* k, const void* v, const void* x, const float* state_in,
                                const void* dy, const float* dstate_out, void* dr, void* dk, void* dv, void* dx,
                                float* dstate_in, int B, int T, int H, int N, void* workspace, size_t workspace_bytes,
                                gf_stream_t stream)
{
    return backward_bf16(r, k, v, x, nullptr, state_in, dy, dstate_out, dr, dk, dv, dx, nullptr, dstate_in, B, T, H, N,
                         workspace, workspace_bytes, stream, true);
}

gf_status_t gf_wkv6_backward_saved(const void* r, const void* k, const void* v, const void* x, const float* u,
                                   const float* state_in, const void* dy, const float* dstate_out, void* dr, void* dk,
                                   void* dv, void* dx, float* du, float* dstate_in, int B, int T, int H, int N,
                                   void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return backward_bf16(r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, B, T, H, N, workspace,
                         workspace_bytes, stream, false, true);
}

gf_status_t gf_wkv6_backward_c2_saved(const void* r, const void* k, const void* v, const void* x, const float* state_in,
                                      const void* dy, const float* dstate_out, void* dr, void* dk, void* dv, void* dx,
                                      float* dstate_in, int B, int T, int H, int N, void* workspace,
                                      size_t workspace_bytes, gf_stream_t stream)
{
    return backward_bf16(r, k, v, x, nullptr, state_in, dy, dstate_out, dr, dk, dv, dx, nullptr, dstate_in, B, T, H, N,
                         workspace, workspace_bytes, stream, true, true);
}

size_t gf_wkv6_backward_varlen_workspace_bytes(int S, int total_T, int H, int N)
{
    if (S <= 0 || total_T < 0 || H <= 0 || N != 64) return 0;
    const int n_sm = gf::sm_count();
    if (n_sm <= 0) return 0;
    return gf::chunked_backward_varlen_workspace_bytes(S, total_T, H, n_sm);
}

namespace {
// bf16 gradient over packed sequences, classic (u, du given) or Finch-C2 form (c2: no bonus)
gf_status_t backward_varlen_bf16(const void* r, const void* k, const void* v, const void* x, const float* u,
                                 const float* state_in, const void* dy, const float* dstate_out, void* dr, void* dk,
                                 void* dv, void* dx, float* du, float* dstate_in, const int32_t* cu_seqlens, int S,
                                 int total_T, int max_seqlen, int H, int N, void* workspace, size_t workspace_bytes,
                                 gf_stream_t stream, bool c2, bool saved = false)
{
    using bf = __nv_bfloat16;
    if (S < 0 || total_T < 0 || max_seqlen < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (S == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t sbytes = (size_t)S * H * 64 * 64 * sizeof(float);
    if (dstate_in && dstate_in == dstate_out) return GF_ERR_INVALID_ARG;
    if (total_T == 0) {
        // no token in any sequence: the state adjoints pass through and the bonus gets no gradient
        if (misaligned(dstate_out) || misaligned(dstate_in) || misaligned(du)) return GF_ERR_INVALID_ARG;
        cudaError_t e = cudaSuccess;
        if (dstate_in && !dstate_out) e = cudaMemsetAsync(dstate_in, 0, sbytes, st);
        else if (dstate_in) e = cudaMemcpyAsync(dstate_in, dstate_out, sbytes, cudaMemcpyDeviceToDevice, st);
        if (e == cudaSuccess && du) e = cudaMemsetAsync(du, 0, (size_t)H * 64 * sizeof(float), st);
        return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
    }
    if (!r || !k || !v || !x || !dy || !dr || !dk || !dv || !dx || !cu_seqlens || (!c2 && (!u || !du))) return GF_ERR_INVALID_ARG;
    if (max_seqlen == 0) return GF_ERR_INVALID_ARG;                  // (tokens exist, so some sequence is longer)
    const void* ptrs[] = {r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, workspace};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(cu_seqlens) % alignof(int32_t)) return GF_ERR_INVALID_ARG;
    const void* ins[] = {r, k, v, x, dy};
    const void* outs[] = {dr, dk, dv, dx};
    for (const void* o : outs)
        for (const void* in : ins)
            if (o == in) return GF_ERR_INVALID_ARG;
    if ((long long)S * H > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    if ((long long)total_T >= (1LL << 31) - 64) return GF_ERR_UNSUPPORTED;
    const size_t need = gf_wkv6_backward_varlen_workspace_bytes(S, total_T, H, N);
    if (need == 0) return GF_ERR_CUDA;
    if (!workspace || workspace_bytes < need) return GF_ERR_WORKSPACE;
    const gf_status_t s = gf::chunked_backward((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, (const bf*)dy,
                                               dstate_out, (bf*)dr, (bf*)dk, (bf*)dv, (bf*)dx, du, dstate_in, S, max_seqlen, H,
                                               static_cast<float*>(workspace), st, &g_launches, c2, saved, cu_seqlens, total_T);
    if (s != GF_OK) return s;
    return launch_result();
}
}  // namespace

gf_status_t gf_wkv6_backward_varlen(const void* r, const void* k, const void* v, const void* x, const float* u,
                                    const float* state_in, const void* dy, const float* dstate_out, void* dr, void* dk,
                                    void* dv, void* dx, float* du, float* dstate_in, const int32_t* cu_seqlens, int S,
                                    int total_T, int max_seqlen, int H, int N, void* workspace, size_t workspace_bytes,
                                    gf_stream_t stream)
{
    return backward_varlen_bf16(r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, cu_seqlens, S,
                                total_T, max_seqlen, H, N, workspace, workspace_bytes, stream, false);
}

gf_status_t gf_wkv6_backward_varlen_c2(const void* r, const void* k, const void* v, const void* x, const float* state_in,
                                       const void* dy, const float* dstate_out, void* dr, void* dk, void* dv, void* dx,
                                       float* dstate_in, const int32_t* cu_seqlens, int S, int total_T, int max_seqlen,
                                       int H, int N, void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return backward_varlen_bf16(r, k, v, x, nullptr, state_in, dy, dstate_out, dr, dk, dv, dx, nullptr, dstate_in,
                                cu_seqlens, S, total_T, max_seqlen, H, N, workspace, workspace_bytes, stream, true);
}

gf_status_t gf_wkv6_backward_varlen_saved(const void* r, const void* k, const void* v, const void* x, const float* u,
                                          const float* state_in, const void* dy, const float* dstate_out, void* dr,
                                          void* dk, void* dv, void* dx, float* du, float* dstate_in,
                                          const int32_t* cu_seqlens, int S, int total_T, int max_seqlen, int H, int N,
                                          void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return backward_varlen_bf16(r, k, v, x, u, state_in, dy, dstate_out, dr, dk, dv, dx, du, dstate_in, cu_seqlens, S,
                                total_T, max_seqlen, H, N, workspace, workspace_bytes, stream, false, true);
}

gf_status_t gf_wkv6_backward_varlen_c2_saved(const void* r, const void* k, const void* v, const void* x,
                                             const float* state_in, const void* dy, const float* dstate_out, void* dr,
                                             void* dk, void* dv, void* dx, float* dstate_in, const int32_t* cu_seqlens,
                                             int S, int total_T, int max_seqlen, int H, int N, void* workspace,
                                             size_t workspace_bytes, gf_stream_t stream)
{
    return backward_varlen_bf16(r, k, v, x, nullptr, state_in, dy, dstate_out, dr, dk, dv, dx, nullptr, dstate_in,
                                cu_seqlens, S, total_T, max_seqlen, H, N, workspace, workspace_bytes, stream, true, true);
}

namespace {
// forward pass of a training step over packed sequences: the packed prefill that also leaves its chunk-start states
// (packed layout) in the packed gradient's workspace; one CTA per sequence and head, never split
gf_status_t prefill_varlen_train(const void* r, const void* k, const void* v, const void* x, const float* u,
                                 const void* u2, const float* state_in, float* state_out, void* y,
                                 const int32_t* cu_seqlens, int S, int total_T, int max_seqlen, int H, int N,
                                 void* workspace, size_t workspace_bytes, gf_stream_t stream, bool c2)
{
    using bf = __nv_bfloat16;
    if (S < 0 || total_T < 0 || max_seqlen < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (S == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (total_T == 0) return pass_state(state_in, state_out, (size_t)S * H, st);
    if (!r || !k || !v || !x || !y || !cu_seqlens || (!c2 && !u) || max_seqlen == 0) return GF_ERR_INVALID_ARG;
    const void* ptrs[] = {r, k, v, x, u, u2, state_in, state_out, y, workspace};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(cu_seqlens) % alignof(int32_t)) return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x || (u2 && y == u2)) return GF_ERR_INVALID_ARG;
    if ((long long)S * H > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    if ((long long)total_T >= (1LL << 31) - 64) return GF_ERR_UNSUPPORTED;
    const size_t need = gf_wkv6_backward_varlen_workspace_bytes(S, total_T, H, N);
    if (need == 0) return GF_ERR_CUDA;
    if (!workspace || workspace_bytes < need) return GF_ERR_WORKSPACE;
    const gf_status_t s = gf::chunked_prefill((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out,
                                              (bf*)y, cu_seqlens, S, max_seqlen, total_T, H, st, &g_launches, nullptr, 0,
                                              (const bf*)u2, c2 ? 1 : 0, static_cast<float*>(workspace));
    if (s != GF_OK) return s;
    return launch_result();
}
}  // namespace

gf_status_t gf_wkv6_prefill_varlen_train(const void* r, const void* k, const void* v, const void* x, const float* u,
                                         const float* state_in, float* state_out, void* y, const int32_t* cu_seqlens,
                                         int S, int total_T, int max_seqlen, int H, int N, void* workspace,
                                         size_t workspace_bytes, gf_stream_t stream)
{
    return prefill_varlen_train(r, k, v, x, u, nullptr, state_in, state_out, y, cu_seqlens, S, total_T, max_seqlen, H, N,
                                workspace, workspace_bytes, stream, false);
}

gf_status_t gf_wkv6_prefill_varlen_c2_train(const void* r, const void* k, const void* v, const void* x, const void* u2,
                                            const float* state_in, float* state_out, void* y, const int32_t* cu_seqlens,
                                            int S, int total_T, int max_seqlen, int H, int N, void* workspace,
                                            size_t workspace_bytes, gf_stream_t stream)
{
    return prefill_varlen_train(r, k, v, x, nullptr, u2, state_in, state_out, y, cu_seqlens, S, total_T, max_seqlen, H, N,
                                workspace, workspace_bytes, stream, true);
}

namespace {
// forward pass of a training step: the prefill that also leaves its chunk-start states in the gradient's workspace
gf_status_t prefill_train(const void* r, const void* k, const void* v, const void* x, const float* u, const void* u2,
                          const float* state_in, float* state_out, void* y, int B, int T, int H, int N, void* workspace,
                          size_t workspace_bytes, gf_stream_t stream, bool c2)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (B == 0 || H == 0) return GF_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (T == 0) return pass_state(state_in, state_out, (size_t)B * H, st);
    if (!r || !k || !v || !x || !y || (!c2 && !u)) return GF_ERR_INVALID_ARG;
    const void* ptrs[] = {r, k, v, x, u, u2, state_in, state_out, y, workspace};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    if (y == r || y == k || y == v || y == x || (u2 && y == u2)) return GF_ERR_INVALID_ARG;
    if ((long long)B * H > 0x7fffffffLL) return GF_ERR_INVALID_ARG;
    if ((long long)B * T >= (1LL << 31) - 64) return GF_ERR_UNSUPPORTED;
    const size_t need = gf_wkv6_backward_bf16_workspace_bytes(B, T, H, N);
    if (need == 0) return GF_ERR_CUDA;
    if (!workspace || workspace_bytes < need) return GF_ERR_WORKSPACE;
    size_t sbytes = 0;
    float* scratch = gf::backward_workspace_forward_scratch(static_cast<float*>(workspace), (long long)B * H, T, gf::sm_count(), &sbytes);
    const gf_status_t s = gf::chunked_prefill((const bf*)r, (const bf*)k, (const bf*)v, (const bf*)x, u, state_in, state_out,
                                              (bf*)y, nullptr, B, T, (long long)B * T, H, st, &g_launches, scratch, sbytes,
                                              (const bf*)u2, c2 ? 1 : 0, static_cast<float*>(workspace));
    if (s != GF_OK) return s;
    return launch_result();
}
}  // namespace

gf_status_t gf_wkv6_prefill_train(const void* r, const void* k, const void* v, const void* x, const float* u,
                                  const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                                  void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return prefill_train(r, k, v, x, u, nullptr, state_in, state_out, y, B, T, H, N, workspace, workspace_bytes, stream, false);
}

gf_status_t gf_wkv6_prefill_c2_train(const void* r, const void* k, const void* v, const void* x, const void* u2,
                                     const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                                     void* workspace, size_t workspace_bytes, gf_stream_t stream)
{
    return prefill_train(r, k, v, x, nullptr, u2, state_in, state_out, y, B, T, H, N, workspace, workspace_bytes, stream, true);
}

size_t gf_wkv6_host_workspace_bytes(int B, int T, int H, int N)
{
    if (B < 0 || T < 0 || H < 0 || N < 0) return 0;
    const size_t tok = (size_t)B * T * H * N * 2;                 // one bf16 tensor
    const size_t pad = 256;
    auto up = [&](size_t b) { return (b + pad - 1) / pad * pad; };
    return 5 * up(tok) + up((size_t)H * N * 4) + 2 * up((size_t)B * H * N * N * 4);
}

gf_status_t gf_wkv6_prefill_host(const void* r, const void* k, const void* v, const void* x, const float* u,
                                 const float* state_in, float* state_out, void* y, int B, int T, int H, int N,
                                 void* dev_ws, size_t dev_ws_bytes, gf_stream_t stream)
{
    if (B < 0 || T < 0 || H < 0 || N < 0) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    if (!r || !k || !v || !x || !u || !y) return GF_ERR_INVALID_ARG;
    if (!dev_ws || (reinterpret_cast<uintptr_t>(dev_ws) & 255u)) return GF_ERR_INVALID_ARG;
    if (dev_ws_bytes < gf_wkv6_host_workspace_bytes(B, T, H, N)) return GF_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t tok = (size_t)B * T * H * N * 2, ub = (size_t)H * N * 4, sb = (size_t)B * H * N * N * 4;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    char* p = static_cast<char*>(dev_ws);
    char* d_r = p; p += up(tok);
    char* d_k = p; p += up(tok);
    char* d_v = p; p += up(tok);
    char* d_x = p; p += up(tok);
    char* d_y = p; p += up(tok);
    float* d_u = reinterpret_cast<float*>(p); p += up(ub);
    float* d_si = reinterpret_cast<float*>(p); p += up(sb);
    float* d_so = reinterpret_cast<float*>(p);
    bool ok = true;
    auto h2d = [&](void* d, const void* h, size_t n) {
        if (n) ok = ok && cudaMemcpyAsync(d, h, n, cudaMemcpyHostToDevice, st) == cudaSuccess;
    };
    h2d(d_r, r, tok); h2d(d_k, k, tok); h2d(d_v, v, tok); h2d(d_x, x, tok); h2d(d_u, u, ub);
    if (state_in) h2d(d_si, state_in, sb);
    if (!ok) return GF_ERR_CUDA;
    gf_status_t s = gf_wkv6_prefill(d_r, d_k, d_v, d_x, d_u, state_in ? d_si : nullptr,
                                    state_out ? d_so : nullptr, d_y, B, T, H, N, stream);
    if (s != GF_OK) return s;
    if (tok) ok = ok && cudaMemcpyAsync(y, d_y, tok, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (state_out && sb) ok = ok && cudaMemcpyAsync(state_out, d_so, sb, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    return ok ? GF_OK : GF_ERR_CUDA;
}

size_t gf_wkv6_workspace_bytes(int B, int T, int H, int N)
{
    if (B <= 0 || T <= 0 || H <= 0 || N != 64) return 0;
    int seg_chunks = 0;
    size_t need = 0;
    gf::choose_split((long long)B * H, T, gf::sm_count(), &seg_chunks, &need);
    // a packed call with more units than SMs draws its units, longest sequences first, from a counter in the workspace
    if (need == 0 && (long long)B * H > gf::sm_count()) need = (gf::persistent_scratch_bytes(B) + 255) / 256 * 256;
    return need;
}

gf_status_t gf_wkv6_split_plan(int B, int T, int H, int N, int n_sm, size_t scratch_cap, int* nseg, int* seg_chunks,
                               size_t* scratch_bytes)
{
    if (B < 0 || T < 0 || H < 0 || n_sm <= 0 || !nseg || !seg_chunks || !scratch_bytes) return GF_ERR_INVALID_ARG;
    if (N != 64) return GF_ERR_UNSUPPORTED;
    *nseg = gf::choose_split((long long)B * H, T, n_sm, seg_chunks, scratch_bytes, scratch_cap ? scratch_cap : ~(size_t)0);
    return GF_OK;
}

gf_status_t gf_wkv6_set_workspace(void* dev_ptr, size_t bytes)
{
    if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255u)) return GF_ERR_INVALID_ARG;
    g_ws_bytes.store(0, std::memory_order_relaxed);
    g_ws.store(static_cast<float*>(dev_ptr), std::memory_order_relaxed);
    g_ws_bytes.store(dev_ptr ? bytes : 0, std::memory_order_relaxed);
    return GF_OK;
}

gf_status_t gf_wkv6_set_kernel(gf_kernel_t kernel)
{
    if (kernel != GF_KERNEL_AUTO && kernel != GF_KERNEL_EXACT && kernel != GF_KERNEL_CHUNKED)
        return GF_ERR_UNSUPPORTED;
    g_kernel.store((int)kernel, std::memory_order_relaxed);
    return GF_OK;
}

gf_status_t gf_wkv6_last_device_status(gf_stream_t stream)
{
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GF_ERR_CUDA;
    int flag = 0;
    if (gf::read_and_clear_device_status(&flag) != cudaSuccess) return GF_ERR_CUDA;
    return flag ? GF_ERR_TIMEOUT : GF_OK;
}

gf_status_t gf_wkv6_set_wait_limit(unsigned int microseconds)
{
    gf::wait_limit_us().store(microseconds, std::memory_order_relaxed);
    return GF_OK;
}

gf_status_t gf_wkv6_selftest_wait_timeout(unsigned int microseconds, gf_stream_t stream)
{
    if (microseconds == 0 || microseconds > 1000000u) return GF_ERR_INVALID_ARG;     // one second at most
    gf::ck::wait_timeout_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(microseconds);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return launch_result();
}

uint64_t gf_wkv6_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

gf_status_t gf_c2_layernorm(const void* y, const float* gamma, const float* beta, float eps, void* out,
                            long long rows, int H, int N, gf_stream_t stream)
{
    return layernorm_call(static_cast<const __nv_bfloat16*>(y), gamma, beta, eps, static_cast<__nv_bfloat16*>(out), rows, H, N, stream);
}

gf_status_t gf_c2_layernorm_f32(const float* y, const float* gamma, const float* beta, float eps, float* out,
                                long long rows, int H, int N, gf_stream_t stream)
{
    return layernorm_call(y, gamma, beta, eps, out, rows, H, N, stream);
}

gf_status_t gf_gold_key_compress(const void* x, const void* w_kd, void* c, long long rows, int D, int Dc, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (rows < 0 || D < 0 || Dc < 0) return GF_ERR_INVALID_ARG;
    if (rows == 0 || Dc == 0) return GF_OK;
    if (D == 0 || (D & 7) || (Dc & 7) || Dc > 256) return GF_ERR_UNSUPPORTED;
    if (rows >= (1LL << 31) - 256) return GF_ERR_INVALID_ARG;
    if (!x || !w_kd || !c || misaligned(x) || misaligned(w_kd) || misaligned(c) || c == x || c == w_kd) return GF_ERR_INVALID_ARG;
    return gf::key_compress((const bf*)x, (const bf*)w_kd, (bf*)c, rows, D, Dc, (cudaStream_t)stream, &g_launches);
}

gf_status_t gf_c2_decay_logit(const void* x, const void* x_prev, const float* mu_x, const void* A_d, const void* B_d,
                              const float* lambda_d, const void* A_w, const void* B_w, const float* lambda_w, void* d,
                              int B, int T, int D, int Rd, int Rw, gf_stream_t stream)
{
    using bf = __nv_bfloat16;
    if (B < 0 || T < 0 || D < 0 || Rd < 0 || Rw < 0) return GF_ERR_INVALID_ARG;
    if (B == 0 || T == 0 || D == 0) return GF_OK;
    if ((D & 63) || Rd == 0 || Rw == 0 || (Rd & 15) || (Rw & 15) || Rd > 64 || Rw > 64) return GF_ERR_UNSUPPORTED;
    if ((long long)B * T >= (1LL << 31) - 128) return GF_ERR_INVALID_ARG;
    if (!x || !mu_x || !A_d || !B_d || !lambda_d || !A_w || !B_w || !lambda_w || !d || d == x) return GF_ERR_INVALID_ARG;
    const void* ptrs[] = {x, x_prev, mu_x, A_d, B_d, lambda_d, A_w, B_w, lambda_w, d};
    for (const void* q : ptrs)
        if (misaligned(q)) return GF_ERR_INVALID_ARG;
    return gf::decay_logit((const bf*)x, (const bf*)x_prev, mu_x, (const bf*)A_d, (const bf*)B_d, lambda_d, (const bf*)A_w,
                           (const bf*)B_w, lambda_w, (bf*)d, B, T, D, Rd, Rw, (cudaStream_t)stream, &g_launches);
}

const char* gf_status_string(gf_status_t s)
{
    switch (s) {
    case GF_OK: return "ok";
    case GF_ERR_INVALID_ARG: return "invalid argument";
    case GF_ERR_UNSUPPORTED: return "unsupported configuration";
    case GF_ERR_CUDA: return "CUDA error";
    case GF_ERR_WORKSPACE: return "workspace too small";
    case GF_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

int gf_wkv6_version(void) { return 100; }

}  // extern "C"
