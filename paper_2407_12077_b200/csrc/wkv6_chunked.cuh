// Chunked tensor-core WKV-6 prefill for sm_100a.
//
// One CTA per (sequence, head) walks the sequence in chunks of L = 64 tokens.  With the
// in-chunk inclusive cumulative log2-decay a_t = sum_{s<=t} log2 w_s (a_0 = 0, fp32, restarted
// every chunk) and the chunk's start state S_0, the recurrence re-associates exactly to
//   y_t  = (r_t * 2^{a_{t-1}}) . S_0 + sum_{i<t} P[t,i] v_i + (sum_c r_t[c] u[c] k_t[c]) v_t
//   P[t,i] = sum_c (r_t[c] 2^{a_{t-1}[c]}) (k_i[c] 2^{-a_i[c]})
//   S_L  = diag(2^{a_L}) ( S_0 + sum_i (k_i * 2^{-a_i})^T v_i )
// so a chunk is four 64x64x64 contractions on bf16 tensor cores (fp32 accumulate) around an
// fp32 elementwise phase.  The single in-chunk reference point is safe while no channel decays
// by more than 2^-96 inside one chunk (always true for w >= 0.36; the benchmark's decays are
// >= 0.69); a chunk that violates it is processed token by token in fp32 instead, so any finite
// or infinite decay logit gives the exact-recurrence result.
//
// Warp roles (544 threads), pipelined across chunks through mbarriers:
//   warp 0      TMA producer: r,k,x tiles (3-stage ring) and v tiles (5-stage ring), 128B swizzle
//   warps 1-8   elementwise: decay, cumulative sum, scaled bf16 operands R^ = r 2^{a_{t-1}},
//               K^ = k 2^{-a_t}, chunk decay 2^{a_L}, bonus coefficients, safety vote
//   warps 9-12  scores: P = tril(R^ K^T, -1) + diag(bonus) -> bf16 tile
//   warps 13-16 state/output: hold S^T in mma accumulators for the whole sequence;
//               Y^T = S^T R^^T + V^T P^T, S^T <- (S^T + V^T K^) diag(2^{a_L}); y staged through
//               shared memory and written with TMA
// Every wait is bounded: on expiry the kernel raises a status flag and all roles leave.
#pragma once
#include <atomic>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gf_wkv6.h"

namespace gf {

__device__ int g_dev_status = 0;

inline cudaError_t read_and_clear_device_status(int* flag)
{
    cudaError_t e = cudaMemcpyFromSymbol(flag, g_dev_status, sizeof(int));
    if (e != cudaSuccess) return e;
    if (*flag) {
        int z = 0;
        e = cudaMemcpyToSymbol(g_dev_status, &z, sizeof(int));
    }
    return e;
}

namespace ck {

constexpr int L = 64;                  // tokens per chunk
constexpr int TILE = 64 * 64 * 2;      // one bf16 [64 x 64] tile
constexpr int NSTAGE_A = 3;            // r,k,x ring depth
constexpr int NSTAGE_V = 5;            // v ring depth
constexpr int NBUF_RK = 2;             // scaled-operand buffers
constexpr int NBUF_P = 2;
constexpr int NBUF_Y = 2;
constexpr int N_EW = 8;                // elementwise warps
constexpr int THREADS = 32 * (1 + N_EW + 4 + 4);
constexpr float A2_MAX = 96.f;         // largest in-chunk |cumulative log2 decay| on the tensor-core path
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LOG2_LOG2E = 0.5287663729448977f;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_A = 0;                                   // [NSTAGE_A][3][TILE]  r,k,x
constexpr int OFF_V = OFF_A + NSTAGE_A * 3 * TILE;         // [NSTAGE_V][TILE]
constexpr int OFF_RK = OFF_V + NSTAGE_V * TILE;            // [NBUF_RK][2][TILE]   R^, K^
constexpr int OFF_P = OFF_RK + NBUF_RK * 2 * TILE;         // [NBUF_P][TILE]
constexpr int OFF_Y = OFF_P + NBUF_P * TILE;               // [NBUF_Y][TILE]
constexpr int OFF_DL = OFF_Y + NBUF_Y * TILE;              // [NBUF_RK][64] float  2^{a_L}
constexpr int OFF_DU = OFF_DL + NBUF_RK * 64 * 4;          // [NBUF_RK][64] float  bonus coefficient per token
constexpr int OFF_TOT = OFF_DU + NBUF_RK * 64 * 4;         // [2][N_EW][64] float  per-warp decay totals
constexpr int OFF_SAFE = OFF_TOT + 2 * N_EW * 64 * 4;      // [NBUF_RK] int
constexpr int OFF_ABORT = OFF_SAFE + 16;                   // int
constexpr int OFF_BAR = OFF_ABORT + 16;                    // mbarriers (8 bytes each)
enum {
    BAR_FULL_A = 0,
    BAR_EMPTY_A = BAR_FULL_A + NSTAGE_A,
    BAR_FULL_V = BAR_EMPTY_A + NSTAGE_A,
    BAR_EMPTY_V = BAR_FULL_V + NSTAGE_V,
    BAR_RK_READY = BAR_EMPTY_V + NSTAGE_V,
    BAR_RK_FREE = BAR_RK_READY + NBUF_RK,
    BAR_P_READY = BAR_RK_FREE + NBUF_RK,
    BAR_P_FREE = BAR_P_READY + NBUF_P,
    BAR_ESYNC = BAR_P_FREE + NBUF_P,
    BAR_YSYNC = BAR_ESYNC + 1,          // two of them
    BAR_COUNT = BAR_YSYNC + 2
};
constexpr int SMEM_BYTES = OFF_BAR + BAR_COUNT * 8;
constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;              // slack for manual 1024-byte alignment

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait.  Returns false if the CTA is aborting or the wait ran out of time (the
// status flag is then raised and the CTA-wide abort flag set so every role leaves).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, bool poll_abort)
{
    const unsigned long long t0 = globaltimer();
    for (;;) {
        for (int it = 0; it < 64; ++it)
            if (mbar_try_wait(bar, parity)) return true;
        if (poll_abort && *abort_flag) return false;
        if (globaltimer() - t0 > WAIT_LIMIT_NS) break;
        __nanosleep(64);
    }
    *abort_flag = 1;
    atomicExch(&g_dev_status, 1);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, bool poll_abort = true)
{
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, poll_abort);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, int c0, int c1, uint32_t src)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(tm), "r"(c0), "r"(c1), "r"(src) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void sts128z(uint32_t a)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0u) : "memory");
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&p);
}
// byte offset of (row, byte-in-row) inside a 128B-swizzled [64 x 128 B] tile
__device__ __forceinline__ uint32_t swz(int row, int byte) { return (uint32_t)(row * 128 + (byte ^ ((row & 7) << 4))); }

__device__ __forceinline__ void ldsm_x4(uint32_t a, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t a, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ __forceinline__ void stsm_x4_t(uint32_t a, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1,%2,%3,%4};"
                 ::"r"(a), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
}
// D(16x8, fp32) += A(16x16, bf16 row) * B(16x8, bf16 col)
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

struct Params {
    const __nv_bfloat16 *r, *k, *v, *x;   // raw pointers, used only by the token-by-token path
    __nv_bfloat16* y;
    const float* u;
    const float* state_in;
    float* state_out;
    const int32_t* cu_seqlens;             // nullptr: dense
    int T;                                 // dense sequence length
    int H;
};

// ---------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(THREADS, 1)
wkv6_chunked_kernel(const __grid_constant__ CUtensorMap tm_r, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_x,
                    const __grid_constant__ CUtensorMap tm_y, const Params p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_ABORT);
    volatile int* safe_flag = reinterpret_cast<volatile int*>(smem + OFF_SAFE);
    auto bar = [&](int i) { return sbase + OFF_BAR + 8 * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int unit = blockIdx.x;
    const int seq = unit / p.H, h = unit % p.H;
    long long row0;
    int len;
    if (p.cu_seqlens) {
        row0 = p.cu_seqlens[seq];
        len = p.cu_seqlens[seq + 1] - p.cu_seqlens[seq];
    } else {
        row0 = (long long)seq * p.T;
        len = p.T;
    }
    const int nchunks = (len + L - 1) / L;
    const int col0 = h * 64;
    const size_t C = (size_t)p.H * 64;

    if (tid == 0) {
        for (int i = 0; i < NSTAGE_A; ++i) { mbar_init(bar(BAR_FULL_A + i), 1); mbar_init(bar(BAR_EMPTY_A + i), N_EW); }
        for (int i = 0; i < NSTAGE_V; ++i) { mbar_init(bar(BAR_FULL_V + i), 1); mbar_init(bar(BAR_EMPTY_V + i), 4); }
        for (int i = 0; i < NBUF_RK; ++i) { mbar_init(bar(BAR_RK_READY + i), N_EW); mbar_init(bar(BAR_RK_FREE + i), 8); }
        for (int i = 0; i < NBUF_P; ++i) { mbar_init(bar(BAR_P_READY + i), 4); mbar_init(bar(BAR_P_FREE + i), 4); }
        mbar_init(bar(BAR_ESYNC), N_EW);
        mbar_init(bar(BAR_YSYNC), 4);
        mbar_init(bar(BAR_YSYNC + 1), 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    if (warp == 0) {
        // ============================== TMA producer ==============================
        if (lane == 0) {
            int issued = 0;
            for (int c = 0; c < nchunks; ++c) {
                const int sa = c % NSTAGE_A, sv = c % NSTAGE_V;
                const int row = (int)(row0 + (long long)c * L);
                if (c >= NSTAGE_A && !mbar_wait(bar(BAR_EMPTY_A + sa), ((c / NSTAGE_A) & 1) ^ 1, abort_flag)) break;
                if (c >= NSTAGE_V && !mbar_wait(bar(BAR_EMPTY_V + sv), ((c / NSTAGE_V) & 1) ^ 1, abort_flag)) break;
                const uint32_t dstA = sbase + OFF_A + sa * 3 * TILE;
                mbar_expect_tx(bar(BAR_FULL_A + sa), 3 * TILE);
                tma_load_2d(dstA, &tm_x, col0, row, bar(BAR_FULL_A + sa));
                tma_load_2d(dstA + TILE, &tm_r, col0, row, bar(BAR_FULL_A + sa));
                tma_load_2d(dstA + 2 * TILE, &tm_k, col0, row, bar(BAR_FULL_A + sa));
                mbar_expect_tx(bar(BAR_FULL_V + sv), TILE);
                tma_load_2d(sbase + OFF_V + sv * TILE, &tm_v, col0, row, bar(BAR_FULL_V + sv));
                issued = c + 1;
            }
            // do not leave while copies into this CTA's shared memory may still be in flight
            for (int c = max(0, issued - NSTAGE_A); c < issued; ++c)
                mbar_wait(bar(BAR_FULL_A + c % NSTAGE_A), (c / NSTAGE_A) & 1, abort_flag, false);
            for (int c = max(0, issued - NSTAGE_V); c < issued; ++c)
                mbar_wait(bar(BAR_FULL_V + c % NSTAGE_V), (c / NSTAGE_V) & 1, abort_flag, false);
        }
    } else if (warp <= N_EW) {
        // ============================== elementwise warps ==============================
        const int tq = warp - 1;                 // tokens 8*tq .. 8*tq+7 of the chunk
        const int cb = lane * 4;                 // byte column of this lane's channel pair (2*lane, 2*lane+1)
        const float2 u2 = *reinterpret_cast<const float2*>(p.u + h * 64 + 2 * lane);
        float* tot = reinterpret_cast<float*>(smem + OFF_TOT);
        for (int c = 0; c < nchunks; ++c) {
            const int sa = c % NSTAGE_A, b = c % NBUF_RK;
            const int valid = min(L, len - c * L);
            const uint32_t tx = sbase + OFF_A + sa * 3 * TILE, tr = tx + TILE, tk = tx + 2 * TILE;
            if (!mbar_wait(bar(BAR_FULL_A + sa), (c / NSTAGE_A) & 1, abort_flag)) break;
            // ---- phase A: log2-decay magnitudes and the warp-local cumulative sums
            float l0[8], l1[8];
            {
                float a0 = 0.f, a1 = 0.f;
#pragma unroll
                for (int tt = 0; tt < 8; ++tt) {
                    const int t = 8 * tq + tt;
                    const uint32_t xw = lds32(tx + swz(t, cb));
                    float e0 = ex2(fmaf(bf_lo(xw), LOG2E, LOG2_LOG2E));
                    float e1 = ex2(fmaf(bf_hi(xw), LOG2E, LOG2_LOG2E));
                    if (t >= valid) { e0 = 0.f; e1 = 0.f; }
                    a0 -= e0; a1 -= e1;
                    l0[tt] = a0; l1[tt] = a1;
                }
            }
            float* totc = tot + (c & 1) * (N_EW * 64);
            *reinterpret_cast<float2*>(totc + tq * 64 + 2 * lane) = make_float2(l0[7], l1[7]);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_ESYNC));
            if (!mbar_wait(bar(BAR_ESYNC), c & 1, abort_flag)) break;
            float off0 = 0.f, off1 = 0.f;
            for (int q = 0; q < tq; ++q) {
                const float2 t2 = *reinterpret_cast<const float2*>(totc + q * 64 + 2 * lane);
                off0 += t2.x; off1 += t2.y;
            }
            if (c >= NBUF_RK && !mbar_wait(bar(BAR_RK_FREE + b), ((c / NBUF_RK) & 1) ^ 1, abort_flag)) break;
            // ---- phase B: scaled operands R^ = r 2^{a_{t-1}}, K^ = k 2^{-a_t}; bonus partials
            const uint32_t trh = sbase + OFF_RK + b * 2 * TILE, tkh = trh + TILE;
            float du[8];
#pragma unroll
            for (int tt = 0; tt < 8; ++tt) {
                const int t = 8 * tq + tt;
                const float ap0 = off0 + (tt ? l0[tt - 1] : 0.f), ap1 = off1 + (tt ? l1[tt - 1] : 0.f);
                const float ac0 = off0 + l0[tt], ac1 = off1 + l1[tt];
                const uint32_t rw = lds32(tr + swz(t, cb)), kw = lds32(tk + swz(t, cb));
                const float r0 = bf_lo(rw), r1 = bf_hi(rw), k0 = bf_lo(kw), k1 = bf_hi(kw);
                uint32_t rh = pack_bf16(r0 * ex2(ap0), r1 * ex2(ap1));
                uint32_t kh = pack_bf16(k0 * ex2(-ac0), k1 * ex2(-ac1));
                float d = fmaf(r0 * k0, u2.x, r1 * k1 * u2.y);
                if (t >= valid) { rh = 0u; kh = 0u; d = 0.f; }
                sts32(trh + swz(t, cb), rh);
                sts32(tkh + swz(t, cb), kh);
                du[tt] = d;
            }
            // reduce the 8 bonus partials over the 32 lanes (transposing butterfly): lane 4m ends with token m
            {
                const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
                float w4[4], w2[2], w1;
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const float send = h16 ? du[m] : du[m + 4], keep = h16 ? du[m + 4] : du[m];
                    w4[m] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
                }
#pragma unroll
                for (int m = 0; m < 2; ++m) {
                    const float send = h8 ? w4[m] : w4[m + 2], keep = h8 ? w4[m + 2] : w4[m];
                    w2[m] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
                }
                {
                    const float send = h4 ? w2[0] : w2[1], keep = h4 ? w2[1] : w2[0];
                    w1 = keep + __shfl_xor_sync(0xffffffffu, send, 4);
                }
                w1 += __shfl_xor_sync(0xffffffffu, w1, 2);
                w1 += __shfl_xor_sync(0xffffffffu, w1, 1);
                if ((lane & 3) == 0)
                    reinterpret_cast<float*>(smem + OFF_DU)[b * 64 + 8 * tq + (lane >> 2)] = w1;
            }
            if (tq == N_EW - 1) {
                const float aL0 = off0 + l0[7], aL1 = off1 + l1[7];
                *reinterpret_cast<float2*>(reinterpret_cast<float*>(smem + OFF_DL) + b * 64 + 2 * lane) =
                    make_float2(ex2(aL0), ex2(aL1));
                const bool ok = (aL0 >= -A2_MAX) && (aL1 >= -A2_MAX);       // false for NaN as well
                const bool all_ok = __all_sync(0xffffffffu, ok);
                if (lane == 0) safe_flag[b] = all_ok ? 1 : 0;
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(BAR_EMPTY_A + sa));
                mbar_arrive(bar(BAR_RK_READY + b));
            }
        }
    } else if (warp <= N_EW + 4) {
        // ============================== score warps ==============================
        const int pw = warp - (N_EW + 1);        // rows t = 16*pw .. 16*pw+15
        const int g = lane >> 2, q = lane & 3;
        for (int c = 0; c < nchunks; ++c) {
            const int b = c % NBUF_RK, pb = c % NBUF_P;
            if (!mbar_wait(bar(BAR_RK_READY + b), (c / NBUF_RK) & 1, abort_flag)) break;
            if (c >= NBUF_P && !mbar_wait(bar(BAR_P_FREE + pb), ((c / NBUF_P) & 1) ^ 1, abort_flag)) break;
            if (safe_flag[b]) {
                const uint32_t trh = sbase + OFF_RK + b * 2 * TILE, tkh = trh + TILE, tp = sbase + OFF_P + pb * TILE;
                const float* du = reinterpret_cast<const float*>(smem + OFF_DU) + b * 64;
                uint32_t a[4][4];
                {
                    const int row = 16 * pw + (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ldsm_x4(trh + swz(row, 32 * kk + 16 * (lane >> 4)), a[kk][0], a[kk][1], a[kk][2], a[kk][3]);
                }
                for (int ib = 0; ib <= pw; ++ib) {
                    float acc[2][4] = {};
                    const int irow = 16 * ib + (lane & 7) + 8 * (lane >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4(tkh + swz(irow, 32 * kk + 16 * ((lane >> 3) & 1)), b0, b1, b2, b3);
                        mma16816(acc[0], a[kk], b0, b1);
                        mma16816(acc[1], a[kk], b2, b3);
                    }
                    if (ib == pw) {
                        // diagonal 16x16 block: strictly-lower entries stay, the diagonal takes the bonus
                        // coefficient, the upper triangle is zero
                        const float d_lo = du[16 * pw + g], d_hi = du[16 * pw + g + 8];
#pragma unroll
                        for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
                            for (int e = 0; e < 2; ++e) {
                                const int il = 8 * nb + 2 * q + e;
                                acc[nb][e] = il < g ? acc[nb][e] : (il == g ? d_lo : 0.f);
                                acc[nb][2 + e] = il < g + 8 ? acc[nb][2 + e] : (il == g + 8 ? d_hi : 0.f);
                            }
                        }
                    }
#pragma unroll
                    for (int nb = 0; nb < 2; ++nb) {
                        const int colb = (16 * ib + 8 * nb + 2 * q) * 2;
                        sts32(tp + swz(16 * pw + g, colb), pack_bf16(acc[nb][0], acc[nb][1]));
                        sts32(tp + swz(16 * pw + g + 8, colb), pack_bf16(acc[nb][2], acc[nb][3]));
                    }
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(BAR_P_READY + pb));
                mbar_arrive(bar(BAR_RK_FREE + b));
            }
        }
    } else {
        // ============================== state / output warps ==============================
        const int yw = warp - (N_EW + 5);        // value channels j = 16*yw .. 16*yw+15
        const int ytid = tid - 32 * (N_EW + 5);  // 0..127
        const int g = lane >> 2, q = lane & 3;
        const int j0 = 16 * yw + g;
        const size_t sb = (size_t)unit * 4096;
        // S^T[j][c] in accumulator layout: st[n][0..1] = (j0, c = 8n+2q, +1), st[n][2..3] = (j0+8, same c)
        float st[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            const int c0 = 8 * n + 2 * q;
            if (p.state_in) {
                st[n][0] = p.state_in[sb + (size_t)c0 * 64 + j0];
                st[n][1] = p.state_in[sb + (size_t)(c0 + 1) * 64 + j0];
                st[n][2] = p.state_in[sb + (size_t)c0 * 64 + j0 + 8];
                st[n][3] = p.state_in[sb + (size_t)(c0 + 1) * 64 + j0 + 8];
            } else {
                st[n][0] = st[n][1] = st[n][2] = st[n][3] = 0.f;
            }
        }
        int ysync_uses[2] = {0, 0};
        int ybuf_uses = 0;
        bool live = true;
        auto ysync = [&](int which) -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_YSYNC + which));
            const bool ok = mbar_wait(bar(BAR_YSYNC + which), ysync_uses[which] & 1, abort_flag);
            ++ysync_uses[which];
            return ok;
        };
        for (int c = 0; c < nchunks && live; ++c) {
            const int sv = c % NSTAGE_V, b = c % NBUF_RK, pb = c % NBUF_P;
            const int valid = min(L, len - c * L);
            const uint32_t tv = sbase + OFF_V + sv * TILE;
            const uint32_t trh = sbase + OFF_RK + b * 2 * TILE, tkh = trh + TILE, tp = sbase + OFF_P + pb * TILE;
            if (!mbar_wait(bar(BAR_FULL_V + sv), (c / NSTAGE_V) & 1, abort_flag)) break;
            if (!mbar_wait(bar(BAR_RK_READY + b), (c / NBUF_RK) & 1, abort_flag)) break;
            if (!mbar_wait(bar(BAR_P_READY + pb), (c / NBUF_P) & 1, abort_flag)) break;
            if (safe_flag[b]) {
                if (valid < L) {
                    // rows past the end of the sequence hold another sequence's tokens (or fill): zero them
                    for (int i = ytid; i < (L - valid) * 8; i += 128)
                        sts128z(tv + (valid + (i >> 3)) * 128 + ((i & 7) << 4));
                    if (!ysync(0)) break;
                }
                float ya[8][4];
#pragma unroll
                for (int n = 0; n < 8; ++n) ya[n][0] = ya[n][1] = ya[n][2] = ya[n][3] = 0.f;
                // ---- Y^T += S^T R^^T   (M = j, N = t, K = c); A straight from the fp32 accumulators
                {
                    const int trow = (lane & 7) + 8 * (lane >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        uint32_t sa[4];
                        sa[0] = pack_bf16(st[2 * kk][0], st[2 * kk][1]);
                        sa[1] = pack_bf16(st[2 * kk][2], st[2 * kk][3]);
                        sa[2] = pack_bf16(st[2 * kk + 1][0], st[2 * kk + 1][1]);
                        sa[3] = pack_bf16(st[2 * kk + 1][2], st[2 * kk + 1][3]);
#pragma unroll
                        for (int np = 0; np < 4; ++np) {
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4(trh + swz(16 * np + trow, 32 * kk + 16 * ((lane >> 3) & 1)), b0, b1, b2, b3);
                            mma16816(ya[2 * np], sa, b0, b1);
                            mma16816(ya[2 * np + 1], sa, b2, b3);
                        }
                    }
                }
                // ---- V^T fragments (M = j, K = i) from the raw v tile [i][j]
                uint32_t va[4][4];
                {
                    const int irow = (lane & 7) + 8 * (lane >> 4);
                    const int jb = (16 * yw + 8 * ((lane >> 3) & 1)) * 2;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ldsm_x4_t(tv + swz(16 * kk + irow, jb), va[kk][0], va[kk][1], va[kk][2], va[kk][3]);
                }
                // ---- Y^T += V^T P^T   (M = j, N = t, K = i), causal: token block np needs i-steps kk <= np
                {
                    const int trow = (lane & 7) + 8 * (lane >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
                        for (int np = kk; np < 4; ++np) {
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4(tp + swz(16 * np + trow, 32 * kk + 16 * ((lane >> 3) & 1)), b0, b1, b2, b3);
                            mma16816(ya[2 * np], va[kk], b0, b1);
                            mma16816(ya[2 * np + 1], va[kk], b2, b3);
                        }
                    }
                }
                // ---- S^T += V^T K^   (M = j, N = c, K = i), then scale column c by 2^{a_L[c]}
                {
                    const int irow = (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
                        for (int cp2 = 0; cp2 < 4; ++cp2) {
                            uint32_t b0, b1, b2, b3;
                            ldsm_x4_t(tkh + swz(16 * kk + irow, 32 * cp2 + 16 * (lane >> 4)), b0, b1, b2, b3);
                            mma16816(st[2 * cp2], va[kk], b0, b1);
                            mma16816(st[2 * cp2 + 1], va[kk], b2, b3);
                        }
                    }
                    const float* dl = reinterpret_cast<const float*>(smem + OFF_DL) + b * 64;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        const float2 d2 = *reinterpret_cast<const float2*>(dl + 8 * n + 2 * q);
                        st[n][0] *= d2.x; st[n][1] *= d2.y; st[n][2] *= d2.x; st[n][3] *= d2.y;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar(BAR_EMPTY_V + sv));
                    mbar_arrive(bar(BAR_RK_FREE + b));
                    mbar_arrive(bar(BAR_P_FREE + pb));
                }
                // ---- epilogue: Y^T accumulators -> bf16 [t][j] tile -> global
                const uint32_t ty = sbase + OFF_Y + (ybuf_uses % NBUF_Y) * TILE;
                ++ybuf_uses;
                if (ytid == 0) bulk_wait_read<NBUF_Y - 1>();     // the store that last used this buffer has read it
                if (!ysync(0)) break;
#pragma unroll
                for (int np = 0; np < 4; ++np) {
                    const int mi = lane >> 3, rr = lane & 7;
                    const int t = 8 * (2 * np + (mi >> 1)) + rr;
                    stsm_x4_t(ty + swz(t, (2 * yw + (mi & 1)) << 4),
                              pack_bf16(ya[2 * np][0], ya[2 * np][1]), pack_bf16(ya[2 * np][2], ya[2 * np][3]),
                              pack_bf16(ya[2 * np + 1][0], ya[2 * np + 1][1]), pack_bf16(ya[2 * np + 1][2], ya[2 * np + 1][3]));
                }
                fence_proxy_async();
                if (!ysync(1)) break;
                if (valid == L) {
                    if (ytid == 0) {
                        tma_store_2d(&tm_y, col0, (int)(row0 + (long long)c * L), ty);
                        bulk_commit();
                    }
                } else {
                    // ragged tail: the rows after `valid` belong to someone else, so copy row by row
                    for (int i = ytid; i < valid * 8; i += 128) {
                        const int t = i >> 3, ch = i & 7;
                        uint4 val;
                        asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                     : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(ty + swz(t, ch << 4)));
                        *reinterpret_cast<uint4*>(p.y + (size_t)(row0 + (long long)c * L + t) * C + col0 + ch * 8) = val;
                    }
                    if (ytid == 0) bulk_commit();
                }
            } else {
                // ---- decay too strong for one in-chunk reference point: exact fp32 recurrence, token by token
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar(BAR_EMPTY_V + sv));
                    mbar_arrive(bar(BAR_RK_FREE + b));
                    mbar_arrive(bar(BAR_P_FREE + pb));
                }
                const float* ug = p.u + h * 64;
                for (int t = 0; t < valid; ++t) {
                    const size_t ro = (size_t)(row0 + (long long)c * L + t) * C + col0;
                    // bonus coefficient over all 64 channels
                    float cf = __bfloat162float(p.r[ro + lane]) * ug[lane] * __bfloat162float(p.k[ro + lane]) +
                               __bfloat162float(p.r[ro + lane + 32]) * ug[lane + 32] * __bfloat162float(p.k[ro + lane + 32]);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) cf += __shfl_xor_sync(0xffffffffu, cf, o);
                    const float v_lo = __bfloat162float(p.v[ro + j0]), v_hi = __bfloat162float(p.v[ro + j0 + 8]);
                    float y_lo = 0.f, y_hi = 0.f;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        const int c0 = 8 * n + 2 * q;
                        const uint32_t rw = *reinterpret_cast<const uint32_t*>(p.r + ro + c0);
                        const uint32_t kw = *reinterpret_cast<const uint32_t*>(p.k + ro + c0);
                        const uint32_t xw = *reinterpret_cast<const uint32_t*>(p.x + ro + c0);
                        const float w0 = expf(-expf(bf_lo(xw))), w1 = expf(-expf(bf_hi(xw)));
                        y_lo = fmaf(bf_lo(rw), st[n][0], y_lo); y_lo = fmaf(bf_hi(rw), st[n][1], y_lo);
                        y_hi = fmaf(bf_lo(rw), st[n][2], y_hi); y_hi = fmaf(bf_hi(rw), st[n][3], y_hi);
                        st[n][0] = fmaf(w0, st[n][0], bf_lo(kw) * v_lo); st[n][1] = fmaf(w1, st[n][1], bf_hi(kw) * v_lo);
                        st[n][2] = fmaf(w0, st[n][2], bf_lo(kw) * v_hi); st[n][3] = fmaf(w1, st[n][3], bf_hi(kw) * v_hi);
                    }
                    y_lo += __shfl_xor_sync(0xffffffffu, y_lo, 1); y_lo += __shfl_xor_sync(0xffffffffu, y_lo, 2);
                    y_hi += __shfl_xor_sync(0xffffffffu, y_hi, 1); y_hi += __shfl_xor_sync(0xffffffffu, y_hi, 2);
                    if (q == 0) {
                        p.y[ro + j0] = __float2bfloat16_rn(fmaf(cf, v_lo, y_lo));
                        p.y[ro + j0 + 8] = __float2bfloat16_rn(fmaf(cf, v_hi, y_hi));
                    }
                }
            }
        }
        if (ytid == 0) bulk_wait<0>();
        if (p.state_out && !*abort_flag) {
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                const int c0 = 8 * n + 2 * q;
                p.state_out[sb + (size_t)c0 * 64 + j0] = st[n][0];
                p.state_out[sb + (size_t)(c0 + 1) * 64 + j0] = st[n][1];
                p.state_out[sb + (size_t)c0 * 64 + j0 + 8] = st[n][2];
                p.state_out[sb + (size_t)(c0 + 1) * 64 + j0 + 8] = st[n][3];
            }
        }
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// [rows][C] bf16 tensor, box = 64 rows x 64 channels (128 bytes), 128-byte swizzle
inline bool make_map(CUtensorMap* tm, const void* base, long long rows, long long C)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)C * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace ck

// Launches the chunked kernel.  Dense: cu == nullptr, n_seq = B, T = sequence length.
// Packed: cu = device cu_seqlens, n_seq = S, T unused.  total_rows = rows of the [rows][H*64] tensors.
inline gf_status_t chunked_prefill(const __nv_bfloat16* r, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                   const __nv_bfloat16* x, const float* u, const float* state_in, float* state_out,
                                   __nv_bfloat16* y, const int32_t* cu, int n_seq, int T, long long total_rows, int H,
                                   cudaStream_t st, std::atomic<uint64_t>* launches)
{
    const long long units = (long long)n_seq * H;
    if (units <= 0 || units > 0x7fffffffLL || total_rows <= 0 || total_rows >= (1LL << 31) - 64) return GF_ERR_INVALID_ARG;
    static bool attr_set = false;
    static int attr_dev = -1;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GF_ERR_CUDA;
    if (!attr_set || attr_dev != dev) {
        if (cudaFuncSetAttribute(ck::wkv6_chunked_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ck::SMEM_ALLOC) != cudaSuccess)
            return GF_ERR_CUDA;
        attr_set = true;
        attr_dev = dev;
    }
    CUtensorMap tr, tk, tv, tx, ty;
    const long long C = (long long)H * 64;
    if (!ck::make_map(&tr, r, total_rows, C) || !ck::make_map(&tk, k, total_rows, C) ||
        !ck::make_map(&tv, v, total_rows, C) || !ck::make_map(&tx, x, total_rows, C) ||
        !ck::make_map(&ty, y, total_rows, C))
        return GF_ERR_CUDA;
    ck::Params p{r, k, v, x, y, u, state_in, state_out, cu, T, H};
    ck::wkv6_chunked_kernel<<<(unsigned)units, ck::THREADS, ck::SMEM_ALLOC, st>>>(tr, tk, tv, tx, ty, p);
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
