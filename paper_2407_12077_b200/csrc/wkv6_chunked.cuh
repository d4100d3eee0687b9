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
// Warp roles (672 threads), pipelined across chunks through mbarriers:
//   warp 0       TMA producer: x tiles (4-stage ring) and {r,k,v} tiles (5-stage ring), 128B swizzle
//   warps 1-8    elementwise: decay, cumulative sum (phase A, one chunk ahead), then in place
//                R^ = r 2^{a_{t-1}}, K^ = k 2^{-a_t} (phase B); chunk decay 2^{a_L}, bonus
//                coefficients, safety vote
//   warps 9-12   state chain: S <- diag(2^{a_L}) (S + K^^T V) in mma accumulators for the whole
//                sequence; publishes a bf16 copy of every chunk-start state
//   warps 13-20  output, two groups alternating chunks: Y = R^ S_0 + (tril(R^ K^^T,-1) + diag(bonus)) V
//                with the score block kept in registers between its two contractions; every warp
//                stores its own 16 rows of y with TMA
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
constexpr int NX = 4;                  // x ring depth
constexpr int NS = 5;                  // {r,k,v} ring depth
constexpr int NSB = 3;                 // bf16 chunk-start state buffers
constexpr int NTOT = 4;                // per-warp decay-total buffers (phase A runs one chunk ahead)
constexpr int N_EW = 8;                // elementwise warps
constexpr int N_SW = 4;                // state warps
constexpr int N_YW = 8;                // output warps (two groups of four)
constexpr int WARP_S0 = 1 + N_EW;      // first state warp
constexpr int WARP_Y0 = WARP_S0 + N_SW;
constexpr int THREADS = 32 * (1 + N_EW + N_SW + N_YW);
constexpr float A2_MAX = 96.f;         // largest in-chunk |cumulative log2 decay| on the tensor-core path
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LOG2_LOG2E = 0.5287663729448977f;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;   // 2 s

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int OFF_X = 0;                                   // [NX][TILE]           x
constexpr int OFF_RKV = OFF_X + NX * TILE;                 // [NS][3][TILE]        r -> R^, k -> K^, v
constexpr int OFF_SB = OFF_RKV + NS * 3 * TILE;            // [NSB][TILE]          bf16 chunk-start state [c][j]
constexpr int OFF_Y = OFF_SB + NSB * TILE;                 // [N_YW][16 rows x 128 B] y staging, one slab per warp
constexpr int OFF_SCR = OFF_Y + N_YW * 2048;               // [64][64] float       state scratch (token-by-token path)
constexpr int OFF_TOT = OFF_SCR + 64 * 64 * 4;             // [NTOT][N_EW][64] float
constexpr int OFF_DL = OFF_TOT + NTOT * N_EW * 64 * 4;     // [NS][64] float       2^{a_L}
constexpr int OFF_DU = OFF_DL + NS * 64 * 4;               // [NS][64] float       bonus coefficient per token
constexpr int OFF_SAFE = OFF_DU + NS * 64 * 4;             // [NS] int (padded)
constexpr int OFF_ABORT = OFF_SAFE + 32;                   // int
constexpr int OFF_BAR = OFF_ABORT + 16;                    // mbarriers (8 bytes each)
enum {
    BAR_FULL_X = 0,
    BAR_EMPTY_X = BAR_FULL_X + NX,
    BAR_FULL_RKV = BAR_EMPTY_X + NX,
    BAR_EMPTY_RKV = BAR_FULL_RKV + NS,
    BAR_RK_READY = BAR_EMPTY_RKV + NS,
    BAR_S_READY = BAR_RK_READY + NS,
    BAR_S_FREE = BAR_S_READY + NSB,
    BAR_ESYNC = BAR_S_FREE + NSB,       // two, alternating by chunk parity
    BAR_SSYNC = BAR_ESYNC + 2,          // state-warp rendezvous (token-by-token path only)
    BAR_COUNT = BAR_SSYNC + 1
};
constexpr int SMEM_BYTES = OFF_BAR + BAR_COUNT * 8;
constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;              // slack for manual 1024-byte alignment
static_assert(SMEM_ALLOC <= 232448, "shared memory budget of one sm_100 CTA");

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
    // not volatile: a pure function of its register operands, so the compiler may schedule the
    // (ordered, volatile) shared-memory loads of later steps ahead of it
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}


__device__ __forceinline__ void stsm_x4(uint32_t a, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.shared.b16 [%0], {%1,%2,%3,%4};"
                 ::"r"(a), "r"(r0), "r"(r1), "r"(r2), "r"(r3) : "memory");
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

// Writes a warp's 16 x 64 fp32 accumulator block (acc[n][0..1] = row g, cols 8n+2q,+1;
// acc[n][2..3] = row g+8) as bf16 into rows row0 .. row0+15 of a 128B-swizzled [rows][64] tile.
__device__ __forceinline__ void store_acc_bf16(uint32_t tile, int row0, const float (&acc)[8][4], int lane)
{
    const int mi = lane >> 3, rr = lane & 7;
    const int row = row0 + rr + 8 * (mi & 1);
#pragma unroll
    for (int m = 0; m < 4; ++m)
        stsm_x4(tile + swz(row, (2 * m + (mi >> 1)) << 4),
                pack_bf16(acc[2 * m][0], acc[2 * m][1]), pack_bf16(acc[2 * m][2], acc[2 * m][3]),
                pack_bf16(acc[2 * m + 1][0], acc[2 * m + 1][1]), pack_bf16(acc[2 * m + 1][2], acc[2 * m + 1][3]));
}

// ---------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(THREADS, 1)
wkv6_chunked_kernel(const __grid_constant__ CUtensorMap tm_r, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_x,
                    const __grid_constant__ CUtensorMap tm_y16, const Params p)
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
        for (int i = 0; i < NX; ++i) { mbar_init(bar(BAR_FULL_X + i), 1); mbar_init(bar(BAR_EMPTY_X + i), N_EW); }
        for (int i = 0; i < NS; ++i) {
            mbar_init(bar(BAR_FULL_RKV + i), 1);
            mbar_init(bar(BAR_EMPTY_RKV + i), N_SW + N_YW / 2);
            mbar_init(bar(BAR_RK_READY + i), N_EW);
        }
        for (int i = 0; i < NSB; ++i) { mbar_init(bar(BAR_S_READY + i), N_SW); mbar_init(bar(BAR_S_FREE + i), N_YW / 2); }
        mbar_init(bar(BAR_ESYNC), N_EW);
        mbar_init(bar(BAR_ESYNC + 1), N_EW);
        mbar_init(bar(BAR_SSYNC), N_SW);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    if (warp == 0) {
        // ============================== TMA producer ==============================
        if (lane == 0) {
            int issued_x = 0, issued_s = 0;
            auto load_x = [&](int c) -> bool {
                const int sx = c % NX;
                if (c >= NX && !mbar_wait(bar(BAR_EMPTY_X + sx), ((c / NX) & 1) ^ 1, abort_flag)) return false;
                mbar_expect_tx(bar(BAR_FULL_X + sx), TILE);
                tma_load_2d(sbase + OFF_X + sx * TILE, &tm_x, col0, (int)(row0 + (long long)c * L), bar(BAR_FULL_X + sx));
                issued_x = c + 1;
                return true;
            };
            bool ok = true;
            for (int c = 0; c < min(NX - 1, nchunks) && ok; ++c) ok = load_x(c);
            for (int c = 0; c < nchunks && ok; ++c) {
                if (c + NX - 1 < nchunks && !load_x(c + NX - 1)) break;
                const int s = c % NS;
                if (c >= NS && !mbar_wait(bar(BAR_EMPTY_RKV + s), ((c / NS) & 1) ^ 1, abort_flag)) break;
                const int row = (int)(row0 + (long long)c * L);
                const uint32_t dst = sbase + OFF_RKV + s * 3 * TILE;
                mbar_expect_tx(bar(BAR_FULL_RKV + s), 3 * TILE);
                tma_load_2d(dst, &tm_r, col0, row, bar(BAR_FULL_RKV + s));
                tma_load_2d(dst + TILE, &tm_k, col0, row, bar(BAR_FULL_RKV + s));
                tma_load_2d(dst + 2 * TILE, &tm_v, col0, row, bar(BAR_FULL_RKV + s));
                issued_s = c + 1;
            }
            // do not leave while copies into this CTA's shared memory may still be in flight
            for (int c = max(0, issued_x - NX); c < issued_x; ++c)
                mbar_wait(bar(BAR_FULL_X + c % NX), (c / NX) & 1, abort_flag, false);
            for (int c = max(0, issued_s - NS); c < issued_s; ++c)
                mbar_wait(bar(BAR_FULL_RKV + c % NS), (c / NS) & 1, abort_flag, false);
        }
    } else if (warp < WARP_S0) {
        // ============================== elementwise warps ==============================
        const int tq = warp - 1;                 // tokens 8*tq .. 8*tq+7 of the chunk
        const int cb = lane * 4;                 // byte column of this lane's channel pair (2*lane, 2*lane+1)
        const int etid = tid - 32;               // 0..255
        const float2 u2 = *reinterpret_cast<const float2*>(p.u + h * 64 + 2 * lane);
        float* tot = reinterpret_cast<float*>(smem + OFF_TOT);
        // phase A of chunk c: log2-decay magnitudes and this warp's local cumulative sums
        auto phase_a = [&](int c, float (&l0)[8], float (&l1)[8]) -> bool {
            const int sx = c % NX;
            const int valid = min(L, len - c * L);
            const uint32_t tx = sbase + OFF_X + sx * TILE;
            if (!mbar_wait(bar(BAR_FULL_X + sx), (c / NX) & 1, abort_flag)) return false;
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
            *reinterpret_cast<float2*>(tot + ((c % NTOT) * N_EW + tq) * 64 + 2 * lane) = make_float2(a0, a1);
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(BAR_EMPTY_X + sx));
                mbar_arrive(bar(BAR_ESYNC + (c & 1)));
            }
            return true;
        };
        float l0[8], l1[8];
        bool live = nchunks > 0 && phase_a(0, l0, l1);
        for (int c = 0; c < nchunks && live; ++c) {
            float n0[8], n1[8];
            if (c + 1 < nchunks && !phase_a(c + 1, n0, n1)) break;
            const int s = c % NS;
            const int valid = min(L, len - c * L);
            if (!mbar_wait(bar(BAR_ESYNC + (c & 1)), (c >> 1) & 1, abort_flag)) break;
            float off0 = 0.f, off1 = 0.f;
            const float* totc = tot + (c % NTOT) * N_EW * 64;
            for (int q = 0; q < tq; ++q) {
                const float2 t2 = *reinterpret_cast<const float2*>(totc + q * 64 + 2 * lane);
                off0 += t2.x; off1 += t2.y;
            }
            if (!mbar_wait(bar(BAR_FULL_RKV + s), (c / NS) & 1, abort_flag)) break;
            // ---- phase B, in place: r -> R^ = r 2^{a_{t-1}}, k -> K^ = k 2^{-a_t}; bonus partials
            const uint32_t tr = sbase + OFF_RKV + s * 3 * TILE, tk = tr + TILE, tv = tr + 2 * TILE;
            float du[8];
            uint32_t rw[8], kw[8];
#pragma unroll
            for (int tt = 0; tt < 8; ++tt) {                 // all loads first: they are ordered with the stores below
                rw[tt] = lds32(tr + swz(8 * tq + tt, cb));
                kw[tt] = lds32(tk + swz(8 * tq + tt, cb));
            }
#pragma unroll
            for (int tt = 0; tt < 8; ++tt) {
                const int t = 8 * tq + tt;
                const float ap0 = off0 + (tt ? l0[tt - 1] : 0.f), ap1 = off1 + (tt ? l1[tt - 1] : 0.f);
                const float ac0 = off0 + l0[tt], ac1 = off1 + l1[tt];
                const float r0 = bf_lo(rw[tt]), r1 = bf_hi(rw[tt]), k0 = bf_lo(kw[tt]), k1 = bf_hi(kw[tt]);
                uint32_t rh = pack_bf16(r0 * ex2(ap0), r1 * ex2(ap1));
                uint32_t kh = pack_bf16(k0 * ex2(-ac0), k1 * ex2(-ac1));
                float d = fmaf(r0 * k0, u2.x, r1 * k1 * u2.y);
                if (t >= valid) { rh = 0u; kh = 0u; d = 0.f; }
                rw[tt] = rh; kw[tt] = kh;
                du[tt] = d;
            }
#pragma unroll
            for (int tt = 0; tt < 8; ++tt) {
                sts32(tr + swz(8 * tq + tt, cb), rw[tt]);
                sts32(tk + swz(8 * tq + tt, cb), kw[tt]);
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
                    reinterpret_cast<float*>(smem + OFF_DU)[s * 64 + 8 * tq + (lane >> 2)] = w1;
            }
            if (tq == N_EW - 1) {
                const float aL0 = off0 + l0[7], aL1 = off1 + l1[7];
                *reinterpret_cast<float2*>(reinterpret_cast<float*>(smem + OFF_DL) + s * 64 + 2 * lane) =
                    make_float2(ex2(aL0), ex2(aL1));
                const bool ok = (aL0 >= -A2_MAX) && (aL1 >= -A2_MAX);       // false for NaN as well
                const bool all_ok = __all_sync(0xffffffffu, ok);
                if (lane == 0) safe_flag[s] = all_ok ? 1 : 0;
            }
            if (valid < L) {
                // v rows past the end of the sequence hold another sequence's tokens (or fill): zero them
                for (int i = etid; i < (L - valid) * 8; i += 32 * N_EW)
                    sts128z(tv + (valid + (i >> 3)) * 128 + ((i & 7) << 4));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_RK_READY + s));
#pragma unroll
            for (int tt = 0; tt < 8; ++tt) { l0[tt] = n0[tt]; l1[tt] = n1[tt]; }
        }
    } else if (warp < WARP_Y0) {
        // ============================== state warps ==============================
        const int sw = warp - WARP_S0;           // key channels c = 16*sw .. 16*sw+15 (state rows)
        const int g = lane >> 2, q = lane & 3;
        const int c_lo = 16 * sw + g;
        const size_t sb = (size_t)unit * 4096;
        // S[c][j] in accumulator layout: st[n][0..1] = (c_lo, j = 8n+2q, +1), st[n][2..3] = (c_lo+8, same j)
        float st[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            if (p.state_in) {
                const float2 lo = *reinterpret_cast<const float2*>(p.state_in + sb + (size_t)c_lo * 64 + 8 * n + 2 * q);
                const float2 hi = *reinterpret_cast<const float2*>(p.state_in + sb + (size_t)(c_lo + 8) * 64 + 8 * n + 2 * q);
                st[n][0] = lo.x; st[n][1] = lo.y; st[n][2] = hi.x; st[n][3] = hi.y;
            } else {
                st[n][0] = st[n][1] = st[n][2] = st[n][3] = 0.f;
            }
        }
        int ssync_uses = 0;
        auto ssync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_SSYNC));
            const bool ok = mbar_wait(bar(BAR_SSYNC), ssync_uses & 1, abort_flag);
            ++ssync_uses;
            return ok;
        };
        if (nchunks > 0) {
            store_acc_bf16(sbase + OFF_SB, 16 * sw, st, lane);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_S_READY));
        }
        for (int c = 0; c < nchunks; ++c) {
            const int s = c % NS;
            const int valid = min(L, len - c * L);
            const uint32_t tk = sbase + OFF_RKV + s * 3 * TILE + TILE, tv = tk + TILE;
            if (!mbar_wait(bar(BAR_FULL_RKV + s), (c / NS) & 1, abort_flag)) break;
            if (!mbar_wait(bar(BAR_RK_READY + s), (c / NS) & 1, abort_flag)) break;
            if (safe_flag[s]) {
                // ---- S += K^^T V   (M = c, N = j, K = i), then scale row c by 2^{a_L[c]}
                uint32_t ka[4][4];
                {
                    const int irow = (lane & 7) + 8 * (lane >> 4);
                    const int cbyte = (16 * sw + 8 * ((lane >> 3) & 1)) * 2;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ldsm_x4_t(tk + swz(16 * kk + irow, cbyte), ka[kk][0], ka[kk][1], ka[kk][2], ka[kk][3]);
                }
                const int krow = (lane & 7) + 8 * ((lane >> 3) & 1);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
                    for (int jp = 0; jp < 4; ++jp) {
                        uint32_t b0, b1, b2, b3;
                        ldsm_x4_t(tv + swz(16 * kk + krow, 32 * jp + 16 * (lane >> 4)), b0, b1, b2, b3);
                        mma16816(st[2 * jp], ka[kk], b0, b1);
                        mma16816(st[2 * jp + 1], ka[kk], b2, b3);
                    }
                }
                const float* dl = reinterpret_cast<const float*>(smem + OFF_DL) + s * 64;
                const float d_lo = dl[c_lo], d_hi = dl[c_lo + 8];
#pragma unroll
                for (int n = 0; n < 8; ++n) { st[n][0] *= d_lo; st[n][1] *= d_lo; st[n][2] *= d_hi; st[n][3] *= d_hi; }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_EMPTY_RKV + s));
            } else {
                // ---- decay too strong for one in-chunk reference point: exact fp32 recurrence, token by
                // token, on a copy of the state in shared memory where a warp owns 16 value channels for
                // all 64 key channels.
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_EMPTY_RKV + s));
                float* scr = reinterpret_cast<float*>(smem + OFF_SCR);
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    *reinterpret_cast<float2*>(scr + c_lo * 64 + 8 * n + 2 * q) = make_float2(st[n][0], st[n][1]);
                    *reinterpret_cast<float2*>(scr + (c_lo + 8) * 64 + 8 * n + 2 * q) = make_float2(st[n][2], st[n][3]);
                }
                if (!ssync()) break;
                {
                    // lane = 16*half + jl works on S[32*half .. +31][16*sw + jl], kept in the fp32 scratch
                    const int half = lane >> 4, j = 16 * sw + (lane & 15);
                    float* scol = scr + (32 * half) * 64 + j;
                    const float* ug = p.u + h * 64 + 32 * half;
                    for (int t = 0; t < valid; ++t) {
                        const size_t ro = (size_t)(row0 + (long long)c * L + t) * C + col0;
                        const float vj = __bfloat162float(p.v[ro + j]);
                        float yj = 0.f, cf = 0.f;
#pragma unroll 4
                        for (int i = 0; i < 32; i += 2) {
                            const uint32_t rw = *reinterpret_cast<const uint32_t*>(p.r + ro + 32 * half + i);
                            const uint32_t kw = *reinterpret_cast<const uint32_t*>(p.k + ro + 32 * half + i);
                            const uint32_t xw = *reinterpret_cast<const uint32_t*>(p.x + ro + 32 * half + i);
                            const float s0 = scol[i * 64], s1 = scol[(i + 1) * 64];
                            cf = fmaf(bf_lo(rw) * ug[i], bf_lo(kw), cf);
                            cf = fmaf(bf_hi(rw) * ug[i + 1], bf_hi(kw), cf);
                            yj = fmaf(bf_lo(rw), s0, yj);
                            yj = fmaf(bf_hi(rw), s1, yj);
                            scol[i * 64] = fmaf(expf(-expf(bf_lo(xw))), s0, bf_lo(kw) * vj);
                            scol[(i + 1) * 64] = fmaf(expf(-expf(bf_hi(xw))), s1, bf_hi(kw) * vj);
                        }
                        yj += __shfl_xor_sync(0xffffffffu, yj, 16);
                        cf += __shfl_xor_sync(0xffffffffu, cf, 16);
                        if (half == 0) p.y[ro + j] = __float2bfloat16_rn(fmaf(cf, vj, yj));
                    }
                }
                if (!ssync()) break;
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                    const float2 lo = *reinterpret_cast<const float2*>(scr + c_lo * 64 + 8 * n + 2 * q);
                    const float2 hi = *reinterpret_cast<const float2*>(scr + (c_lo + 8) * 64 + 8 * n + 2 * q);
                    st[n][0] = lo.x; st[n][1] = lo.y; st[n][2] = hi.x; st[n][3] = hi.y;
                }
                if (!ssync()) break;          // everyone has re-read the scratch before it can be rewritten
            }
            if (c + 1 < nchunks) {
                const int nb = (c + 1) % NSB;
                if (c + 1 >= NSB && !mbar_wait(bar(BAR_S_FREE + nb), (((c + 1) / NSB) & 1) ^ 1, abort_flag)) break;
                store_acc_bf16(sbase + OFF_SB + nb * TILE, 16 * sw, st, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(BAR_S_READY + nb));
            }
        }
        if (p.state_out && !*abort_flag) {
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                *reinterpret_cast<float2*>(p.state_out + sb + (size_t)c_lo * 64 + 8 * n + 2 * q) = make_float2(st[n][0], st[n][1]);
                *reinterpret_cast<float2*>(p.state_out + sb + (size_t)(c_lo + 8) * 64 + 8 * n + 2 * q) = make_float2(st[n][2], st[n][3]);
            }
        }
    } else {
        // ============================== output warps ==============================
        const int yw = warp - WARP_Y0;           // 0..7
        const int grp = yw >> 2, w4 = yw & 3;    // group grp takes chunks grp, grp+2, ...
        const int g = lane >> 2, q = lane & 3;
        const uint32_t slab = sbase + OFF_Y + yw * 2048;
        const int krow = (lane & 7) + 8 * ((lane >> 3) & 1);      // [k][n] tiles read with .trans
        for (int c = grp; c < nchunks; c += 2) {
            const int s = c % NS, sbi = c % NSB;
            const int valid = min(L, len - c * L);
            // alternate the row block between rounds so the causal triangle's work evens out
            const int rb = ((c >> 1) & 1) ? 3 - w4 : w4;          // rows t = 16*rb .. 16*rb+15
            const uint32_t tr = sbase + OFF_RKV + s * 3 * TILE, tk = tr + TILE, tv = tr + 2 * TILE;
            const uint32_t tsb = sbase + OFF_SB + sbi * TILE;
            if (!mbar_wait(bar(BAR_FULL_RKV + s), (c / NS) & 1, abort_flag)) break;
            if (!mbar_wait(bar(BAR_RK_READY + s), (c / NS) & 1, abort_flag)) break;
            if (!mbar_wait(bar(BAR_S_READY + sbi), (c / NSB) & 1, abort_flag)) break;
            if (!safe_flag[s]) {
                __syncwarp();
                if (lane == 0) { mbar_arrive(bar(BAR_S_FREE + sbi)); mbar_arrive(bar(BAR_EMPTY_RKV + s)); }
                continue;
            }
            // R^ rows of this block are re-read from shared memory at every use (A fragments, 4 registers
            // at a time) instead of being held for the whole chunk: registers are the scarcer resource
            const uint32_t ta = tr + (16 * rb + (lane & 7) + 8 * ((lane >> 3) & 1)) * 128;
            const int ta_x = (lane & 7) << 4, ta_c = 16 * (lane >> 4);
            float ya[8][4];
#pragma unroll
            for (int n = 0; n < 8; ++n) ya[n][0] = ya[n][1] = ya[n][2] = ya[n][3] = 0.f;
            // ---- Y = R^ S_0   (M = t, N = j, K = c)
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                uint32_t a[4];
                ldsm_x4(ta + ((32 * kk + ta_c) ^ ta_x), a[0], a[1], a[2], a[3]);
#pragma unroll
                for (int jp = 0; jp < 4; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(tsb + swz(16 * kk + krow, 32 * jp + 16 * (lane >> 4)), b0, b1, b2, b3);
                    mma16816(ya[2 * jp], a, b0, b1);
                    mma16816(ya[2 * jp + 1], a, b2, b3);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_S_FREE + sbi));
            // ---- Y += (tril(R^ K^^T, -1) + diag(bonus)) V, one 16-token block of past tokens at a time
            const float* du = reinterpret_cast<const float*>(smem + OFF_DU) + s * 64;
            for (int ib = 0; ib <= rb; ++ib) {
                float acc[2][4];
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[0][e] = acc[1][e] = 0.f;
                const int irow = 16 * ib + (lane & 7) + 8 * (lane >> 4);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    uint32_t a[4], b0, b1, b2, b3;
                    ldsm_x4(ta + ((32 * kk + ta_c) ^ ta_x), a[0], a[1], a[2], a[3]);
                    ldsm_x4(tk + swz(irow, 32 * kk + 16 * ((lane >> 3) & 1)), b0, b1, b2, b3);
                    mma16816(acc[0], a, b0, b1);
                    mma16816(acc[1], a, b2, b3);
                }
                if (ib == rb) {
                    // diagonal block: strictly-lower entries stay, the diagonal takes the bonus
                    // coefficient, the upper triangle is zero
                    const float d_lo = du[16 * rb + g], d_hi = du[16 * rb + g + 8];
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
                uint32_t pa[4];
                pa[0] = pack_bf16(acc[0][0], acc[0][1]);
                pa[1] = pack_bf16(acc[0][2], acc[0][3]);
                pa[2] = pack_bf16(acc[1][0], acc[1][1]);
                pa[3] = pack_bf16(acc[1][2], acc[1][3]);
#pragma unroll
                for (int jp = 0; jp < 4; ++jp) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(tv + swz(16 * ib + krow, 32 * jp + 16 * (lane >> 4)), b0, b1, b2, b3);
                    mma16816(ya[2 * jp], pa, b0, b1);
                    mma16816(ya[2 * jp + 1], pa, b2, b3);
                }
            }
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar(BAR_EMPTY_RKV + s));
                bulk_wait_read<0>();              // this warp's previous store has finished reading the slab
            }
            __syncwarp();
            // ---- epilogue: this warp's 16 rows of y -> bf16 slab -> global
            store_acc_bf16(slab, 0, ya, lane);
            fence_proxy_async();
            __syncwarp();
            const int rows = valid - 16 * rb;
            const long long grow = row0 + (long long)c * L + 16 * rb;
            if (rows >= 16) {
                if (lane == 0) {
                    tma_store_2d(&tm_y16, col0, (int)grow, slab);
                    bulk_commit();
                }
            } else {
                // ragged tail: the rows after `valid` belong to someone else, so copy row by row
                for (int i = lane; i < rows * 8; i += 32) {
                    const int t = i >> 3, ch = i & 7;
                    uint4 val;
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                                 : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(slab + swz(t, ch << 4)));
                    *reinterpret_cast<uint4*>(p.y + (size_t)(grow + t) * C + col0 + ch * 8) = val;
                }
                __syncwarp();
            }
        }
        if (lane == 0) bulk_wait<0>();
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

// [rows][C] bf16 tensor, box = box_rows rows x 64 channels (128 bytes), 128-byte swizzle
inline bool make_map(CUtensorMap* tm, const void* base, long long rows, long long C, int box_rows)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)C, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)C * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
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
    if (!ck::make_map(&tr, r, total_rows, C, 64) || !ck::make_map(&tk, k, total_rows, C, 64) ||
        !ck::make_map(&tv, v, total_rows, C, 64) || !ck::make_map(&tx, x, total_rows, C, 64) ||
        !ck::make_map(&ty, y, total_rows, C, 16))
        return GF_ERR_CUDA;
    ck::Params p{r, k, v, x, y, u, state_in, state_out, cu, T, H};
    ck::wkv6_chunked_kernel<<<(unsigned)units, ck::THREADS, ck::SMEM_ALLOC, st>>>(tr, tk, tv, tx, ty, p);
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
