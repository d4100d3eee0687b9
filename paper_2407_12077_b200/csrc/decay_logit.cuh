// The decay logit of the Finch-C2 block for sm_100a: d_t = lora_omega( ddlerp_d( x_t, x_{t-1} ) ), i.e. with
//   lerp(a, b, t) = a + (b - a) t,   lora(v) = lambda + tanh(v A) B,   ddlerp(a, b) = a + (b - a) lora_d(lerp(a, b, mu_x)):
//   z_t = x_t + (x_{t-1} - x_t) mu_x                       (token shift, per channel)
//   h1  = tanh(z_t A_d)                                    [R_d]
//   m_t = x_t + (x_{t-1} - x_t) (lambda_d + h1 B_d)        (the data-dependent mix)
//   h2  = tanh(m_t A_w)                                    [R_w]
//   d_t = lambda_w + h2 B_w                                (the logit the WKV kernels take as x: w_t = exp(-exp(d_t)))
// x, d: [rows][D] bf16 with rows = B*T (x_{t-1} of a sequence's first token: x_prev[b], or zero); A_*: [D][R], B_*: [R][D]
// bf16; mu_x, lambda_*: [D] fp32.  Four skinny products (2 D (2 R_d + 2 R_w) flops per token) around elementwise
// work on a tensor that is read twice and written once: HBM-bound (4 D bytes per token when the second read of x
// hits L2), so the products run on the tensor cores and everything else is shaped to stream.
//
// One persistent CTA per SM walks tiles of 128 tokens in three passes over the D channels, 64 at a time:
//   pass 1: z slice -> bf16 operand tile -> acc1 += z A_d[slice]           then h1 = tanh(acc1) -> operand tile
//   pass 2: l = h1 B_d[:, slice] -> tensor memory -> m slice -> bf16 operand tile -> acc3 += m A_w[slice]
//           then h2 = tanh(acc3) -> operand tile
//   pass 3: d slice = lambda_w + h2 B_w[:, slice] -> bf16 -> TMA store
//   warp 0      TMA producer of the x ring (5 stages): per slice the x rows of the tile (plus the one row above it)
//               and the 64 per-channel constants of the pass; a stage is free as soon as its rows are in registers
//   warp 3      TMA producer of the weight ring (5 stages): the slice's weight tiles, free when their products are done
//   warp 1      tensor-memory allocation; an elected lane issues the products whose operands come from the weight
//               ring and the h tile (z A_d, h1 B_d, h2 B_w; tcgen05.mma 128 x 64 x 16, bf16 -> fp32)
//   warp 2      an elected lane issues m A_w, the product that waits for the workers inside pass 2 (an issuer of
//               its own, so that the l products of later slices are not held up behind it)
//   warps 4-11  two sets of four warps taking alternate slices; a lane owns one token row (the accumulator row
//               of its tensor-memory sub-partition): reads its row and the row above from the swizzled x tiles,
//               forms z / m / d for the 64 channels of the slice, writes the bf16 operand row (or the output slab)
// All operand tiles are the 128-byte-swizzled [64 rows][64 bf16] tiles of the prefill kernel; weight tiles narrower
// than 64 (R < 64) are zero-filled by TMA beyond their extent.  Every wait is bounded, as in the prefill kernel.
#pragma once
#include "key_compress.cuh"
#include "wkv6_chunked.cuh"

namespace gf {
namespace dl {

using namespace ck;

constexpr int DL_NSET = 2;                             // worker sets
constexpr int DL_W0 = 4;                               // first worker warp
constexpr int DL_THREADS = 32 * (DL_W0 + 4 * DL_NSET);
// Two rings.  The x ring holds, per slice, the tile's x rows (two swizzled 64-row tiles), the row above the tile and the
// pass's 64 per-channel constants; a worker set frees its stage as soon as the rows are in registers, so that ring
// runs a load latency ahead of the arithmetic.  The weight ring holds up to two weight tiles per slice and is freed
// by the products that read them (weights come from L2).
constexpr int DL_NSX = 5, DL_NSW = 5;
constexpr int DL_NACC = 6;                             // l / d accumulators in tensor memory: the products h1 B_d and h2 B_w depend on
                                                       // nothing the workers make, so they run this many slices ahead of them
constexpr int DL_XSTAGE = 2 * TILE + 1024;
constexpr int DL_OFF_PREV = 2 * TILE;                  // [64] bf16: the x row just above the tile (this slice)
constexpr int DL_OFF_VEC = 2 * TILE + 256;             // [64] fp32: mu_x / lambda_d / lambda_w of this slice
constexpr int DL_WSTAGE = 2 * TILE;
constexpr int DL_OFF_W = DL_NSX * DL_XSTAGE;           // weight ring
constexpr int DL_OFF_OP = DL_OFF_W + DL_NSW * DL_WSTAGE;         // [sets][128 rows x 128 B]: z / m operand, output slabs in pass 3
constexpr int DL_OFF_H = DL_OFF_OP + DL_NSET * 2 * TILE;         // [128 rows x 128 B]: h1 / h2 operand
constexpr int DL_OFF_MISC = DL_OFF_H + 2 * TILE;       // abort word + limit, tensor-memory address, barriers
constexpr int DL_SMEM = DL_OFF_MISC + 512 + 1024;      // + slack for manual 1024-byte alignment
enum {
    DL_XFULL = 0,                      // x stage loaded
    DL_XEMPTY = DL_XFULL + DL_NSX,     // ... and read into registers by the four warps of its set
    DL_WFULL = DL_XEMPTY + DL_NSX,     // weight stage loaded
    DL_WEMPTY = DL_WFULL + DL_NSW,     // ... and the last product that reads it is done
    DL_OP_READY = DL_WEMPTY + DL_NSW,  // per set: operand rows written
    DL_OP_FREE = DL_OP_READY + DL_NSET,    // per set: the product that read them is done
    DL_ACC_FULL = DL_OP_FREE + DL_NSET,    // per accumulator: l (pass 2) or d (pass 3) of a slice is in tensor memory
    DL_ACC_FREE = DL_ACC_FULL + DL_NACC,   // ... and read back by the four warps of the slice's set
    DL_SUM_FULL = DL_ACC_FREE + DL_NACC,   // acc1 / acc3 complete
    DL_H_READY = DL_SUM_FULL + 1,      // h1 / h2 operand written by all worker warps
    DL_PASS2 = DL_H_READY + 1,         // pass 2 of a tile has begun (first issuer -> second issuer: one phase per tile)
    DL_BAR_COUNT = DL_PASS2 + 1
};
static_assert(16 + 8 * DL_BAR_COUNT <= 512, "barrier block");
static_assert(DL_SMEM <= 232448, "shared memory budget of one sm_100 CTA");
constexpr int DL_TM_ACC1 = 0, DL_TM_ACC3 = 64, DL_TM_RING = 128;       // + 64 * accumulator (l in pass 2, d in pass 3)
static_assert(DL_TM_RING + 64 * DL_NACC <= 512, "tensor memory columns");
// fp32 accumulator, bf16 A (K-major) and B (MN-major), M = 128, N = 64
constexpr uint32_t DL_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

struct DlParams {
    long long rows;                    // B * T
    int T;                             // tokens per sequence (token shift restarts every T rows)
    int nslices;                       // D / 64
    int kd, kw;                        // 16-wide contraction steps over the two ranks: R_d / 16, R_w / 16
    const __nv_bfloat16* x_prev;       // [B][D] or NULL
    int D;
    const float *mu_x, *lambda_d, *lambda_w;
};

__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v)
{
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ float tanh_fast(float v)
{
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(v));
    return y;
}
// 16 consecutive fp32 columns of this lane's accumulator row
__device__ __forceinline__ void tmem_ld_row16(uint32_t taddr, float (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]),
          "=f"(v[8]), "=f"(v[9]), "=f"(v[10]), "=f"(v[11]), "=f"(v[12]), "=f"(v[13]), "=f"(v[14]), "=f"(v[15])
        : "r"(taddr) : "memory");
}

__global__ void __launch_bounds__(DL_THREADS, 1)
decay_logit_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_x1,
                   const __grid_constant__ CUtensorMap tm_ad, const __grid_constant__ CUtensorMap tm_bd,
                   const __grid_constant__ CUtensorMap tm_aw, const __grid_constant__ CUtensorMap tm_bw,
                   const __grid_constant__ CUtensorMap tm_d32, const DlParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t abort_flag = sbase + DL_OFF_MISC;
    auto bar = [&](int i) { return sbase + DL_OFF_MISC + 16 + 8 * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long n_tiles = (p.rows + 127) / 128;
    const int S = p.nslices;

    if (tid == 0) {
        for (int i = 0; i < DL_NSX; ++i) {
            mbar_init(bar(DL_XFULL + i), 1);
            mbar_init(bar(DL_XEMPTY + i), 4);
        }
        for (int i = 0; i < DL_NSW; ++i) {
            mbar_init(bar(DL_WFULL + i), 1);
            mbar_init(bar(DL_WEMPTY + i), 1);
        }
        for (int i = 0; i < DL_NSET; ++i) {
            mbar_init(bar(DL_OP_READY + i), 4);
            mbar_init(bar(DL_OP_FREE + i), 1);
        }
        for (int i = 0; i < DL_NACC; ++i) {
            mbar_init(bar(DL_ACC_FULL + i), 1);
            mbar_init(bar(DL_ACC_FREE + i), 4);
        }
        mbar_init(bar(DL_SUM_FULL), 1);
        mbar_init(bar(DL_H_READY), 4 * DL_NSET);
        mbar_init(bar(DL_PASS2), 1);
        sts32(abort_flag, 0u);
        sts32(abort_flag + 4, WAIT_LIMIT_US);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(sbase + DL_OFF_MISC + 8, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32(sbase + DL_OFF_MISC + 8);
    auto wstage = [&](int i) { return sbase + DL_OFF_W + (i % DL_NSW) * DL_WSTAGE; };

    if (warp == 0) {
        // ============================== TMA producer: x rows and per-channel constants ==============================
        int it = 0, issued = 0;
        bool alive = true;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x) {
            const int row0 = (int)(t * 128);
            for (int pass = 0; pass < 3 && alive; ++pass)
                for (int s = 0; s < S; ++s, ++it) {
                    const int st = it % DL_NSX;
                    if (it >= DL_NSX && !mbar_wait_warp(bar(DL_XEMPTY + st), ((it / DL_NSX) + 1) & 1, abort_flag)) { alive = false; break; }
                    const uint32_t dst = sbase + st * DL_XSTAGE, full = bar(DL_XFULL + st);
                    if (elect_one()) {
                        const float* vec = pass == 0 ? p.mu_x : pass == 1 ? p.lambda_d : p.lambda_w;
                        if (pass < 2) {
                            mbar_expect_tx(full, 2 * TILE + 128 + 256);
                            tma_load_2d(dst, &tm_x, 64 * s, row0, full);
                            tma_load_2d(dst + TILE, &tm_x, 64 * s, row0 + 64, full);
                            tma_load_2d(dst + DL_OFF_PREV, &tm_x1, 64 * s, row0 - 1, full);      // (row -1 reads as zero)
                        } else {
                            mbar_expect_tx(full, 256);
                        }
                        bulk_load_1d(dst + DL_OFF_VEC, vec + 64 * s, 256, full);
                    }
                    __syncwarp();
                    issued = it + 1;
                }
        }
        // do not leave while copies into this CTA's shared memory may still be in flight
        for (int c = max(0, issued - DL_NSX); c < issued; ++c)
            mbar_wait_warp(bar(DL_XFULL + c % DL_NSX), (c / DL_NSX) & 1, abort_flag, false);
    } else if (warp == 3) {
        // ============================== TMA producer: weight tiles ==============================
        int it = 0, issued = 0;
        bool alive = true;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x)
            for (int pass = 0; pass < 3 && alive; ++pass)
                for (int s = 0; s < S; ++s, ++it) {
                    const int st = it % DL_NSW;
                    if (it >= DL_NSW && !mbar_wait_warp(bar(DL_WEMPTY + st), ((it / DL_NSW) + 1) & 1, abort_flag)) { alive = false; break; }
                    const uint32_t dst = wstage(it), full = bar(DL_WFULL + st);
                    if (elect_one()) {
                        if (pass == 0) {
                            mbar_expect_tx(full, TILE);
                            tma_load_2d(dst, &tm_ad, 0, 64 * s, full);
                        } else if (pass == 1) {
                            mbar_expect_tx(full, 2 * TILE);
                            tma_load_2d(dst, &tm_bd, 64 * s, 0, full);
                            tma_load_2d(dst + TILE, &tm_aw, 0, 64 * s, full);
                        } else {
                            mbar_expect_tx(full, TILE);
                            tma_load_2d(dst, &tm_bw, 64 * s, 0, full);
                        }
                    }
                    __syncwarp();
                    issued = it + 1;
                }
        for (int c = max(0, issued - DL_NSW); c < issued; ++c)
            mbar_wait_warp(bar(DL_WFULL + c % DL_NSW), (c / DL_NSW) & 1, abort_flag, false);
    } else if (warp == 1) {
        // ============================== MMA issuer: z A_d, h1 B_d, h2 B_w ==============================
        int it = 0;
        int op_uses[DL_NSET] = {};                           // per set: operand tiles consumed
        int an = 0;                                          // l / d accumulators produced so far (their ring position)
        bool alive = true;
        auto weights_in = [&](int i) { return mbar_wait_warp(bar(DL_WFULL + i % DL_NSW), (i / DL_NSW) & 1, abort_flag); };
        const uint64_t dh = smem_desc(sbase + DL_OFF_H);
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x) {
            // ---- pass 1: acc1 += z A_d[slice]
            for (int s = 0; s < S; ++s, ++it) {
                const int h = s % DL_NSET;
                if (!weights_in(it) || !mbar_wait_warp(bar(DL_OP_READY + h), op_uses[h] & 1, abort_flag)) { alive = false; break; }
                ++op_uses[h];
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t da = smem_desc(sbase + DL_OFF_OP + h * 2 * TILE);
                    const uint64_t db = smem_desc(wstage(it));
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma(tmem + DL_TM_ACC1, da + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk), DL_IDESC, (s > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar(DL_OP_FREE + h));
                    tc_commit(bar(DL_WEMPTY + it % DL_NSW));
                    if (s == S - 1) tc_commit(bar(DL_SUM_FULL));
                }
                __syncwarp();
            }
            if (!alive) break;
            // ---- pass 2: l = h1 B_d[:, slice] (the other issuer follows with acc3 += m A_w[slice] and frees the stage)
            if (!mbar_wait_warp(bar(DL_H_READY), 0, abort_flag)) break;          // (two uses per tile: parities 0, 1)
            tc_fence_after();
            if (elect_one()) mbar_arrive(bar(DL_PASS2));                           // every operand-row phase of pass 1 is over
            __syncwarp();
            for (int s = 0; s < S; ++s, ++it) {
                const int h = s % DL_NSET;
                if (!weights_in(it)) { alive = false; break; }
                const int a = an % DL_NACC;
                if (an >= DL_NACC && !mbar_wait_warp(bar(DL_ACC_FREE + a), ((an / DL_NACC) + 1) & 1, abort_flag)) { alive = false; break; }
                ++an;
                ++op_uses[h];                                 // (the other issuer consumes this slice's operand rows)
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t db = smem_desc(wstage(it));
                    for (int kk = 0; kk < p.kd; ++kk)
                        tc_mma(tmem + DL_TM_RING + 64 * a, dh + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk), DL_IDESC, kk > 0 ? 1u : 0u);
                    tc_commit(bar(DL_ACC_FULL + a));
                }
                __syncwarp();
            }
            if (!alive) break;
            // ---- pass 3: d slice = h2 B_w[:, slice]
            if (!mbar_wait_warp(bar(DL_H_READY), 1, abort_flag)) break;
            tc_fence_after();
            for (int s = 0; s < S; ++s, ++it) {
                if (!weights_in(it)) { alive = false; break; }
                const int a = an % DL_NACC;
                if (an >= DL_NACC && !mbar_wait_warp(bar(DL_ACC_FREE + a), ((an / DL_NACC) + 1) & 1, abort_flag)) { alive = false; break; }
                ++an;
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t db = smem_desc(wstage(it));
                    for (int kk = 0; kk < p.kw; ++kk)
                        tc_mma(tmem + DL_TM_RING + 64 * a, dh + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk), DL_IDESC, kk > 0 ? 1u : 0u);
                    tc_commit(bar(DL_ACC_FULL + a));
                    tc_commit(bar(DL_WEMPTY + it % DL_NSW));
                }
                __syncwarp();
            }
        }
    } else if (warp == 2) {
        // ============================== MMA issuer: m A_w (pass 2) ==============================
        int ti = 0;
        int op_uses[DL_NSET] = {};
        bool alive = true;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x, ++ti) {
            // A wait names a phase by its parity alone, so it must not start more than one phase ahead of the barrier:
            // the operand-row barriers go through pass 1's phases first (the other issuer's), hence the go-ahead.
            if (!mbar_wait_warp(bar(DL_PASS2), ti & 1, abort_flag)) break;
            for (int s = 0; s < S; ++s) op_uses[s % DL_NSET] += 1;        // pass 1's uses of the operand rows
            const int it2 = ti * 3 * S + S;                               // ring position of pass 2, slice 0
            for (int s = 0; s < S; ++s) {
                const int h = s % DL_NSET, i = it2 + s;
                if (!mbar_wait_warp(bar(DL_OP_READY + h), op_uses[h] & 1, abort_flag)) { alive = false; break; }
                ++op_uses[h];
                // (complete by now: the other issuer saw this stage full before it made the l this operand was built from)
                if (!mbar_wait_warp(bar(DL_WFULL + i % DL_NSW), (i / DL_NSW) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t da = smem_desc(sbase + DL_OFF_OP + h * 2 * TILE);
                    const uint64_t db = smem_desc(wstage(i) + TILE);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        tc_mma(tmem + DL_TM_ACC3, da + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk), DL_IDESC, (s > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(bar(DL_OP_FREE + h));
                    tc_commit(bar(DL_WEMPTY + i % DL_NSW));
                    if (s == S - 1) tc_commit(bar(DL_SUM_FULL));
                }
                __syncwarp();
            }
        }
    } else {
        // ============================== worker warps ==============================
        const int set = (warp - DL_W0) >> 2;             // takes the slices s with s mod DL_NSET == set
        const int sp = warp & 3;                         // tensor-memory sub-partition: accumulator rows 32*sp .. 32*sp+31
        const int row = 32 * sp + lane;                  // this lane's token row inside the tile
        const uint32_t tlane = (uint32_t)(32 * sp) << 16;
        const uint32_t own_tile = (uint32_t)(row >> 6) * TILE, own_row = (uint32_t)(row & 63);
        const uint32_t up_tile = (uint32_t)((row - 1) >> 6) * TILE, up_row = (uint32_t)((row - 1) & 63);   // (row > 0)
        const uint32_t own_xor = (own_row & 7) << 4;
        const uint32_t out_base = sbase + DL_OFF_OP + set * 2 * TILE + own_tile + own_row * 128;   // this lane's operand row
        const uint32_t slab = sbase + DL_OFF_OP + set * 2 * TILE + sp * 4096;       // pass 3: this warp's 32-row output slab
        const uint32_t h_row = sbase + DL_OFF_H + own_tile + own_row * 128;
        int op_uses = 0;
        bool alive = true;

        // h = tanh(acc) for this warp's 32 rows and this set's share of the 64 columns -> bf16 operand rows
        auto squash = [&](uint32_t tacc) {
            constexpr int HC = 64 / DL_NSET;             // columns per set
#pragma unroll
            for (int g = 0; g < HC / 16; ++g) {
                float a[16];
                tmem_ld_row16(tacc + HC * set + 16 * g, a);
#pragma unroll
                for (int qq = 0; qq < 2; ++qq) {
                    uint32_t ow[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        ow[e] = pack_bf16(tanh_fast(a[8 * qq + 2 * e]), tanh_fast(a[8 * qq + 2 * e + 1]));
                    sts128(h_row + ((uint32_t)((HC / 8 * set + 2 * g + qq) << 4) ^ own_xor), make_uint4(ow[0], ow[1], ow[2], ow[3]));
                }
            }
        };

        int it = 0, ti = 0;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x, ++ti) {
            const long long tok = t * 128 + row;
            const bool seq_start = (tok % p.T) == 0;     // the row above belongs to another sequence: x_prev or zero
            const bool any_start = __any_sync(0xffffffffu, seq_start);
            const __nv_bfloat16* gp0 = (seq_start && p.x_prev && tok < p.rows) ? p.x_prev + (tok / p.T) * (long long)p.D : nullptr;
            // ---- passes 1 and 2: out = x + (x_above - x) * mix, mix = the pass's constants (+ l from tensor memory in pass 2).
            // The interpolation runs on packed bf16 pairs (difference, then one fused multiply-add with a single rounding):
            // its inputs and its output are bf16 anyway, and the mix is smooth in them.
            for (int pass = 0; pass < 2 && alive; ++pass) {
                for (int s = 0; s < S; ++s, ++it) {
                    if (s % DL_NSET != set) continue;
                    const uint32_t stage = sbase + (it % DL_NSX) * DL_XSTAGE;
                    if (!mbar_wait(bar(DL_XFULL + it % DL_NSX), (it / DL_NSX) & 1, abort_flag)) { alive = false; break; }
                    uint32_t mixw[32];                   // the mix of the 64 channels as bf16 pairs
                    if (pass == 1) {
                        const int an = ti * 2 * S + s, a = an % DL_NACC;       // this slice's l: the an-th accumulator made
                        if (!mbar_wait(bar(DL_ACC_FULL + a), (an / DL_NACC) & 1, abort_flag)) { alive = false; break; }
                        tc_fence_after();
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t l[32];
                            kc::tmem_ld_row32(tmem + tlane + DL_TM_RING + 64 * a + 32 * half, l);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float4 v4 = ldsf4(stage + DL_OFF_VEC + 128 * half + 16 * q);
                                mixw[16 * half + 2 * q] = pack_bf16(v4.x + __uint_as_float(l[4 * q]), v4.y + __uint_as_float(l[4 * q + 1]));
                                mixw[16 * half + 2 * q + 1] = pack_bf16(v4.z + __uint_as_float(l[4 * q + 2]), v4.w + __uint_as_float(l[4 * q + 3]));
                            }
                        }
                        tc_fence_before();               // the accumulator row has been read: hand it back
                        __syncwarp();
                        mbar_arrive_if(bar(DL_ACC_FREE + a), lane == 0);
                    } else {
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            const float4 v4 = ldsf4(stage + DL_OFF_VEC + 16 * q);
                            mixw[2 * q] = pack_bf16(v4.x, v4.y);
                            mixw[2 * q + 1] = pack_bf16(v4.z, v4.w);
                        }
                    }
                    // this lane's row and the row above it (inside the tiles, or the extra row of the stage for the tile's
                    // first row), all into registers; then the stage is free for a later slice
                    const uint32_t up_base = row == 0 ? stage + DL_OFF_PREV : stage + up_tile + up_row * 128;
                    const uint32_t up_xor = row == 0 ? 0u : (up_row & 7) << 4;
                    const uint32_t own_base = stage + own_tile + own_row * 128;
                    uint4 a[8], b[8];
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        a[q] = lds128(own_base + ((uint32_t)(q << 4) ^ own_xor));
                        b[q] = lds128(up_base + ((uint32_t)(q << 4) ^ up_xor));
                    }
                    __syncwarp();
                    mbar_arrive_if(bar(DL_XEMPTY + it % DL_NSX), lane == 0);
                    if (any_start && seq_start) {
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            b[q] = gp0 ? *reinterpret_cast<const uint4*>(gp0 + 64 * s + 8 * q) : make_uint4(0u, 0u, 0u, 0u);
                    }
                    // the operand rows: free of the product that read them last (and of this warp's own output store)
                    if (op_uses >= 1 && !mbar_wait(bar(DL_OP_FREE + set), (op_uses - 1) & 1, abort_flag)) { alive = false; break; }
                    ++op_uses;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const uint32_t aw[4] = {a[q].x, a[q].y, a[q].z, a[q].w}, bw[4] = {b[q].x, b[q].y, b[q].z, b[q].w};
                        uint32_t ow[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            uint32_t delta;
                            asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(delta) : "r"(bw[e]), "r"(aw[e]));
                            asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(ow[e]) : "r"(delta), "r"(mixw[4 * q + e]), "r"(aw[e]));
                        }
                        sts128(out_base + ((uint32_t)(q << 4) ^ own_xor), make_uint4(ow[0], ow[1], ow[2], ow[3]));
                    }
                    fence_proxy_async();
                    __syncwarp();
                    mbar_arrive_if(bar(DL_OP_READY + set), lane == 0);
                }
                if (!alive) break;
                // the pass's low-rank sum is complete: squash it into the operand of the next product
                if (!mbar_wait(bar(DL_SUM_FULL), pass, abort_flag)) { alive = false; break; }      // (two uses per tile)
                tc_fence_after();
                squash(tmem + tlane + (pass == 0 ? DL_TM_ACC1 : DL_TM_ACC3));
                fence_proxy_async();
                tc_fence_before();
                __syncwarp();
                mbar_arrive_if(bar(DL_H_READY), lane == 0);
            }
            if (!alive) break;
            // ---- pass 3: d slice -> bf16 slab -> TMA store
            for (int s = 0; s < S; ++s, ++it) {
                if (s % DL_NSET != set) continue;
                const uint32_t stage = sbase + (it % DL_NSX) * DL_XSTAGE;
                if (!mbar_wait(bar(DL_XFULL + it % DL_NSX), (it / DL_NSX) & 1, abort_flag)) { alive = false; break; }
                float lam[64];                           // lambda_w of the slice; then its stage is free
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const float4 v4 = ldsf4(stage + DL_OFF_VEC + 16 * q);
                    lam[4 * q] = v4.x; lam[4 * q + 1] = v4.y; lam[4 * q + 2] = v4.z; lam[4 * q + 3] = v4.w;
                }
                __syncwarp();
                mbar_arrive_if(bar(DL_XEMPTY + it % DL_NSX), lane == 0);
                const int an = ti * 2 * S + S + s, a = an % DL_NACC;          // this slice's d: the an-th accumulator made
                if (!mbar_wait(bar(DL_ACC_FULL + a), (an / DL_NACC) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (lane == 0) bulk_wait_read<0>();      // this warp's previous store has finished reading the slab
                __syncwarp();
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t acc[32];
                    kc::tmem_ld_row32(tmem + tlane + DL_TM_RING + 64 * a + 32 * half, acc);
                    if (half == 1) {
                        tc_fence_before();
                        __syncwarp();
                        mbar_arrive_if(bar(DL_ACC_FREE + a), lane == 0);
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float* lm = lam + 32 * half + 8 * q;
                        sts128(slab + swz(lane, (4 * half + q) << 4),
                               make_uint4(pack_bf16(__uint_as_float(acc[8 * q]) + lm[0], __uint_as_float(acc[8 * q + 1]) + lm[1]),
                                          pack_bf16(__uint_as_float(acc[8 * q + 2]) + lm[2], __uint_as_float(acc[8 * q + 3]) + lm[3]),
                                          pack_bf16(__uint_as_float(acc[8 * q + 4]) + lm[4], __uint_as_float(acc[8 * q + 5]) + lm[5]),
                                          pack_bf16(__uint_as_float(acc[8 * q + 6]) + lm[6], __uint_as_float(acc[8 * q + 7]) + lm[7])));
                    }
                }
                fence_proxy_async();
                __syncwarp();
                const long long grow = t * 128 + 32 * sp;
                if (lane == 0 && grow < p.rows) {
                    tma_store_2d(&tm_d32, 64 * s, (int)grow, slab);
                    bulk_commit();
                }
            }
            // the slab doubles as this warp's operand rows of the next tile
            if (lane == 0) bulk_wait_read<0>();
            __syncwarp();
        }
        if (lane == 0) bulk_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, 512);
    }
}

// [rows][cols] bf16 tensor map with a box of box_rows x box_cols (box_cols * 2 bytes <= 128)
inline bool make_map_box(CUtensorMap* tm, const void* base, long long rows, long long cols, int box_rows, int box_cols, bool swizzle)
{
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace dl

// d = lora_omega(ddlerp_d(x, shifted x)) over rows = B*T tokens of D channels; see the top of this file.
inline gf_status_t decay_logit(const __nv_bfloat16* x, const __nv_bfloat16* x_prev, const float* mu_x,
                               const __nv_bfloat16* A_d, const __nv_bfloat16* B_d, const float* lambda_d,
                               const __nv_bfloat16* A_w, const __nv_bfloat16* B_w, const float* lambda_w,
                               __nv_bfloat16* d, int B, int T, int D, int Rd, int Rw, cudaStream_t st,
                               std::atomic<uint64_t>* launches)
{
    const long long rows = (long long)B * T;
    static PerDeviceFlag attr_set;
    const int dev = current_device();
    if (dev < 0) return GF_ERR_CUDA;
    if (!attr_set.is_set(dev)) {
        if (cudaFuncSetAttribute(dl::decay_logit_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dl::DL_SMEM) != cudaSuccess)
            return GF_ERR_CUDA;
        attr_set.set(dev);
    }
    CUtensorMap tx, tx1, tad, tbd, taw, tbw, td;
    if (!dl::make_map_box(&tx, x, rows, D, 64, 64, true) || !dl::make_map_box(&tx1, x, rows, D, 1, 64, false) ||
        !dl::make_map_box(&tad, A_d, D, Rd, 64, 64, true) || !dl::make_map_box(&tbd, B_d, Rd, D, 64, 64, true) ||
        !dl::make_map_box(&taw, A_w, D, Rw, 64, 64, true) || !dl::make_map_box(&tbw, B_w, Rw, D, 64, 64, true) ||
        !dl::make_map_box(&td, d, rows, D, 32, 64, true))
        return GF_ERR_CUDA;
    dl::DlParams p{rows, T, D / 64, Rd / 16, Rw / 16, x_prev, D, mu_x, lambda_d, lambda_w};
    const long long n_tiles = (rows + 127) / 128;
    const int n_sm = sm_count();
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);
    dl::decay_logit_kernel<<<grid, dl::DL_THREADS, dl::DL_SMEM, st>>>(tx, tx1, tad, tbd, taw, tbw, td, p);
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
