// Gradient of the WKV-6 recurrence in chunks of 64 tokens on the tensor cores (bf16 in and out, fp32 state adjoint).
//
// Forward, per (sequence, head), chunk with start state S_0, in-chunk inclusive cumulative log-decay a_t (a_0 = 0),
// R^_t = r_t e^{a_{t-1}}, K^_i = k_i e^{-a_i}, D = e^{a_L}, b_t = sum_c r_t[c] u[c] k_t[c]:
//   y_t = R^_t S_0 + sum_{i<t} (R^_t . K^_i) v_i + b_t v_t,      S_L = diag(D) (S_0 + K^^T V).
// Backward, chunks from the last to the first, with G_L = dL/dS_L carried (G of the last chunk = dstate_out) and
// G^ = diag(D) G_L, P' = tril(R^ K^^T, -1) + diag(b), dP' = tril(dY V^T, -1), dpd_t = dy_t . v_t:
//   dV  = P'^T dY + K^ G^                                  dv_i = dV_i
//   dR^ = dP' K^ + dY S_0^T                                dr_t = dR^_t e^{a_{t-1}} + u k_t dpd_t
//   dK^ = dP'^T R^ + V G^^T                                dk_i = dK^_i e^{-a_i}    + u r_i dpd_i
//   G_0 = G^ + R^^T dY                                     du  += sum_t r_t k_t dpd_t
// and for the decay, with q_t = dR^_t R^_t, m_t = dK^_t K^_t (per channel) and E = rowsum(G_L * S_L):
//   dL/d(log w_s) = E + sum_{t>s} q_t - sum_{t>=s} m_t,     dx_s = dL/d(log w_s) * log w_s       (log w = -e^x).
// (log w_s enters a_t for every t >= s: R^_t through a_{t-1}, K^_t through a_t, D through a_L; the D term is
// rowsum(G_L * diag(D)(S_0 + K^^T V)) = rowsum(G_L * S_L).)
// Nine 64x64x64 bf16 tcgen05 products per chunk, accumulators in tensor memory.  The chunk-start states S_0 come from
// a checkpoint pass of the forward kernel (state only), one 64x64 fp32 block per chunk.
//
// One CTA of 512 threads per unit works in phases separated by CTA barriers; an elected thread issues the TMA
// copies and the products.  Every elementwise step uses the accumulator layout of the 64-row products: warp
// (sp = warp % 4, cq = warp / 4) owns rows 16 sp .. +15 and columns 16 cq .. +15 of every 64x64 tile, a lane
// (g = lane / 4, q = lane % 4) rows 16 sp + g and + 8, columns 16 cq + 8 n + 2 q + e (n, e in {0, 1}); bf16 tiles
// move through ldmatrix / stmatrix in that layout, so scale factors computed for the operands stay in registers
// until the epilogue needs them.  Sums along the tokens (cumulative decay, the suffix sums of the decay gradient)
// run over lanes by shuffles and over the four row groups through shared memory.
// A chunk in which some channel decays by more than 2^-96 is processed token by token in fp32 on the ALUs (its
// states recomputed into a per-SM scratch in global memory), so any decay logit gives the gradient of the exact
// recurrence.  Every wait is bounded; on expiry the status flag is raised and the whole CTA leaves together.
#pragma once
#include "wkv6_chunked.cuh"

namespace gf {
namespace bc {

using namespace ck;          // PTX wrappers, descriptors, layout helpers of the forward kernel

constexpr bool B_ISSUER = false;                 // a 17th warp issues the products and the TMA copies (else thread 0 does)
constexpr int B_CTHREADS = 512;                  // 16 compute warps
constexpr int B_THREADS = B_CTHREADS + (B_ISSUER ? 32 : 0);
constexpr float LN2 = 0.6931471805599453f;
// tensor memory columns of the six accumulators
constexpr int BT_P = 0, BT_DP = 64, BT_DV = 128, BT_DR = 192, BT_DK = 256, BT_DG = 320, BT_COLS = 512;
// shared memory map (offsets from a 1024-byte aligned base); input stage: x, r, k, v, dy
constexpr int B_STAGE = 5 * TILE;
constexpr int BO_IN = 0;                          // [2][B_STAGE]
constexpr int BO_RH = BO_IN + 2 * B_STAGE;        // [2] R^ [t][c]        (by chunk parity, like the input stages)
constexpr int BO_KH = BO_RH + 2 * TILE;           // [2] K^ [i][c]
constexpr int BO_SB = BO_KH + 2 * TILE;           // [2] S_0 [c][j] bf16
constexpr int BO_GB = BO_SB + 2 * TILE;           // [2] G^  [c][j] bf16
constexpr int BO_PP = BO_GB + 2 * TILE;           // P' [t][i]
constexpr int BO_DPP = BO_PP + TILE;              // dP' [t][i]
constexpr int BO_OUT = BO_DPP + TILE;             // dr, dk, dv, dx staging [t][c]
constexpr int BO_TOT = BO_OUT + 4 * TILE;         // [4][64] float: row-group totals of a scan
constexpr int BO_EP = BO_TOT + 1024;              // [2][4][64] float: partial E by column group (by chunk parity)
constexpr int BO_BP = BO_EP + 2048;               // [4][64] float: partial bonus by column group
constexpr int BO_DPD = BO_BP + 1024;              // [64] float: dy_t . v_t
constexpr int BO_RED = BO_DPD + 256;              // token-by-token path: [4][3][64] + [4][64] + du[64] + 2 floats
constexpr int BO_RED_V = BO_RED + 4 * 3 * 64 * 4;
constexpr int BO_DU_FB = BO_RED_V + 4 * 64 * 4;
constexpr int BO_SCAL = BO_DU_FB + 256;
constexpr int BO_ABORT = BO_SCAL + 16;            // abort word, wait limit
constexpr int BO_TMEM = BO_ABORT + 8;
constexpr int BO_CMD = BO_TMEM + 8;               // [4] {command, argument} for the issuing warp
constexpr int BO_BAR = BO_CMD + 32;               // mbarriers: input full [2], first / second group of products done,
// ... staging tiles read by the TMA unit, command slots [4]
enum { BB_IN = 0, BB_MMA1 = 2, BB_MMA2 = 3, BB_STAGING = 4, BB_CMD = 5, BB_COUNT = 9 };
enum { CMD_QUIT = 0, CMD_MMA1 = 1, CMD_MMA2 = 2, CMD_STORE = 3 };
constexpr int B_SMEM_BYTES = BO_BAR + 8 * BB_COUNT;
constexpr int B_SMEM_ALLOC = B_SMEM_BYTES + 1024;
static_assert(B_SMEM_ALLOC <= 232448, "shared memory budget of one sm_100 CTA");
constexpr size_t FB_SLOT_FLOATS = (size_t)64 * 4096;      // scratch of the token-by-token path per SM: 64 states

struct BParams {
    const float* u;              // [H][64]
    const float* dstate_out;     // [units][64][64] or NULL (zero)
    float* dstate_in;            // [units][64][64] or NULL (not written)
    const float* ckpt;           // [units][chunks + 1][64][64]
    float* du_part;              // [units][64]
    float* fb_scratch;           // [n_slots][64][4096]
    __nv_bfloat16 *dr, *dk, *dv, *dx;
    int T, H, n_slots;
    uint32_t wait_limit_us;
};

__device__ __forceinline__ float lds_bf16(uint32_t a)
{
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a) : "memory");
    return __uint_as_float((uint32_t)v << 16);
}
__device__ __forceinline__ void sts_bf16(uint32_t a, float f)
{
    const __nv_bfloat16 b = __float2bfloat16_rn(f);
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"(*reinterpret_cast<const uint16_t*>(&b)) : "memory");
}
__device__ __forceinline__ void lds_v4(uint32_t a, uint32_t (&w)[4])
{
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(a) : "memory");
}
__device__ __forceinline__ unsigned smid()
{
    unsigned v;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(v));
    return v;
}

// Barrier over the 16 compute warps (the issuing warp does not take part), and the same with an AND over a predicate.
__device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, 512;" ::: "memory"); }
__device__ __forceinline__ bool cbar_and(bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.and.pred q, 1, 512, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"((uint32_t)ok) : "memory");
    return r != 0;
}

// 1 - 2^l for l <= 0 without the cancellation of the direct form near l = 0 (slow decays): the series of -expm1 there.
__device__ __forceinline__ float one_minus_ex2(float l)
{
    const float t = l * LN2;
    const float series = -t * (1.f + t * (0.5f + t * (0.16666667f + t * 0.041666668f)));
    return l > -0.125f ? series : 1.f - ex2(l);
}

// tcgen05.ld of a 16 x 16 fp32 block without the wait for its data (tmem_ld_done() before the first use): several
// loads can then be in flight together.
__device__ __forceinline__ void tmem_ld_16x16_async(uint32_t taddr, float (&v)[2][4])
{
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0][0]), "=f"(v[0][1]), "=f"(v[0][2]), "=f"(v[0][3]), "=f"(v[1][0]), "=f"(v[1][1]), "=f"(v[1][2]), "=f"(v[1][3])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_done() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// v[n][0..1] = (row g, columns 8n+2q, +1), v[n][2..3] = (row g+8, same columns) of this warp's 16 x 16 block
__device__ __forceinline__ void load_block_bf16(uint32_t addr, float (&v)[2][4])
{
    uint32_t w0, w1, w2, w3;
    ldsm_x4(addr, w0, w1, w2, w3);
    v[0][0] = bf_lo(w0); v[0][1] = bf_hi(w0); v[0][2] = bf_lo(w1); v[0][3] = bf_hi(w1);
    v[1][0] = bf_lo(w2); v[1][1] = bf_hi(w2); v[1][2] = bf_lo(w3); v[1][3] = bf_hi(w3);
}
__device__ __forceinline__ void store_block_bf16(uint32_t addr, const float (&v)[2][4])
{
    stsm_x4(addr, pack_bf16(v[0][0], v[0][1]), pack_bf16(v[0][2], v[0][3]), pack_bf16(v[1][0], v[1][1]), pack_bf16(v[1][2], v[1][3]));
}

// Inclusive sums along the 64 rows of a tile held in the accumulator layout: forwards (REV = false: row t gets the
// sum over rows <= t) or backwards (REV = true: rows >= t).  tot: [4][64] floats of shared memory.  Contains one
// barrier of the compute warps (all 512 threads call it together), which also forms the AND of `ok` over them: the
// result is returned (a wait that ran out on some thread makes every thread leave together).
template <bool REV>
__device__ __forceinline__ bool scan_rows(float (&v)[2][4], uint32_t tot, int sp, int cq, int lane, bool ok)
{
    const int g = lane >> 2, q = lane & 3;
#pragma unroll
    for (int d = 4; d < 32; d <<= 1) {
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float o = REV ? __shfl_down_sync(0xffffffffu, v[n][e], d) : __shfl_up_sync(0xffffffffu, v[n][e], d);
                if (REV ? lane + d < 32 : lane >= d) v[n][e] += o;
            }
    }
    // the other half's total: rows g+8 follow rows g
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if (REV) v[n][e] += __shfl_sync(0xffffffffu, v[n][2 + e], q);
            else v[n][2 + e] += __shfl_sync(0xffffffffu, v[n][e], 28 + q);
        }
    if (g == (REV ? 0 : 7)) {
#pragma unroll
        for (int n = 0; n < 2; ++n)
            *reinterpret_cast<float2*>(__cvta_shared_to_generic((size_t)(tot + 4 * (sp * 64 + 16 * cq + 8 * n + 2 * q)))) =
                REV ? make_float2(v[n][0], v[n][1]) : make_float2(v[n][2], v[n][3]);
    }
    ok = cbar_and(ok);
#pragma unroll
    for (int o = 0; o < 4; ++o) {
        if (REV ? o > sp : o < sp) {
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                const float2 t = *reinterpret_cast<const float2*>(__cvta_shared_to_generic((size_t)(tot + 4 * (o * 64 + 16 * cq + 8 * n + 2 * q))));
                v[n][0] += t.x; v[n][1] += t.y; v[n][2] += t.x; v[n][3] += t.y;
            }
        }
    }
    return ok;
}

// C2 = true: the Finch-C2 form (keys times one minus their decay, no bonus; the second-value vector only adds to the
// output, so its gradient is dy itself and nothing here depends on it).
template <bool C2>
__global__ void __launch_bounds__(B_THREADS, 1)
wkv6_backward_chunked_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_r,
                             const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                             const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_dr,
                             const __grid_constant__ CUtensorMap tm_dk, const __grid_constant__ CUtensorMap tm_dv,
                             const __grid_constant__ CUtensorMap tm_dx, const BParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t abort_flag = sbase + BO_ABORT;
    auto bar = [&](int i) { return sbase + BO_BAR + 8 * i; };
    auto fsm = [&](int off) { return reinterpret_cast<float*>(smem + off); };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int sp = warp & 3, cq = warp >> 2, g = lane >> 2, q = lane & 3;
    const int unit = blockIdx.x, seq = unit / p.H, h = unit % p.H;
    const int T = p.T, nchunks = (T + L - 1) / L;
    const long long row0 = (long long)seq * T;
    const int col0 = h * 64;
    const size_t C = (size_t)p.H * 64;
    const int R0 = 16 * sp + g, R1 = R0 + 8;         // this lane's two rows
    const int cb = 16 * cq + 2 * q;                  // its columns: cb + 8 n + e
    // byte offset of this lane's ldmatrix / stmatrix row inside a tile (the warp's 16 x 16 block)
    const uint32_t moff = swz(16 * sp + (lane & 7) + 8 * ((lane >> 3) & 1), (2 * cq + (lane >> 4)) << 4);

    if (tid == 0) {
        for (int i = 0; i < BB_COUNT; ++i) mbar_init(bar(i), 1);
        sts32(abort_flag, 0u);
        sts32(abort_flag + 4, p.wait_limit_us ? p.wait_limit_us : WAIT_LIMIT_US);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (tid < 64) fsm(BO_DU_FB)[tid] = 0.f;
    if (warp == 1) tmem_alloc(sbase + BO_TMEM, BT_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32(sbase + BO_TMEM);
    const uint32_t tacc = tmem + ((uint32_t)(32 * sp) << 16) + 16 * cq;      // this warp's block of an accumulator

    // Chunks are numbered by iteration: iteration `it` handles chunk nchunks - 1 - it; its input stage and the
    // double-buffered operand tiles are those of parity it & 1.
    auto chunk_of = [&](int it) { return nchunks - 1 - it; };

    // ---- issuing: the products, the TMA stores of a chunk's gradient tiles and the input copies.  With B_ISSUER a
    // warp of its own does it: one lane takes commands from the compute warps (a ring of four slots, one mbarrier each:
    // at most three are ever outstanding), so that no compute warp waits for an instruction to be issued, only for
    // its completion.  Without it thread 0 issues in place.
    int last_load[2] = {-1, -1};                     // (issuing thread) per stage: the last iteration whose copies were issued
    auto issue_loads = [&](int it) {
        const int stage = it & 1;
        const uint32_t dst = sbase + BO_IN + stage * B_STAGE;
        const int row = (int)(row0 + (long long)chunk_of(it) * L);
        mbar_expect_tx(bar(BB_IN + stage), B_STAGE);
        tma_load_2d(dst, &tm_x, col0, row, bar(BB_IN + stage));
        tma_load_2d(dst + TILE, &tm_r, col0, row, bar(BB_IN + stage));
        tma_load_2d(dst + 2 * TILE, &tm_k, col0, row, bar(BB_IN + stage));
        tma_load_2d(dst + 3 * TILE, &tm_v, col0, row, bar(BB_IN + stage));
        tma_load_2d(dst + 4 * TILE, &tm_dy, col0, row, bar(BB_IN + stage));
        last_load[stage] = it;
    };
    auto execute = [&](uint32_t cmd, uint32_t arg) {
        if (cmd == CMD_MMA1 || cmd == CMD_MMA2) {
            const int pb = (int)arg;
            const uint32_t tin = sbase + BO_IN + pb * B_STAGE;
            const uint64_t dR = smem_desc(sbase + BO_RH + pb * TILE), dK = smem_desc(sbase + BO_KH + pb * TILE);
            const uint64_t dV = smem_desc(tin + 3 * TILE), dY = smem_desc(tin + 4 * TILE);
            tc_fence_after();
            if (cmd == CMD_MMA1) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk, ms = 128 * kk;       // K-major / MN-major step of 16 contraction indices
                    tc_mma(tmem + BT_P, dR + ks, dK + ks, IDESC_K_K, kk > 0);          // P[t][i]  = R^ K^^T
                    tc_mma(tmem + BT_DP, dY + ks, dV + ks, IDESC_K_K, kk > 0);         // dP[t][i] = dY V^T
                    tc_mma(tmem + BT_DG, dR + ms, dY + ms, IDESC_MN_MN, kk > 0);       // dG[c][j] = R^^T dY
                }
                tc_commit(bar(BB_MMA1));
            } else {
                const uint64_t dS = smem_desc(sbase + BO_SB + pb * TILE), dG = smem_desc(sbase + BO_GB + pb * TILE);
                const uint64_t dP = smem_desc(sbase + BO_PP), dD = smem_desc(sbase + BO_DPP);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk, ms = 128 * kk;
                    tc_mma(tmem + BT_DV, dK + ks, dG + ms, IDESC_K_MN, kk > 0);        // dV[i][j] = K^ G^
                    tc_mma(tmem + BT_DR, dY + ks, dS + ks, IDESC_K_K, kk > 0);         // dR[t][c] = dY S_0^T
                    tc_mma(tmem + BT_DK, dV + ks, dG + ks, IDESC_K_K, kk > 0);         // dK[i][c] = V G^^T
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk, ms = 128 * kk;
                    tc_mma(tmem + BT_DV, dP + ms, dY + ms, IDESC_MN_MN, 1);            // dV += P'^T dY
                    tc_mma(tmem + BT_DR, dD + ks, dK + ms, IDESC_K_MN, 1);             // dR += dP' K^
                    tc_mma(tmem + BT_DK, dD + ms, dR + ms, IDESC_MN_MN, 1);            // dK += dP'^T R^
                }
                tc_commit(bar(BB_MMA2));
            }
        } else {                             // CMD_STORE: arg = iteration, bit 31: whole chunk (TMA stores)
            const int it = (int)(arg & 0x7fffffffu);
            const bool whole = (arg >> 31) != 0;
            if (whole) {
                const int row = (int)(row0 + (long long)chunk_of(it) * L);
                tma_store_2d(&tm_dr, col0, row, sbase + BO_OUT);
                tma_store_2d(&tm_dk, col0, row, sbase + BO_OUT + TILE);
                tma_store_2d(&tm_dv, col0, row, sbase + BO_OUT + 2 * TILE);
                tma_store_2d(&tm_dx, col0, row, sbase + BO_OUT + 3 * TILE);
                bulk_commit();
            }
            if (it + 2 < nchunks) issue_loads(it + 2);
            if (B_ISSUER) {
                if (whole) bulk_wait_read<0>();      // the staging tiles may be rewritten
                mbar_arrive(bar(BB_STAGING));
            }
        }
    };
    auto issuer_done = [&]() {
        bulk_wait<0>();                              // the gradient tiles have reached memory
        for (int s2 = 0; s2 < 2; ++s2)               // no copy into this CTA's shared memory may stay in flight
            if (last_load[s2] >= 0) mbar_wait(bar(BB_IN + s2), (last_load[s2] >> 1) & 1, abort_flag, false);
    };
    if (B_ISSUER ? (warp == B_CTHREADS / 32 && lane == 0) : tid == 0) {
        if (nchunks > 0) issue_loads(0);
        if (nchunks > 1) issue_loads(1);
    }

    if (B_ISSUER && warp == B_CTHREADS / 32) {
        // ============================== issuing warp ==============================
        if (lane == 0) {
            for (int kc = 0;; ++kc) {
                if (!mbar_wait(bar(BB_CMD + (kc & 3)), (kc >> 2) & 1, abort_flag)) break;
                const uint32_t cmd = lds32(sbase + BO_CMD + 8 * (kc & 3)), arg = lds32(sbase + BO_CMD + 8 * (kc & 3) + 4);
                if (cmd == CMD_QUIT) break;
                execute(cmd, arg);
            }
            issuer_done();
        }
    } else {
    // ============================== compute warps ==============================
    // Every thread waits for itself on an mbarrier; the outcomes are made uniform at the next barrier of the compute
    // warps (cbar_and), so that after a wait that ran out all of them leave together.
    int n_cmd = 0;                                   // (thread 0) commands posted so far
    auto post = [&](uint32_t cmd, uint32_t arg) {    // thread 0, after a barrier that follows the operands' writes
        if (!B_ISSUER) {
            if (cmd != CMD_QUIT) execute(cmd, arg); else issuer_done();
            return;
        }
        const uint32_t slot = sbase + BO_CMD + 8 * (n_cmd & 3);
        sts32(slot, cmd);
        sts32(slot + 4, arg);
        mbar_arrive(bar(BB_CMD + (n_cmd & 3)));
        ++n_cmd;
    };
    int n_store = 0;                                 // store commands posted so far (every thread counts)
    auto load_f32_block = [&](const float* src, float (&v)[2][4]) {      // [64][64] fp32 block, accumulator layout
#pragma unroll
        for (int n = 0; n < 2; ++n) {
            const float2 lo = *reinterpret_cast<const float2*>(src + (size_t)R0 * 64 + cb + 8 * n);
            const float2 hi = *reinterpret_cast<const float2*>(src + (size_t)R1 * 64 + cb + 8 * n);
            v[n][0] = lo.x; v[n][1] = lo.y; v[n][2] = hi.x; v[n][3] = hi.y;
        }
    };

    float uu[2][2];                                  // bonus of this lane's columns (as channels)
#pragma unroll
    for (int n = 0; n < 2; ++n) { uu[n][0] = C2 ? 0.f : p.u[col0 + cb + 8 * n]; uu[n][1] = C2 ? 0.f : p.u[col0 + cb + 8 * n + 1]; }
    float G[2][4], SL[2][4], du_acc[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    const float* ck_unit = p.ckpt + (size_t)unit * (nchunks + 1) * 4096;
    if (p.dstate_out) load_f32_block(p.dstate_out + (size_t)unit * 4096, G);
    else {
#pragma unroll
        for (int n = 0; n < 2; ++n) G[n][0] = G[n][1] = G[n][2] = G[n][3] = 0.f;
    }
    load_f32_block(ck_unit + (size_t)nchunks * 4096, SL);
    int mph1 = 0, mph2 = 0;                          // phase bits of the two product barriers
    bool alive = true;

    // ---- operands of a chunk from its inputs and from the adjoint G = G_L at its end; first group of products.
    // Returns 0 (products issued), 1 (the chunk decays too fast for this form: nothing issued) or -1 (a wait ran out).
    // On return SL holds the chunk's start state; a, lw2 its cumulative and per-token log2 decays in this lane's cells.
    auto prepare = [&](int it, float (&a)[2][4], float (&lw2)[2][4], float (&dch)[2]) -> int {
        const int c = chunk_of(it), pb = it & 1;
        const int valid = min(L, T - c * L);
        const uint32_t tin = sbase + BO_IN + pb * B_STAGE;
        const uint32_t tx = tin, tr = tin + TILE, tk = tin + 2 * TILE, tv = tin + 3 * TILE, tdy = tin + 4 * TILE;
        const uint32_t t_rh = sbase + BO_RH + pb * TILE, t_kh = sbase + BO_KH + pb * TILE;
        const uint32_t t_sb = sbase + BO_SB + pb * TILE, t_gb = sbase + BO_GB + pb * TILE;
        float S0[2][4];
        load_f32_block(ck_unit + (size_t)c * 4096, S0);
        if (c > 0 && tid < 128)                      // the next chunk's start state: in L2 by the time it is loaded
            asm volatile("prefetch.global.L2 [%0];" ::"l"(ck_unit + (size_t)(c - 1) * 4096 + 32 * tid));
        // E = rowsum(G_L * S_L): partial over this lane's columns, then over the four lanes of a row
        {
            float e0 = 0.f, e1 = 0.f;
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                e0 = fmaf(G[n][0], SL[n][0], fmaf(G[n][1], SL[n][1], e0));
                e1 = fmaf(G[n][2], SL[n][2], fmaf(G[n][3], SL[n][3], e1));
            }
            e0 += __shfl_xor_sync(0xffffffffu, e0, 1); e1 += __shfl_xor_sync(0xffffffffu, e1, 1);
            e0 += __shfl_xor_sync(0xffffffffu, e0, 2); e1 += __shfl_xor_sync(0xffffffffu, e1, 2);
            if (q == 0) { fsm(BO_EP)[(pb * 4 + cq) * 64 + R0] = e0; fsm(BO_EP)[(pb * 4 + cq) * 64 + R1] = e1; }
        }
        bool ok = mbar_wait(bar(BB_IN + pb), (it >> 1) & 1, abort_flag);
        if (valid < L) {
            // ragged last chunk: the rows past the sequence's end hold other tokens (or the out-of-range fill)
            for (int i = tid; i < (L - valid) * 8; i += B_CTHREADS) {
                const uint32_t o = (valid + (i >> 3)) * 128 + ((i & 7) << 4);
                sts128z(tr + o); sts128z(tk + o); sts128z(tv + o); sts128z(tdy + o);
            }
        }
        // decay: log2-domain magnitudes, cumulative sums over the tokens
        {
            float xv[2][4];
            load_block_bf16(tx + moff, xv);
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool live = (e < 2 ? R0 : R1) < valid;
                    lw2[n][e] = live ? -ex2(fmaf(xv[n][e], LOG2E, LOG2_LOG2E)) : 0.f;
                    a[n][e] = lw2[n][e];
                }
        }
        ok = scan_rows<false>(a, sbase + BO_TOT, sp, cq, lane, ok);      // (barrier: the zeroed rows are visible after it)
        if (!ok) return -1;
        // a_L = the sum of the four row-group totals; this lane needs it for the channels that are its rows of G
        bool safe;
        {
            float al0 = 0.f, al1 = 0.f;
#pragma unroll
            for (int o = 0; o < 4; ++o) { al0 += fsm(BO_TOT)[o * 64 + R0]; al1 += fsm(BO_TOT)[o * 64 + R1]; }
            dch[0] = ex2(al0); dch[1] = ex2(al1);
            safe = (al0 >= -A2_MAX) && (al1 >= -A2_MAX);                   // false for NaN as well
        }
        {
            float rv[2][4], kv[2][4];
            load_block_bf16(tr + moff, rv);
            load_block_bf16(tk + moff, kv);
            float b0 = 0.f, b1 = 0.f;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (C2) kv[n][e] *= one_minus_ex2(lw2[n][e]);      // the key that enters the state
                    const float t = rv[n][e] * kv[n][e] * uu[n][e & 1];
                    if (e < 2) b0 += t; else b1 += t;
                    rv[n][e] *= ex2(a[n][e] - lw2[n][e]);
                    kv[n][e] *= ex2(-a[n][e]);
                }
            store_block_bf16(t_rh + moff, rv);
            store_block_bf16(t_kh + moff, kv);
            b0 += __shfl_xor_sync(0xffffffffu, b0, 1); b1 += __shfl_xor_sync(0xffffffffu, b1, 1);
            b0 += __shfl_xor_sync(0xffffffffu, b0, 2); b1 += __shfl_xor_sync(0xffffffffu, b1, 2);
            if (q == 0) { fsm(BO_BP)[cq * 64 + R0] = b0; fsm(BO_BP)[cq * 64 + R1] = b1; }
        }
        store_block_bf16(t_sb + moff, S0);
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) SL[n][e] = S0[n][e];
        {
            float gh[2][4];
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                gh[n][0] = dch[0] * G[n][0]; gh[n][1] = dch[0] * G[n][1];
                gh[n][2] = dch[1] * G[n][2]; gh[n][3] = dch[1] * G[n][3];
            }
            store_block_bf16(t_gb + moff, gh);
        }
        fence_proxy_async();
        tc_fence_before();
        const bool unsafe = !cbar_and(safe);         // (every channel is some lane's row)
        if (tid == 0 && !unsafe) post(CMD_MMA1, (uint32_t)pb);
        return unsafe ? 1 : 0;
    };

    // ---- the chunk's four gradient tiles leave: TMA for a whole chunk, plain stores for a ragged one; then the
    // input stage of this iteration is free for the chunk two iterations on.
    auto store_and_refill = [&](int it) {
        const int c = chunk_of(it), valid = min(L, T - c * L);
        fence_proxy_async();
        cbar();
        if (valid < L) {
            __nv_bfloat16* outs[4] = {p.dr, p.dk, p.dv, p.dx};
            for (int i = tid; i < 4 * valid * 8; i += B_CTHREADS) {
                const int tile = i / (valid * 8), rem = i % (valid * 8), t = rem >> 3, blk = rem & 7;
                uint32_t w[4];
                lds_v4(sbase + BO_OUT + tile * TILE + swz(t, blk << 4), w);
                *reinterpret_cast<uint4*>(outs[tile] + (size_t)(row0 + (long long)c * L + t) * C + col0 + 8 * blk) = make_uint4(w[0], w[1], w[2], w[3]);
            }
        }
        if (tid == 0) post(CMD_STORE, (uint32_t)it | (valid == L ? 0x80000000u : 0u));
        ++n_store;
    };
    // The staging tiles may be rewritten once the TMA unit has read the previous chunk's (a barrier of the compute
    // warps follows in every caller, which also orders a ragged chunk's plain reads before the rewrite).
    auto staging_free = [&]() -> bool {
        if (!B_ISSUER) {                             // thread 0 issued the stores itself: it waits for their reads
            if (tid == 0) bulk_wait_read<0>();
            return true;
        }
        return n_store == 0 || mbar_wait(bar(BB_STAGING), (n_store - 1) & 1, abort_flag);
    };

    float a_cur[2][4], lw_cur[2][4], d_cur[2];       // of the chunk in flight: cumulative / per-token log2 decays, chunk decay
    int st = nchunks > 0 ? prepare(0, a_cur, lw_cur, d_cur) : 0;
    if (st < 0) alive = false;

    for (int it = 0; alive && it < nchunks; ++it) {
        const int c = chunk_of(it), pb = it & 1;
        const int valid = min(L, T - c * L);
        const uint32_t tin = sbase + BO_IN + pb * B_STAGE;
        const uint32_t tx = tin, tr = tin + TILE, tk = tin + 2 * TILE, tv = tin + 3 * TILE, tdy = tin + 4 * TILE;
        const uint32_t t_rh = sbase + BO_RH + pb * TILE, t_kh = sbase + BO_KH + pb * TILE;

        if (st == 1) {
            // ---- token by token: the chunk's states recomputed into this SM's scratch, then the reverse recurrence
            const unsigned slot = smid();
            if (slot >= (unsigned)p.n_slots) {       // (no scratch for this SM: report it and leave)
                if (tid == 0) { sts32(abort_flag, 1u); atomicExch(&g_dev_status, 1); }
                alive = false;
                break;
            }
            if (!cbar_and(staging_free())) { alive = false; break; }
            float* scr = p.fb_scratch + (size_t)slot * FB_SLOT_FLOATS + (size_t)tid * 8;
            // rows are key channels here: this lane's channels R0, R1 of S and G; its columns are value channels
            float S[2][4];
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) S[n][e] = SL[n][e];
            for (int t = 0; t < valid; ++t) {
                *reinterpret_cast<float4*>(scr + (size_t)t * 4096) = make_float4(S[0][0], S[0][1], S[0][2], S[0][3]);
                *reinterpret_cast<float4*>(scr + (size_t)t * 4096 + 4) = make_float4(S[1][0], S[1][1], S[1][2], S[1][3]);
                const float e0 = expf(lds_bf16(tx + swz(t, 2 * R0))), e1 = expf(lds_bf16(tx + swz(t, 2 * R1)));
                const float w0 = expf(-e0), w1 = expf(-e1);
                float k0 = lds_bf16(tk + swz(t, 2 * R0)), k1 = lds_bf16(tk + swz(t, 2 * R1));
                if (C2) { k0 *= -expm1f(-e0); k1 *= -expm1f(-e1); }
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float vj = lds_bf16(tv + swz(t, 2 * (cb + 8 * n + e)));
                        S[n][e] = fmaf(w0, S[n][e], k0 * vj);
                        S[n][2 + e] = fmaf(w1, S[n][2 + e], k1 * vj);
                    }
            }
            float* red = fsm(BO_RED);                // [cq][3][64]
            float* redv = fsm(BO_RED_V);             // [sp][64]
            float* scal = fsm(BO_SCAL);              // v . dy, sum r u k
            for (int t = valid - 1; t >= 0; --t) {
                const float4 sa = *reinterpret_cast<const float4*>(scr + (size_t)t * 4096);
                const float4 sb4 = *reinterpret_cast<const float4*>(scr + (size_t)t * 4096 + 4);
                const float Sp[2][4] = {{sa.x, sa.y, sa.z, sa.w}, {sb4.x, sb4.y, sb4.z, sb4.w}};
                const float x0 = lds_bf16(tx + swz(t, 2 * R0)), x1 = lds_bf16(tx + swz(t, 2 * R1));
                const float w0 = expf(-expf(x0)), w1 = expf(-expf(x1));
                float k0 = lds_bf16(tk + swz(t, 2 * R0)), k1 = lds_bf16(tk + swz(t, 2 * R1));
                if (C2) { k0 *= -expm1f(-expf(x0)); k1 *= -expm1f(-expf(x1)); }
                const float r0 = lds_bf16(tr + swz(t, 2 * R0)), r1 = lds_bf16(tr + swz(t, 2 * R1));
                float pr0 = 0.f, pr1 = 0.f, pk0 = 0.f, pk1 = 0.f, pg0 = 0.f, pg1 = 0.f, pv[2][2];
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int j = cb + 8 * n + e;
                        const float vj = lds_bf16(tv + swz(t, 2 * j)), dyj = lds_bf16(tdy + swz(t, 2 * j));
                        pr0 = fmaf(dyj, Sp[n][e], pr0); pr1 = fmaf(dyj, Sp[n][2 + e], pr1);
                        pk0 = fmaf(G[n][e], vj, pk0); pk1 = fmaf(G[n][2 + e], vj, pk1);
                        pg0 = fmaf(G[n][e], Sp[n][e], pg0); pg1 = fmaf(G[n][2 + e], Sp[n][2 + e], pg1);
                        pv[n][e] = fmaf(G[n][e], k0, G[n][2 + e] * k1);
                        G[n][e] = fmaf(w0, G[n][e], r0 * dyj);
                        G[n][2 + e] = fmaf(w1, G[n][2 + e], r1 * dyj);
                    }
#pragma unroll
                for (int d = 1; d < 4; d <<= 1) {
                    pr0 += __shfl_xor_sync(0xffffffffu, pr0, d); pr1 += __shfl_xor_sync(0xffffffffu, pr1, d);
                    pk0 += __shfl_xor_sync(0xffffffffu, pk0, d); pk1 += __shfl_xor_sync(0xffffffffu, pk1, d);
                    pg0 += __shfl_xor_sync(0xffffffffu, pg0, d); pg1 += __shfl_xor_sync(0xffffffffu, pg1, d);
                }
#pragma unroll
                for (int d = 4; d < 32; d <<= 1)
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) pv[n][e] += __shfl_xor_sync(0xffffffffu, pv[n][e], d);
                if (q == 0) {
                    red[(cq * 3 + 0) * 64 + R0] = pr0; red[(cq * 3 + 0) * 64 + R1] = pr1;
                    red[(cq * 3 + 1) * 64 + R0] = pk0; red[(cq * 3 + 1) * 64 + R1] = pk1;
                    red[(cq * 3 + 2) * 64 + R0] = pg0; red[(cq * 3 + 2) * 64 + R1] = pg1;
                }
                if (g == 0) {
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) redv[sp * 64 + cb + 8 * n + e] = pv[n][e];
                }
                if (warp == 0) {
                    float vd = 0.f, ruk = 0.f;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int cc = 2 * lane + e;
                        vd = fmaf(lds_bf16(tv + swz(t, 2 * cc)), lds_bf16(tdy + swz(t, 2 * cc)), vd);
                        if (!C2) ruk = fmaf(lds_bf16(tr + swz(t, 2 * cc)) * p.u[col0 + cc], lds_bf16(tk + swz(t, 2 * cc)), ruk);
                    }
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        vd += __shfl_xor_sync(0xffffffffu, vd, d);
                        ruk += __shfl_xor_sync(0xffffffffu, ruk, d);
                    }
                    if (lane == 0) { scal[0] = vd; scal[1] = ruk; }
                }
                cbar();
                if (tid < 64) {
                    const int cc = tid;
                    float s_r = 0.f, s_k = 0.f, s_g = 0.f;
#pragma unroll
                    for (int o = 0; o < 4; ++o) { s_r += red[(o * 3 + 0) * 64 + cc]; s_k += red[(o * 3 + 1) * 64 + cc]; s_g += red[(o * 3 + 2) * 64 + cc]; }
                    const float xc = lds_bf16(tx + swz(t, 2 * cc)), kc = lds_bf16(tk + swz(t, 2 * cc)), rc = lds_bf16(tr + swz(t, 2 * cc));
                    const float ec = expf(xc), wc = expf(-ec);
                    if (C2) {
                        sts_bf16(sbase + BO_OUT + swz(t, 2 * cc), s_r);
                        sts_bf16(sbase + BO_OUT + TILE + swz(t, 2 * cc), s_k * -expm1f(-ec));
                        sts_bf16(sbase + BO_OUT + 3 * TILE + swz(t, 2 * cc), (s_g - s_k * kc) * (-wc * ec));
                    } else {
                        const float uc = p.u[col0 + cc], vd = scal[0];
                        sts_bf16(sbase + BO_OUT + swz(t, 2 * cc), fmaf(uc * kc, vd, s_r));
                        sts_bf16(sbase + BO_OUT + TILE + swz(t, 2 * cc), fmaf(rc * uc, vd, s_k));
                        sts_bf16(sbase + BO_OUT + 3 * TILE + swz(t, 2 * cc), s_g * (-wc * ec));
                        fsm(BO_DU_FB)[cc] = fmaf(rc * kc, vd, fsm(BO_DU_FB)[cc]);
                    }
                } else if (tid < 128) {
                    const int j = tid - 64;
                    const float s_v = redv[j] + redv[64 + j] + redv[128 + j] + redv[192 + j];
                    sts_bf16(sbase + BO_OUT + 2 * TILE + swz(t, 2 * j), fmaf(scal[1], lds_bf16(tdy + swz(t, 2 * j)), s_v));
                }
                cbar();
            }
            store_and_refill(it);
            if (it + 1 < nchunks) {
                st = prepare(it + 1, a_cur, lw_cur, d_cur);
                if (st < 0) alive = false;
            }
            continue;
        }

        // ---- masked scores and their adjoint as operands
        bool ok = mbar_wait(bar(BB_MMA1), mph1, abort_flag);
        mph1 ^= 1;
        tc_fence_after();
        if (cq < sp) {
            // a block below the diagonal: every score and every adjoint entry is kept
            float pp[2][4], dp[2][4];
            tmem_ld_16x16_async(tacc + BT_P, pp);
            tmem_ld_16x16_async(tacc + BT_DP, dp);
            tmem_ld_done();
            store_block_bf16(sbase + BO_PP + moff, pp);
            store_block_bf16(sbase + BO_DPP + moff, dp);
        } else if (cq > sp) {
            // above the diagonal: masked out
            stsm_x4(sbase + BO_PP + moff, 0u, 0u, 0u, 0u);
            stsm_x4(sbase + BO_DPP + moff, 0u, 0u, 0u, 0u);
        } else {
            float pp[2][4], dp[2][4];
            tmem_ld_16x16_async(tacc + BT_P, pp);
            tmem_ld_16x16_async(tacc + BT_DP, dp);
            float bon0 = 0.f, bon1 = 0.f;
#pragma unroll
            for (int o = 0; o < 4; ++o) { bon0 += fsm(BO_BP)[o * 64 + R0]; bon1 += fsm(BO_BP)[o * 64 + R1]; }
            tmem_ld_done();
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int row = e < 2 ? g : g + 8, col = 2 * q + 8 * n + (e & 1);       // inside the 16 x 16 block
                    if (col == row) fsm(BO_DPD)[16 * sp + row] = dp[n][e];
                    pp[n][e] = col < row ? pp[n][e] : (col == row ? (e < 2 ? bon0 : bon1) : 0.f);
                    dp[n][e] = col < row ? dp[n][e] : 0.f;
                }
            store_block_bf16(sbase + BO_PP + moff, pp);
            store_block_bf16(sbase + BO_DPP + moff, dp);
        }
        fence_proxy_async();
        tc_fence_before();
        if (!cbar_and(ok)) { alive = false; break; }
        if (tid == 0) post(CMD_MMA2, (uint32_t)pb);
        // ---- G_0 = diag(D) G_L + R^^T dY
        {
            const float d_lo = d_cur[0], d_hi = d_cur[1];
            float dg[2][4];
            tmem_ld_16x16(tacc + BT_DG, dg);
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                G[n][0] = fmaf(d_lo, G[n][0], dg[n][0]); G[n][1] = fmaf(d_lo, G[n][1], dg[n][1]);
                G[n][2] = fmaf(d_hi, G[n][2], dg[n][2]); G[n][3] = fmaf(d_hi, G[n][3], dg[n][3]);
            }
            tc_fence_before();
        }
        // ---- while the second group of products runs: the next chunk's operands and its first group of products
        float a_nxt[2][4], lw_nxt[2][4], d_nxt[2] = {0.f, 0.f};
        int st_nxt = 0;
        if (it + 1 < nchunks) {
            st_nxt = prepare(it + 1, a_nxt, lw_nxt, d_nxt);
            if (st_nxt < 0) { alive = false; break; }
        }
        ok = staging_free() & mbar_wait(bar(BB_MMA2), mph2, abort_flag);     // (made uniform at the barrier of the suffix sums)
        mph2 ^= 1;
        tc_fence_after();
        // ---- epilogue
        {
            float z[2][4], qv[2][4];
            {
                // q and m take the operands as the tensor core saw them (rounded to bf16): the pair terms that q and
                // m share, and that cancel in the suffix sums, are then the same products on both sides
                float acc[2][4], o[2][4], hat[2][4], rv[2][4], kv[2][4];
                const float pd0 = fsm(BO_DPD)[R0], pd1 = fsm(BO_DPD)[R1];
                float acc2[2][4], acc3[2][4];
                tmem_ld_16x16_async(tacc + BT_DR, acc);
                tmem_ld_16x16_async(tacc + BT_DK, acc2);
                tmem_ld_16x16_async(tacc + BT_DV, acc3);
                load_block_bf16(tr + moff, rv);
                load_block_bf16(tk + moff, kv);
                load_block_bf16(t_rh + moff, hat);
                tmem_ld_done();
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float pd = e < 2 ? pd0 : pd1;
                        o[n][e] = fmaf(uu[n][e & 1] * kv[n][e], pd, acc[n][e] * ex2(a_cur[n][e] - lw_cur[n][e]));
                        qv[n][e] = acc[n][e] * hat[n][e];
                        if (!C2) du_acc[n][e & 1] = fmaf(rv[n][e] * kv[n][e], pd, du_acc[n][e & 1]);
                    }
                store_block_bf16(sbase + BO_OUT + moff, o);
                load_block_bf16(t_kh + moff, hat);
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float pd = e < 2 ? pd0 : pd1;
                        o[n][e] = fmaf(uu[n][e & 1] * rv[n][e], pd, acc2[n][e] * ex2(-a_cur[n][e]));
                        z[n][e] = qv[n][e] - acc2[n][e] * hat[n][e];
                        if (C2) {
                            // o is the gradient of k (1 - w): the key gets (1 - w) of it, and the decay logit its
                            // share through the key factor, folded into the term that leaves the suffix sums
                            const float omw = one_minus_ex2(lw_cur[n][e]);
                            qv[n][e] = fmaf(o[n][e] * kv[n][e], 1.f - omw, qv[n][e]);
                            o[n][e] *= omw;
                        }
                    }
                store_block_bf16(sbase + BO_OUT + TILE + moff, o);
                store_block_bf16(sbase + BO_OUT + 2 * TILE + moff, acc3);
            }
            tc_fence_before();
            ok = scan_rows<true>(z, sbase + BO_TOT, sp, cq, lane, ok);
            if (!ok) { alive = false; break; }
            float o[2][4];
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                float E0 = 0.f, E1 = 0.f;
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    E0 += fsm(BO_EP)[(pb * 4 + w) * 64 + cb + 8 * n];
                    E1 += fsm(BO_EP)[(pb * 4 + w) * 64 + cb + 8 * n + 1];
                }
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    o[n][e] = ((e & 1 ? E1 : E0) + z[n][e] - qv[n][e]) * (lw_cur[n][e] * LN2);
            }
            store_block_bf16(sbase + BO_OUT + 3 * TILE + moff, o);
        }
        store_and_refill(it);
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) { a_cur[n][e] = a_nxt[n][e]; lw_cur[n][e] = lw_nxt[n][e]; }
        d_cur[0] = d_nxt[0]; d_cur[1] = d_nxt[1];
        st = st_nxt;
    }

    cbar();
    if (alive) {
        if (p.dstate_in) {
            float* dst = p.dstate_in + (size_t)unit * 4096;
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                *reinterpret_cast<float2*>(dst + (size_t)R0 * 64 + cb + 8 * n) = make_float2(G[n][0], G[n][1]);
                *reinterpret_cast<float2*>(dst + (size_t)R1 * 64 + cb + 8 * n) = make_float2(G[n][2], G[n][3]);
            }
        }
        // the bonus gradient of this unit: over the lanes' rows, then over the four row groups, in a fixed order
#pragma unroll
        for (int d = 4; d < 32; d <<= 1)
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 2; ++e) du_acc[n][e] += __shfl_xor_sync(0xffffffffu, du_acc[n][e], d);
        if (g == 0) {
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 2; ++e) fsm(BO_RED_V)[sp * 64 + cb + 8 * n + e] = du_acc[n][e];
        }
        cbar();
        if (!C2 && tid < 64) {
            const float* rv4 = fsm(BO_RED_V);
            p.du_part[(size_t)unit * 64 + tid] = ((rv4[tid] + rv4[64 + tid]) + (rv4[128 + tid] + rv4[192 + tid])) + fsm(BO_DU_FB)[tid];
        }
    }
    if (tid == 0) post(CMD_QUIT, 0u);
    }   // compute warps
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, BT_COLS);
    }
}

// du[h][i] = sum over the batch of the units' partial sums, in batch order
__global__ void __launch_bounds__(64)
wkv6_backward_chunked_du_kernel(const float* __restrict__ du_part, int B, int H, float* __restrict__ du)
{
    const int h = blockIdx.x, i = threadIdx.x;
    float acc = 0.f;
    for (int b = 0; b < B; ++b) acc += du_part[((size_t)b * H + h) * 64 + i];
    du[h * 64 + i] = acc;
}

}  // namespace bc

}  // namespace gf
