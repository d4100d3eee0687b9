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
// a checkpoint pass of the forward kernel (state only), one 64x64 bf16 block per chunk: the operand tile of dY S_0^T,
// which the kernel fetches by TMA (the state is rounded to bf16 at that use in any case).
//
// Two chunks are in flight per CTA.  A chunk's phases (decay -> cumulative sum -> operands -> products -> masks ->
// products -> epilogue -> suffix sums) depend on one another and each keeps a different pipe busy, so one set of warps
// that walks them in lock step leaves most issue slots empty.  The CTA's 16 warps therefore form two groups of 8 that
// take alternate chunks and run half a period apart: while one group waits for its products or sits in a
// latency-bound phase, the other one issues.  The only thing a chunk needs from the chunk after it (in time) is the
// adjoint at its end, G_L = G_0 of that chunk, and it enters late (the operand G^ = diag(D) G_L and G_0 = G^ + R^^T dY,
// whose product needs no G), so the groups hand G to each other through a pair of fp32 tiles in shared memory, each
// guarded by an mbarrier that all threads of the writing group arrive on; the row sums E travel with it (the group
// that made G_L forms them from its own chunk-start state, which is the next chunk's end state).
//
// Layout inside a group: warp (sp = warp % 4, cx = warp / 4 % 2) owns rows 16 sp .. +15 and columns 32 cx .. +31 of
// every 64x64 tile; lane (g = lane / 4, q = lane % 4) rows 16 sp + g and + 8, columns 32 cx + 8 n + 2 q + e (n < 4,
// e < 2): 16 cells, the accumulator layout of the 64-row products, in which bf16 tiles move through ldmatrix /
// stmatrix, so nothing is transposed and a lane's cells are the same in every phase.  (G_NB = 2 gives groups of 16
// warps with 8 cells per lane at 64 registers instead: measured slower, the spills cost more than the warps bring.)
// Each group has its own input stage (x, v, dy and r, k by TMA, each part re-filled as soon as its tiles fall free),
// operand tiles, tensor-memory columns (three accumulators that the second group of products reuses once the first
// group's have been read) and barriers; the four staging tiles of the gradients lie over operand tiles that are dead
// by the time they are written.  One lane of a group issues its copies, two others (in other warps) its two groups of
// products, so that no warp carries all the issuing.  Sums along the tokens (the
// cumulative decay; the suffix sums of the decay gradient) run over lanes by shuffles and across the four row groups
// through shared memory.  Waits are per thread and bounded; their outcome is made uniform over the group at its next
// barrier, and the hand-over waits watch the CTA's abort word, so after a wait that ran out both groups leave.
// A chunk in which a channel decays by more than 2^-96 runs token by token in fp32 on its group's warps (its 64
// states recomputed into a scratch slot of the workspace), so any decay logit gives the gradient of the exact
// recurrence.
#pragma once
#include "wkv6_chunked.cuh"

namespace gf {
namespace bc {

using namespace ck;          // PTX wrappers, descriptors, layout helpers of the forward kernel

constexpr float LN2 = 0.6931471805599453f;
constexpr size_t FB_SLOT_FLOATS = (size_t)64 * 4096;      // scratch of the token-by-token path per SM and group: 64 states

struct BParams {
    const float* u;              // [H][64]
    const float* dstate_out;     // [units][64][64] or NULL (zero)
    float* dstate_in;            // [units][64][64] or NULL (not written)
    const __nv_bfloat16* ckpt;   // [units][chunks + 1][64][64] bf16 (read through the tensor map tm_ck and, rarely, directly)
    float* du_part;              // [units][64]
    float* fb_scratch;           // [n_slots][64][4096]
    __nv_bfloat16 *dr, *dk, *dv, *dx;
    int T, H, n_slots;
    uint32_t wait_limit_us;
    // Sequence split (calls with few units): every sequence is cut into nseg segments of seg_chunks chunks (the last
    // takes the rest) and the grid is units x nseg.  The state adjoint at a segment's end follows from dstate_out and the
    // summaries of the segments after it, G <- diag(D_s) G + dG_s for s = nseg-1 down to seg+1, which a first launch
    // (the kernel's summary variant, grid units x (nseg-1)) leaves in gsum: [unit][s-1][64 + 64*64] fp32.  nseg = 1: no
    // split.  du_part is [unit][seg][64].
    const float* gsum;
    float* gsum_out;             // summary variant: where the summaries go (same layout)
    int nseg, seg_chunks;
};
// What the packed variants take on top (the dense variants keep the plain parameter block).
struct BParamsPacked : BParams {
    // Packed sequences (split by the longest one: segments past a sequence's end are empty): rows cu[s] .. cu[s+1]-1 of the [rows][H*64] tensors form sequence s, T is unused,
    // and the checkpoints are [H][ckpt_slots][64][64] with sequence s of head h from slot cu[s] / 64 + 2 s on.
    const int32_t* cu;
    long long ckpt_slots;
    // The sequence indices by decreasing length (the grid's first CTAs take the longest sequences, so that the launch
    // does not end on a long one while the other SMs idle); NULL: in index order.
    const int32_t* order;
};
template <bool PACKED> struct BParamsOf { using type = BParams; };
template <> struct BParamsOf<true> { using type = BParamsPacked; };
constexpr int GSUM_FLOATS = 64 + 64 * 64;
constexpr size_t CKPT_FLOATS = 64 * 64 / 2;               // a checkpoint (one bf16 [64][64] state) in units of the workspace's floats

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

// 1 - 2^l for l <= 0 without the cancellation of the direct form near l = 0 (slow decays): the series of -expm1 there.
__device__ __forceinline__ float one_minus_ex2(float l)
{
    const float t = l * LN2;
    const float series = -t * (1.f + t * (0.5f + t * (0.16666667f + t * 0.041666668f)));
    return l > -0.125f ? series : 1.f - ex2(l);
}

__device__ __forceinline__ void tmem_ld_done() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// NB = 8-column blocks per lane: 4 (groups of 8 warps, 16 cells per lane, 128 registers) or 2 (groups of 16 warps,
// 8 cells per lane, 64 registers)
constexpr int G_NB = 4;
constexpr int G_NSLAB = 8 / G_NB;                 // column slabs of 8 NB columns per tile = warps per row group
constexpr int G_H2 = G_NB / 2;                    // 16-column blocks per lane
constexpr int G_GT = 32 * 4 * G_NSLAB;            // threads of one group
constexpr int G_THREADS = 2 * G_GT;               // the CTA
// tensor memory: per group 256 columns, three accumulators used twice
constexpr int GT_P = 0, GT_DP = 64, GT_DG = 128, GT_DV = 0, GT_DR = 64, GT_DK = 128, GT_COLS = 512;
// shared memory of one group
constexpr int GO_IN = 0;                          // x, r, k, v, dy
constexpr int GO_RH = GO_IN + 5 * TILE;           // R^ [t][c]
constexpr int GO_KH = GO_RH + TILE;               // K^ [i][c]
constexpr int GO_T4 = GO_KH + TILE;               // S_0, G^, P', dP' operand tiles; later the dr, dk, dv, dx staging tiles
constexpr int GO_TOT = GO_T4 + 4 * TILE;          // [4][64] float: row-group totals of a scan
constexpr int GO_EP = GO_TOT + 1024;              // [NSLAB][64] float: partial E by column slab
constexpr int GO_BP = GO_EP + 1024;               // [NSLAB][64] float: partial bonus by column slab
constexpr int GO_DPD = GO_BP + 1024;              // [64] float: dy_t . v_t
constexpr int GO_RED = GO_DPD + 256;              // token-by-token path: [NSLAB][3][64]
constexpr int GO_REDV = GO_RED + 4 * 3 * 64 * 4;  //   [4][64]
constexpr int GO_DUFB = GO_REDV + 1024;           //   du [64]
constexpr int GO_SCAL = GO_DUFB + 256;            //   v . dy, sum r u k
constexpr int GO_BYTES = (GO_SCAL + 16 + 1023) & ~1023;
// shared by the groups
constexpr int GS_GBUF = 2 * GO_BYTES;             // [2][64][64] float: the adjoint handed from chunk to chunk
constexpr int GS_EH = GS_GBUF + 2 * 16384;        // [2][NSLAB][64] float: partial E = rowsum(G * S) handed on with G
constexpr int GS_U = GS_EH + 2 * G_NSLAB * 256;   // [64] float: the bonus
constexpr int GS_ABORT = GS_U + 256;              // abort word, wait limit
constexpr int GS_TMEM = GS_ABORT + 8;
// mbarriers, per group: inputs x, v, dy / inputs r, k / first group of products / dR^ and dK^ / dV; then the hand-over pair
constexpr int GS_BAR = GS_TMEM + 8;
enum { GB_INA = 0, GB_INB = 1, GB_MA = 2, GB_MRK = 3, GB_MV = 4, GB_S0 = 5, GB_PER_GROUP = 6, GB_GREADY = 12, GB_COUNT = 14 };
constexpr int G_SMEM_BYTES = GS_BAR + 8 * GB_COUNT;
constexpr int G_SMEM_ALLOC = G_SMEM_BYTES + 1024;
static_assert(G_SMEM_ALLOC <= 232448, "shared memory budget of one sm_100 CTA");

// barrier over one group's 8 warps (ids 1 and 2), plain and with an AND over a predicate
__device__ __forceinline__ void gbar(int grp) { asm volatile("bar.sync %0, %1;" ::"r"(grp + 1), "n"(G_GT) : "memory"); }
__device__ __forceinline__ bool gbar_and(int grp, bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "bar.red.and.pred q, %1, %3, p;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r) : "r"(grp + 1), "r"((uint32_t)ok), "n"(G_GT) : "memory");
    return r != 0;
}

// explicit shared-space accesses (a pointer rebuilt from an integer would make them generic loads)
__device__ __forceinline__ float2 ldsf2(uint32_t a)
{
    float2 v;
    asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void stsf2(uint32_t a, float2 v) { asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(a), "f"(v.x), "f"(v.y) : "memory"); }

// 16 rows x 16 columns of an accumulator, without the wait (tmem_ld_done() before the first use)
__device__ __forceinline__ void tmem_ld_16x16_async2(uint32_t taddr, float (&v)[2][4])
{
    asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(v[0][0]), "=f"(v[0][1]), "=f"(v[0][2]), "=f"(v[0][3]), "=f"(v[1][0]), "=f"(v[1][1]), "=f"(v[1][2]), "=f"(v[1][3])
                 : "r"(taddr) : "memory");
}

// 16 x 16 bf16 blocks of a swizzled tile <-> two column blocks (n = 2 h2, 2 h2 + 1) of the lane's cells
__device__ __forceinline__ void ld_half(uint32_t addr, float (&v)[2][4])
{
    uint32_t w0, w1, w2, w3;
    ldsm_x4(addr, w0, w1, w2, w3);
    v[0][0] = bf_lo(w0); v[0][1] = bf_hi(w0); v[0][2] = bf_lo(w1); v[0][3] = bf_hi(w1);
    v[1][0] = bf_lo(w2); v[1][1] = bf_hi(w2); v[1][2] = bf_lo(w3); v[1][3] = bf_hi(w3);
}
__device__ __forceinline__ void st_half(uint32_t addr, const float (&v)[2][4])
{
    stsm_x4(addr, pack_bf16(v[0][0], v[0][1]), pack_bf16(v[0][2], v[0][3]), pack_bf16(v[1][0], v[1][1]), pack_bf16(v[1][2], v[1][3]));
}
__device__ __forceinline__ void ld_tile(uint32_t tile, const uint32_t (&moff)[G_H2], float (&v)[G_NB][4])
{
#pragma unroll
    for (int h2 = 0; h2 < G_H2; ++h2) ld_half(tile + moff[h2], reinterpret_cast<float (&)[2][4]>(v[2 * h2]));
}
__device__ __forceinline__ void st_tile(uint32_t tile, const uint32_t (&moff)[G_H2], const float (&v)[G_NB][4])
{
#pragma unroll
    for (int h2 = 0; h2 < G_H2; ++h2) st_half(tile + moff[h2], reinterpret_cast<const float (&)[2][4]>(v[2 * h2]));
}

// Inclusive sums along the 64 rows of a tile in the group's layout, forwards (rows <= t) or backwards (rows >= t).
// tot: [4][64] floats of the group's shared memory.  Contains one barrier of the group, which also forms the AND of
// `ok` over it (returned).
template <bool REV>
__device__ __forceinline__ bool scan_rows(float (&v)[G_NB][4], uint32_t tot, int grp, int sp, int cb, int lane, bool ok)
{
    const int g = lane >> 2, q = lane & 3;           // (cb: the lane's first column, a multiple of 2)
    // (the additions run on the pairs of neighbouring columns: one two-lane instruction for two cells)
#pragma unroll
    for (int d = 4; d < 32; d <<= 1) {
        const bool take = REV ? lane + d < 32 : lane >= d;
#pragma unroll
        for (int n = 0; n < G_NB; ++n)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float2 o;
                o.x = REV ? __shfl_down_sync(0xffffffffu, v[n][2 * h], d) : __shfl_up_sync(0xffffffffu, v[n][2 * h], d);
                o.y = REV ? __shfl_down_sync(0xffffffffu, v[n][2 * h + 1], d) : __shfl_up_sync(0xffffffffu, v[n][2 * h + 1], d);
                if (take) {
                    const float2 r = add2(make_float2(v[n][2 * h], v[n][2 * h + 1]), o);
                    v[n][2 * h] = r.x; v[n][2 * h + 1] = r.y;
                }
            }
    }
#pragma unroll
    for (int n = 0; n < G_NB; ++n) {
        float2 o;
        if (REV) {
            o.x = __shfl_sync(0xffffffffu, v[n][2], q); o.y = __shfl_sync(0xffffffffu, v[n][3], q);
            const float2 r = add2(make_float2(v[n][0], v[n][1]), o);
            v[n][0] = r.x; v[n][1] = r.y;
        } else {
            o.x = __shfl_sync(0xffffffffu, v[n][0], 28 + q); o.y = __shfl_sync(0xffffffffu, v[n][1], 28 + q);
            const float2 r = add2(make_float2(v[n][2], v[n][3]), o);
            v[n][2] = r.x; v[n][3] = r.y;
        }
    }
    if (g == (REV ? 0 : 7)) {
#pragma unroll
        for (int n = 0; n < G_NB; ++n)
            stsf2(tot + 4 * (sp * 64 + cb + 8 * n), REV ? make_float2(v[n][0], v[n][1]) : make_float2(v[n][2], v[n][3]));
    }
    ok = gbar_and(grp, ok);
    // the totals of the row groups before (after) this one: summed first, then added to both rows
    float2 t[G_NB];
#pragma unroll
    for (int n = 0; n < G_NB; ++n) t[n] = make_float2(0.f, 0.f);
    bool any = false;
#pragma unroll
    for (int o = 0; o < 4; ++o) {
        if (REV ? o > sp : o < sp) {
#pragma unroll
            for (int n = 0; n < G_NB; ++n) t[n] = add2(t[n], ldsf2(tot + 4 * (o * 64 + cb + 8 * n)));
            any = true;
        }
    }
    if (any) {
#pragma unroll
        for (int n = 0; n < G_NB; ++n) {
            const float2 lo = add2(make_float2(v[n][0], v[n][1]), t[n]), hi = add2(make_float2(v[n][2], v[n][3]), t[n]);
            v[n][0] = lo.x; v[n][1] = lo.y; v[n][2] = hi.x; v[n][3] = hi.y;
        }
    }
    return ok;
}

// GSUM = true: the summary variant of a split call (see BParams::gsum): only the adjoint's own recurrence
// G <- diag(D) G + R^^T dY over a segment, from zero, and the product of the chunk decays; it reads x, r, dy only and
// needs no token-by-token path (R^ never exceeds r: no exponent can overflow).
// PACKED: packed variable-length sequences (BParams::cu), one CTA per sequence and head.
template <bool C2, bool GSUM = false, bool PACKED = false>
__global__ void __launch_bounds__(G_THREADS, 1)
wkv6_backward_chunked_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_r,
                            const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                            const __grid_constant__ CUtensorMap tm_dy, const __grid_constant__ CUtensorMap tm_dr,
                            const __grid_constant__ CUtensorMap tm_dk, const __grid_constant__ CUtensorMap tm_dv,
                            const __grid_constant__ CUtensorMap tm_dx, const __grid_constant__ CUtensorMap tm_ck,
                            const typename BParamsOf<PACKED>::type p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t abort_flag = sbase + GS_ABORT;
    auto bar = [&](int i) { return sbase + GS_BAR + 8 * i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = tid / G_GT, gt = tid % G_GT;                    // group, thread inside the group
    const int sp = warp & 3, cx = (warp >> 2) % G_NSLAB, g = lane >> 2, q = lane & 3;       // row group, column slab
    // summary variant: segments 1 .. nseg-1 of every unit; else every segment
    const int gsegs = GSUM ? p.nseg - 1 : p.nseg;
    const int slot = blockIdx.x / gsegs, seg = blockIdx.x % gsegs + (GSUM ? 1 : 0);
    int unit = slot, seq = unit / p.H;
    const int h = unit % p.H;
    int T = p.T;
    long long row0 = (long long)seq * T;
    size_t ck_first = 0;                             // the unit's first checkpoint slot (packed)
    if constexpr (PACKED) {
        if (p.order) { seq = p.order[seq]; unit = seq * p.H + h; }
        row0 = p.cu[seq];
        T = p.cu[seq + 1] - p.cu[seq];
        ck_first = (size_t)h * p.ckpt_slots + (size_t)(p.cu[seq] >> 6) + 2 * (size_t)seq;
    }
    const int nchunks = (T + L - 1) / L;
    const int c_lo = p.nseg > 1 ? min(nchunks, seg * p.seg_chunks) : 0;                      // this CTA's chunks: c_lo .. c_hi-1,
    const int c_hi = (p.nseg > 1 && seg < p.nseg - 1) ? min(nchunks, c_lo + p.seg_chunks) : nchunks;   // walked from the last
    const int nit = c_hi - c_lo;
    const int col0 = h * 64;
    const size_t C = (size_t)p.H * 64;
    const int R0 = 16 * sp + g, R1 = R0 + 8;         // this lane's two rows
    const int cb = 8 * G_NB * cx + 2 * q;            // its columns: cb + 8 n + e, n < G_NB
    // byte offsets of this lane's ldmatrix / stmatrix rows inside a tile: the warp's 16 x 16 blocks
    uint32_t moff[G_H2];
#pragma unroll
    for (int h2 = 0; h2 < G_H2; ++h2)
        moff[h2] = swz(16 * sp + (lane & 7) + 8 * ((lane >> 3) & 1), (G_NB * cx + 2 * h2 + (lane >> 4)) << 4);
    const uint32_t gbase = sbase + grp * GO_BYTES;   // this group's shared memory
    auto gsm = [&](int off) { return reinterpret_cast<float*>(smem + grp * GO_BYTES + off); };
    // the adjoint tiles handed between the groups: [buffer][cell of the lane][thread of the group] (conflict-free)
    auto g_put = [&](int b, const float (&v)[G_NB][4]) {
#pragma unroll
        for (int n = 0; n < G_NB; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) stsf(sbase + GS_GBUF + 4 * ((b * 4 * G_NB + 4 * n + e) * G_GT + gt), v[n][e]);
    };
    auto g_get = [&](int b, float (&v)[G_NB][4]) {
#pragma unroll
        for (int n = 0; n < G_NB; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) v[n][e] = ldsf(sbase + GS_GBUF + 4 * ((b * 4 * G_NB + 4 * n + e) * G_GT + gt));
    };
    auto gld = [&](int off) { return ldsf(gbase + off); };           // a float of this group's small arrays
    const float* ub = reinterpret_cast<const float*>(smem + GS_U);
    auto gb = [&](int i) { return bar(grp * GB_PER_GROUP + i); };      // this group's barriers

    if (tid == 0) {
        for (int i = 0; i < GB_GREADY; ++i) mbar_init(bar(i), 1);
        mbar_init(bar(GB_GREADY), G_GT);
        mbar_init(bar(GB_GREADY + 1), G_GT);
        sts32(abort_flag, 0u);
        sts32(abort_flag + 4, p.wait_limit_us ? p.wait_limit_us : WAIT_LIMIT_US);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (tid < 64) reinterpret_cast<float*>(smem + GS_U)[tid] = (C2 || GSUM) ? 0.f : p.u[col0 + tid];
    if (gt < 64) gsm(GO_DUFB)[gt] = 0.f;
    if (warp == 1) tmem_alloc(sbase + GS_TMEM, GT_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32(sbase + GS_TMEM) + 256 * grp;                 // this group's columns
    const uint32_t tacc = tmem + ((uint32_t)(32 * sp) << 16) + 8 * G_NB * cx;      // this warp's block of an accumulator

    auto chunk_of = [&](int it) { return c_hi - 1 - it; };
    const uint32_t tin = gbase + GO_IN;
    const uint32_t tx = tin, tr = tin + TILE, tk = tin + 2 * TILE, tv = tin + 3 * TILE, tdy = tin + 4 * TILE;
    const uint32_t t_rh = gbase + GO_RH, t_kh = gbase + GO_KH;
    const uint32_t t_sb = gbase + GO_T4, t_gb = t_sb + TILE, t_pp = t_sb + 2 * TILE, t_dpp = t_sb + 3 * TILE;
    // staging tiles of the four gradients, each over an operand tile that is dead when it is written: dr over S_0 and
    // dk over dP' (free once dR^ and dK^ are complete), dv over P' and dx over G^ (free once dV is complete)
    const uint32_t o_dr = t_sb, o_dk = t_dpp, o_dv = t_pp, o_dx = t_gb;
    // The input copies of a chunk come in two parts, each issued as soon as its tiles are free: x, v, dy once the
    // chunk before (of this group) has finished its products, r, k once its epilogue has read them.
    int last_a = -1, last_b = -1, last_s = -1;       // (thread 0 of the group) the last iterations whose copies were issued
    auto issue_loads_a = [&](int it) {               // thread 0 of the group
        const int row = (int)(row0 + (long long)chunk_of(it) * L);
        mbar_expect_tx(gb(GB_INA), 3 * TILE);
        tma_load_2d(tx, &tm_x, col0, row, gb(GB_INA));
        tma_load_2d(tv, &tm_v, col0, row, gb(GB_INA));
        tma_load_2d(tdy, &tm_dy, col0, row, gb(GB_INA));
        last_a = it;
    };
    auto issue_loads_b = [&](int it) {
        const int row = (int)(row0 + (long long)chunk_of(it) * L);
        mbar_expect_tx(gb(GB_INB), 2 * TILE);
        tma_load_2d(tr, &tm_r, col0, row, gb(GB_INB));
        tma_load_2d(tk, &tm_k, col0, row, gb(GB_INB));
        last_b = it;
    };
    auto load_f32_block = [&](const float* src, float (&v)[G_NB][4]) {      // [64][64] fp32 block, the lane's cells
#pragma unroll
        for (int n = 0; n < G_NB; ++n) {
            const float2 lo = *reinterpret_cast<const float2*>(src + (size_t)R0 * 64 + cb + 8 * n);
            const float2 hi = *reinterpret_cast<const float2*>(src + (size_t)R1 * 64 + cb + 8 * n);
            v[n][0] = lo.x; v[n][1] = lo.y; v[n][2] = hi.x; v[n][3] = hi.y;
        }
    };
    auto store_f32_block = [&](float* dst, const float (&v)[G_NB][4]) {
#pragma unroll
        for (int n = 0; n < G_NB; ++n) {
            *reinterpret_cast<float2*>(dst + (size_t)R0 * 64 + cb + 8 * n) = make_float2(v[n][0], v[n][1]);
            *reinterpret_cast<float2*>(dst + (size_t)R1 * 64 + cb + 8 * n) = make_float2(v[n][2], v[n][3]);
        }
    };

    const size_t ck_slot0 = PACKED ? ck_first : (size_t)unit * (nchunks + 1);       // this unit's first checkpoint
    const __nv_bfloat16* ck_unit = p.ckpt + ck_slot0 * 4096;
    // the chunk-start state is a bf16 [64][64] tile in memory: it lands in its operand tile by TMA (rows of the
    // checkpoint array seen as [slots * 64][64])
    auto issue_load_s = [&](int it) {                // thread 0 of the group
        mbar_expect_tx(gb(GB_S0), TILE);
        tma_load_2d(t_sb, &tm_ck, 0, (int)((ck_slot0 + (size_t)chunk_of(it)) * 64), gb(GB_S0));
        last_s = it;
    };
    auto load_bf16_block = [&](const __nv_bfloat16* src, float (&v)[G_NB][4]) {     // a checkpoint, the lane's cells
#pragma unroll
        for (int n = 0; n < G_NB; ++n) {
            const float2 lo = bf_pair(*reinterpret_cast<const uint32_t*>(src + (size_t)R0 * 64 + cb + 8 * n));
            const float2 hi = bf_pair(*reinterpret_cast<const uint32_t*>(src + (size_t)R1 * 64 + cb + 8 * n));
            v[n][0] = lo.x; v[n][1] = lo.y; v[n][2] = hi.x; v[n][3] = hi.y;
        }
    };
    float du_acc[G_NB][2];
#pragma unroll
    for (int n = 0; n < G_NB; ++n) du_acc[n][0] = du_acc[n][1] = 0.f;
    if (gt == 0 && grp < nit) { issue_loads_a(grp); issue_loads_b(grp); }
    int mph = 0;                                     // phase bit of this group's two product barriers
    float dprod_lo = 1.f, dprod_hi = 1.f;            // summary variant: product of this group's chunk decays (rows R0, R1)
    bool alive = true;

    for (int it = grp; it < nit; it += 2) {
        const int c = chunk_of(it), valid = min(L, T - c * L);
        const int use = it >> 1;                     // how often this group's input stage has been filled before
        if (it + 2 < nit && gt == 128) {
            // this group's next chunk: its start state and its input tiles into L2 now, so that the copies issued
            // later find them there
            const int row = (int)(row0 + (long long)(c - 2) * L);
            tma_prefetch_2d(&tm_x, col0, row); tma_prefetch_2d(&tm_r, col0, row); tma_prefetch_2d(&tm_k, col0, row);
            tma_prefetch_2d(&tm_v, col0, row); tma_prefetch_2d(&tm_dy, col0, row);
            if (!GSUM) tma_prefetch_2d(&tm_ck, 0, (int)((ck_slot0 + (size_t)(c - 2)) * 64));
        }
        // ---- decay: log2-domain magnitudes, cumulative sums over the tokens
        bool ok = mbar_wait(gb(GB_INA), use & 1, abort_flag);
        if (gt == 0) {
            if (it > 1) bulk_wait_read<0>();         // the previous chunk's staging tiles have been read by the TMA unit
            if (!GSUM) issue_load_s(it);             // (the start state's tile doubles as the staging tile of dr)
        }
        float a[G_NB][4], lw2[G_NB][4];
        {
            float xv[G_NB][4];
            ld_tile(tx, moff, xv);
#pragma unroll
            for (int n = 0; n < G_NB; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool live = (e < 2 ? R0 : R1) < valid;
                    lw2[n][e] = live ? -ex2(fmaf(xv[n][e], LOG2E, LOG2_LOG2E)) : 0.f;
                    a[n][e] = lw2[n][e];
                }
        }
        ok = scan_rows<false>(a, gbase + GO_TOT, grp, sp, cb, lane, ok);      // (barrier: the zeroed rows are visible after it)
        if (!ok) { alive = false; break; }
        float d_lo, d_hi;                            // the chunk's decay for the channels that are this lane's rows of G
        bool safe;
        {
            float al0 = 0.f, al1 = 0.f;
#pragma unroll
            for (int o = 0; o < 4; ++o) { al0 += gld(GO_TOT + 4 * (o * 64 + R0)); al1 += gld(GO_TOT + 4 * (o * 64 + R1)); }
            d_lo = ex2(al0); d_hi = ex2(al1);
            safe = GSUM || ((al0 >= -A2_MAX) && (al1 >= -A2_MAX));         // false for NaN as well
            if (GSUM) { dprod_lo *= d_lo; dprod_hi *= d_hi; }
        }
        // ---- operands from the inputs: R^, K^ (and the bonus), the chunk-start state
        if (!mbar_wait(gb(GB_INB), use & 1, abort_flag)) ok = false;        // (made uniform at a later barrier)
        if (valid < L) {
            // ragged last chunk: the rows past the sequence's end hold other tokens (or the out-of-range fill)
            for (int i = gt; i < (L - valid) * 8; i += G_GT) {
                const uint32_t o = (valid + (i >> 3)) * 128 + ((i & 7) << 4);
                sts128z(tr + o); sts128z(tk + o); sts128z(tv + o); sts128z(tdy + o);
            }
            gbar(grp);
        }
        {
            float rv[G_NB][4], kv[G_NB][4];
            ld_tile(tr, moff, rv);
            ld_tile(tk, moff, kv);
            float b0 = 0.f, b1 = 0.f;
            // (two-lane fp32 arithmetic on the pairs of neighbouring columns: half the multiply / add instructions)
#pragma unroll
            for (int n = 0; n < G_NB; ++n) {
                const float2 u2 = (!C2 && !GSUM) ? ldsf2(sbase + GS_U + 4 * (cb + 8 * n)) : make_float2(0.f, 0.f);
#pragma unroll
                for (int h = 0; h < 2; ++h) {                          // h = 0: row R0, h = 1: row R1
                    float2 rr = make_float2(rv[n][2 * h], rv[n][2 * h + 1]), kk = make_float2(kv[n][2 * h], kv[n][2 * h + 1]);
                    const float2 aa = make_float2(a[n][2 * h], a[n][2 * h + 1]), ll = make_float2(lw2[n][2 * h], lw2[n][2 * h + 1]);
                    if (C2) kk = mul2(kk, make_float2(one_minus_ex2(ll.x), one_minus_ex2(ll.y)));      // the key that enters the state
                    if (!C2 && !GSUM) {
                        const float2 t = mul2(mul2(rr, kk), u2);
                        if (h == 0) b0 += t.x + t.y; else b1 += t.x + t.y;
                    }
                    rr = mul2(rr, ex2_2(sub2(aa, ll)));
                    kk = mul2(kk, make_float2(ex2(-aa.x), ex2(-aa.y)));
                    rv[n][2 * h] = rr.x; rv[n][2 * h + 1] = rr.y; kv[n][2 * h] = kk.x; kv[n][2 * h + 1] = kk.y;
                }
            }
            st_tile(t_rh, moff, rv);
            if (!GSUM) st_tile(t_kh, moff, kv);
            if (!C2 && !GSUM) {
                b0 += __shfl_xor_sync(0xffffffffu, b0, 1); b1 += __shfl_xor_sync(0xffffffffu, b1, 1);
                b0 += __shfl_xor_sync(0xffffffffu, b0, 2); b1 += __shfl_xor_sync(0xffffffffu, b1, 2);
                if (q == 0) { stsf(gbase + GO_BP + 4 * (cx * 64 + R0), b0); stsf(gbase + GO_BP + 4 * (cx * 64 + R1), b1); }
            }
        }
        if (!GSUM && !mbar_wait(gb(GB_S0), use & 1, abort_flag)) ok = false;       // the chunk-start state is in its tile
        fence_proxy_async();
        tc_fence_before();
        const bool unsafe = !gbar_and(grp, safe);    // (every channel is some lane's row)
        if (!unsafe && gt == 64) {
            // the products that need nothing but the inputs; the adjoint is not needed for R^^T dY either
            tc_fence_after();
            const uint64_t dR = smem_desc(t_rh), dK = smem_desc(t_kh), dV = smem_desc(tv), dY = smem_desc(tdy);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const uint64_t ks = 2 * kk, ms = 128 * kk;       // K-major / MN-major step of 16 contraction indices
                tc_mma(tmem + GT_DG, dR + ms, dY + ms, IDESC_MN_MN, kk > 0);       // dG[c][j] = R^^T dY
                if (GSUM) continue;
                tc_mma(tmem + GT_P, dR + ks, dK + ks, IDESC_K_K, kk > 0);          // P[t][i]  = R^ K^^T
                tc_mma(tmem + GT_DP, dY + ks, dV + ks, IDESC_K_K, kk > 0);         // dP[t][i] = dY V^T
            }
            tc_commit(gb(GB_MA));
        }
        // ---- the adjoint at the chunk's end, from the other group (the call's dstate_out for the last chunk)
        float G[G_NB][4];
        if (it == 0) {
            if (!GSUM && p.dstate_out) load_f32_block(p.dstate_out + (size_t)unit * 4096, G);
            else {
#pragma unroll
                for (int n = 0; n < G_NB; ++n) G[n][0] = G[n][1] = G[n][2] = G[n][3] = 0.f;
            }
            if (!GSUM) {
                // a segment but the last: the adjoint at its end through the segments after it, from the last down
                for (int sg = p.nseg - 1; sg > seg; --sg) {
                    const float* sm = p.gsum + ((size_t)unit * (p.nseg - 1) + (sg - 1)) * GSUM_FLOATS;
                    const float dl = sm[R0], dh = sm[R1];
                    float dG[G_NB][4];
                    load_f32_block(sm + 64, dG);
#pragma unroll
                    for (int n = 0; n < G_NB; ++n) {
                        G[n][0] = fmaf(dl, G[n][0], dG[n][0]); G[n][1] = fmaf(dl, G[n][1], dG[n][1]);
                        G[n][2] = fmaf(dh, G[n][2], dG[n][2]); G[n][3] = fmaf(dh, G[n][3], dG[n][3]);
                    }
                }
            }
        } else {
            if (!mbar_wait(bar(GB_GREADY + ((it - 1) & 1)), ((it - 1) >> 1) & 1, abort_flag)) ok = false;
            g_get((it - 1) & 1, G);
        }
        // E = rowsum(G_L * S_L), S_L the state at the chunk's end, as partial sums per column slab: for the call's last
        // chunk from the final state; else the group that made G_L formed them from its chunk-start state (e_put below)
        auto e_put = [&](uint32_t dst, const float (&Gm)[G_NB][4], const float (&Sm)[G_NB][4]) {
            float e0 = 0.f, e1 = 0.f;
#pragma unroll
            for (int n = 0; n < G_NB; ++n) {
                e0 = fmaf(Gm[n][0], Sm[n][0], fmaf(Gm[n][1], Sm[n][1], e0));
                e1 = fmaf(Gm[n][2], Sm[n][2], fmaf(Gm[n][3], Sm[n][3], e1));
            }
            e0 += __shfl_xor_sync(0xffffffffu, e0, 1); e1 += __shfl_xor_sync(0xffffffffu, e1, 1);
            e0 += __shfl_xor_sync(0xffffffffu, e0, 2); e1 += __shfl_xor_sync(0xffffffffu, e1, 2);
            if (q == 0) { stsf(dst + 4 * (cx * 64 + R0), e0); stsf(dst + 4 * (cx * 64 + R1), e1); }
        };
        if (GSUM) {
        } else if (it == 0) {
            float SL[G_NB][4];
            load_bf16_block(ck_unit + (size_t)(c + 1) * 4096, SL);
            e_put(gbase + GO_EP, G, SL);
        } else if (gt < G_NSLAB * 64) {
            stsf(gbase + GO_EP + 4 * gt, ldsf(sbase + GS_EH + 4 * (((it - 1) & 1) * G_NSLAB * 64 + gt)));      // (a private copy: the slot is rewritten two chunks on)
        }

        if (unsafe) {
            // ---- token by token: the chunk's states recomputed into this group's scratch, then the reverse recurrence
            const unsigned slot = 2 * smid() + grp;
            if (slot >= (unsigned)p.n_slots) {       // (no scratch for this SM: report it and leave)
                if (gt == 0) { sts32(abort_flag, 1u); atomicExch(&g_dev_status, 1); }
                alive = false;
                break;
            }
            if (!gbar_and(grp, ok)) { alive = false; break; }
            float* scr = p.fb_scratch + (size_t)slot * FB_SLOT_FLOATS + (size_t)gt * (4 * G_NB);
            float S[G_NB][4];
            load_bf16_block(ck_unit + (size_t)c * 4096, S);
            for (int t = 0; t < valid; ++t) {
#pragma unroll
                for (int n = 0; n < G_NB; ++n)
                    *reinterpret_cast<float4*>(scr + (size_t)t * 4096 + 4 * n) = make_float4(S[n][0], S[n][1], S[n][2], S[n][3]);
                const float e0 = expf(lds_bf16(tx + swz(t, 2 * R0))), e1 = expf(lds_bf16(tx + swz(t, 2 * R1)));
                const float w0 = expf(-e0), w1 = expf(-e1);
                float k0 = lds_bf16(tk + swz(t, 2 * R0)), k1 = lds_bf16(tk + swz(t, 2 * R1));
                if (C2) { k0 *= -expm1f(-e0); k1 *= -expm1f(-e1); }
#pragma unroll
                for (int n = 0; n < G_NB; ++n)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float vj = lds_bf16(tv + swz(t, 2 * (cb + 8 * n + e)));
                        S[n][e] = fmaf(w0, S[n][e], k0 * vj);
                        S[n][2 + e] = fmaf(w1, S[n][2 + e], k1 * vj);
                    }
            }
            float* red = gsm(GO_RED);                // [slab][3][64]
            float* redv = gsm(GO_REDV);              // [sp][64]
            float* scal = gsm(GO_SCAL);              // v . dy, sum r u k
            for (int t = valid - 1; t >= 0; --t) {
                float Sp[G_NB][4];
#pragma unroll
                for (int n = 0; n < G_NB; ++n) {
                    const float4 s4 = *reinterpret_cast<const float4*>(scr + (size_t)t * 4096 + 4 * n);
                    Sp[n][0] = s4.x; Sp[n][1] = s4.y; Sp[n][2] = s4.z; Sp[n][3] = s4.w;
                }
                const float x0 = lds_bf16(tx + swz(t, 2 * R0)), x1 = lds_bf16(tx + swz(t, 2 * R1));
                const float w0 = expf(-expf(x0)), w1 = expf(-expf(x1));
                float k0 = lds_bf16(tk + swz(t, 2 * R0)), k1 = lds_bf16(tk + swz(t, 2 * R1));
                if (C2) { k0 *= -expm1f(-expf(x0)); k1 *= -expm1f(-expf(x1)); }
                const float r0 = lds_bf16(tr + swz(t, 2 * R0)), r1 = lds_bf16(tr + swz(t, 2 * R1));
                float pr0 = 0.f, pr1 = 0.f, pk0 = 0.f, pk1 = 0.f, pg0 = 0.f, pg1 = 0.f, pv[G_NB][2];
#pragma unroll
                for (int n = 0; n < G_NB; ++n)
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
                    for (int n = 0; n < G_NB; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) pv[n][e] += __shfl_xor_sync(0xffffffffu, pv[n][e], d);
                if (q == 0) {
                    red[(cx * 3 + 0) * 64 + R0] = pr0; red[(cx * 3 + 0) * 64 + R1] = pr1;
                    red[(cx * 3 + 1) * 64 + R0] = pk0; red[(cx * 3 + 1) * 64 + R1] = pk1;
                    red[(cx * 3 + 2) * 64 + R0] = pg0; red[(cx * 3 + 2) * 64 + R1] = pg1;
                }
                if (g == 0) {
#pragma unroll
                    for (int n = 0; n < G_NB; ++n)
#pragma unroll
                        for (int e = 0; e < 2; ++e) redv[sp * 64 + cb + 8 * n + e] = pv[n][e];
                }
                if (gt < 32) {
                    float vd = 0.f, ruk = 0.f;
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int cc = 2 * lane + e;
                        vd = fmaf(lds_bf16(tv + swz(t, 2 * cc)), lds_bf16(tdy + swz(t, 2 * cc)), vd);
                        if (!C2) ruk = fmaf(lds_bf16(tr + swz(t, 2 * cc)) * ub[cc], lds_bf16(tk + swz(t, 2 * cc)), ruk);
                    }
#pragma unroll
                    for (int d = 1; d < 32; d <<= 1) {
                        vd += __shfl_xor_sync(0xffffffffu, vd, d);
                        ruk += __shfl_xor_sync(0xffffffffu, ruk, d);
                    }
                    if (lane == 0) { scal[0] = vd; scal[1] = ruk; }
                }
                gbar(grp);
                if (gt < 64) {
                    const int cc = gt;
                    float s_r = 0.f, s_k = 0.f, s_g = 0.f;
#pragma unroll
                    for (int o = 0; o < G_NSLAB; ++o) { s_r += red[(o * 3 + 0) * 64 + cc]; s_k += red[(o * 3 + 1) * 64 + cc]; s_g += red[(o * 3 + 2) * 64 + cc]; }
                    const float xc = lds_bf16(tx + swz(t, 2 * cc)), kc = lds_bf16(tk + swz(t, 2 * cc)), rc = lds_bf16(tr + swz(t, 2 * cc));
                    const float ec = expf(xc), wc = expf(-ec);
                    if (C2) {
                        sts_bf16(o_dr + swz(t, 2 * cc), s_r);
                        sts_bf16(o_dk + swz(t, 2 * cc), s_k * -expm1f(-ec));
                        sts_bf16(o_dx + swz(t, 2 * cc), (s_g - s_k * kc) * (-wc * ec));
                    } else {
                        const float uc = ub[cc], vd = scal[0];
                        sts_bf16(o_dr + swz(t, 2 * cc), fmaf(uc * kc, vd, s_r));
                        sts_bf16(o_dk + swz(t, 2 * cc), fmaf(rc * uc, vd, s_k));
                        sts_bf16(o_dx + swz(t, 2 * cc), s_g * (-wc * ec));
                        gsm(GO_DUFB)[cc] = fmaf(rc * kc, vd, gsm(GO_DUFB)[cc]);
                    }
                } else if (gt < 128) {
                    const int j = gt - 64;
                    const float s_v = redv[j] + redv[64 + j] + redv[128 + j] + redv[192 + j];
                    sts_bf16(o_dv + swz(t, 2 * j), fmaf(scal[1], lds_bf16(tdy + swz(t, 2 * j)), s_v));
                }
                gbar(grp);
            }
            // hand the adjoint on (and the row sums the next chunk needs, from the fp32 state: the operand tile is gone)
            if (it + 1 < nit) {
                g_put(it & 1, G);
                load_bf16_block(ck_unit + (size_t)c * 4096, S);
                e_put(sbase + GS_EH + 4 * ((it & 1) * G_NSLAB * 64), G, S);
                mbar_arrive(bar(GB_GREADY + (it & 1)));
            } else if (p.dstate_in && seg == 0) {
                store_f32_block(p.dstate_in + (size_t)unit * 4096, G);
            }
        } else {
            // ---- G^ as an operand; G_0 = G^ + R^^T dY handed on
            if (!GSUM) {
                float gh[G_NB][4];
#pragma unroll
                for (int n = 0; n < G_NB; ++n) {
                    const float2 lo = mul2(make_float2(d_lo, d_lo), make_float2(G[n][0], G[n][1]));
                    const float2 hi = mul2(make_float2(d_hi, d_hi), make_float2(G[n][2], G[n][3]));
                    gh[n][0] = lo.x; gh[n][1] = lo.y; gh[n][2] = hi.x; gh[n][3] = hi.y;
                }
                st_tile(t_gb, moff, gh);
            }
            if (!mbar_wait(gb(GB_MA), mph, abort_flag)) ok = false;
            tc_fence_after();
            {
                float dg[G_NB][4];
#pragma unroll
                for (int h2 = 0; h2 < G_H2; ++h2) tmem_ld_16x16_async2(tacc + GT_DG + 16 * h2, reinterpret_cast<float (&)[2][4]>(dg[2 * h2]));
                tmem_ld_done();
#pragma unroll
                for (int n = 0; n < G_NB; ++n) {
                    const float2 lo = fma2(make_float2(d_lo, d_lo), make_float2(G[n][0], G[n][1]), make_float2(dg[n][0], dg[n][1]));
                    const float2 hi = fma2(make_float2(d_hi, d_hi), make_float2(G[n][2], G[n][3]), make_float2(dg[n][2], dg[n][3]));
                    G[n][0] = lo.x; G[n][1] = lo.y; G[n][2] = hi.x; G[n][3] = hi.y;
                }
            }
            if (it + 1 < nit) {
                g_put(it & 1, G);
                if (!GSUM) {
                    float sb[G_NB][4];               // this chunk's start state is the next chunk's end state (bf16 copy: the operand tile)
                    ld_tile(t_sb, moff, sb);
                    e_put(sbase + GS_EH + 4 * ((it & 1) * G_NSLAB * 64), G, sb);
                }
                mbar_arrive(bar(GB_GREADY + (it & 1)));
            } else if (GSUM) {
                store_f32_block(p.gsum_out + ((size_t)unit * (p.nseg - 1) + (seg - 1)) * GSUM_FLOATS + 64, G);      // the segment's dG
            } else if (p.dstate_in && seg == 0) {
                store_f32_block(p.dstate_in + (size_t)unit * 4096, G);
            }
            if (GSUM) {
                // nothing else in the summary variant: once every lane is done with the tiles, the next chunk's copies
                mph ^= 1;
                tc_fence_before();
                if (!gbar_and(grp, ok)) { alive = false; break; }
                if (gt == 0 && it + 2 < nit) { issue_loads_a(it + 2); issue_loads_b(it + 2); }
                continue;
            }
            // ---- masked scores and their adjoint as operands
#pragma unroll
            for (int h2 = 0; h2 < G_H2; ++h2) {
                const int blk = G_H2 * cx + h2;          // 16-column block of the tile; the diagonal one is blk == sp
                if (blk < sp) {
                    float pp[2][4], dp[2][4];
                    tmem_ld_16x16_async2(tacc + GT_P + 16 * h2, pp);
                    tmem_ld_16x16_async2(tacc + GT_DP + 16 * h2, dp);
                    tmem_ld_done();
                    st_half(t_pp + moff[h2], pp);
                    st_half(t_dpp + moff[h2], dp);
                } else if (blk > sp) {
                    stsm_x4(t_pp + moff[h2], 0u, 0u, 0u, 0u);
                    stsm_x4(t_dpp + moff[h2], 0u, 0u, 0u, 0u);
                } else {
                    float pp[2][4], dp[2][4];
                    tmem_ld_16x16_async2(tacc + GT_P + 16 * h2, pp);
                    tmem_ld_16x16_async2(tacc + GT_DP + 16 * h2, dp);
                    float bon0 = 0.f, bon1 = 0.f;
                    if (!C2) {
#pragma unroll
                        for (int o = 0; o < G_NSLAB; ++o) { bon0 += gld(GO_BP + 4 * (o * 64 + R0)); bon1 += gld(GO_BP + 4 * (o * 64 + R1)); }
                    }
                    tmem_ld_done();
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int row = e < 2 ? g : g + 8, col = 2 * q + 8 * n + (e & 1);       // inside the 16 x 16 block
                            if (col == row) stsf(gbase + GO_DPD + 4 * (16 * sp + row), dp[n][e]);
                            pp[n][e] = col < row ? pp[n][e] : (col == row ? (e < 2 ? bon0 : bon1) : 0.f);
                            dp[n][e] = col < row ? dp[n][e] : 0.f;
                        }
                    st_half(t_pp + moff[h2], pp);
                    st_half(t_dpp + moff[h2], dp);
                }
            }
            fence_proxy_async();
            tc_fence_before();
            if (!gbar_and(grp, ok)) { alive = false; break; }
            if (gt == 160) {
                tc_fence_after();
                const uint64_t dR = smem_desc(t_rh), dK = smem_desc(t_kh), dV = smem_desc(tv), dY = smem_desc(tdy);
                const uint64_t dS = smem_desc(t_sb), dG = smem_desc(t_gb), dP = smem_desc(t_pp), dD = smem_desc(t_dpp);
                // dR^ and dK^ first (interleaved: products on one accumulator wait for each other), with a commit of
                // their own: the epilogue starts on them while dV is still being formed
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk;
                    tc_mma(tmem + GT_DR, dY + ks, dS + ks, IDESC_K_K, kk > 0);         // dR[t][c] = dY S_0^T
                    tc_mma(tmem + GT_DK, dV + ks, dG + ks, IDESC_K_K, kk > 0);         // dK[i][c] = V G^^T
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk, ms = 128 * kk;
                    tc_mma(tmem + GT_DR, dD + ks, dK + ms, IDESC_K_MN, 1);             // dR += dP' K^
                    tc_mma(tmem + GT_DK, dD + ms, dR + ms, IDESC_MN_MN, 1);            // dK += dP'^T R^
                }
                tc_commit(gb(GB_MRK));
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ks = 2 * kk, ms = 128 * kk;
                    tc_mma(tmem + GT_DV, dK + ks, dG + ms, IDESC_K_MN, kk > 0);        // dV[i][j] = K^ G^
                }
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t ms = 128 * kk;
                    tc_mma(tmem + GT_DV, dP + ms, dY + ms, IDESC_MN_MN, 1);            // dV += P'^T dY
                }
                tc_commit(gb(GB_MV));
            }
            ok = mbar_wait(gb(GB_MRK), mph, abort_flag);
            tc_fence_after();
            // ---- epilogue (the staging tiles take the place of the operand tiles S_0, G^, P', dP': all read by now)
            float z[G_NB][4], qv[G_NB][4];
#pragma unroll
            for (int h2 = 0; h2 < G_H2; ++h2) {
                // q and m take the operands as the tensor core saw them (rounded to bf16): the pair terms that q and
                // m share, and that cancel in the suffix sums, are then the same products on both sides
                float acc[2][4], o[2][4], hat[2][4], rv[2][4], kv[2][4];
                const float pd0 = C2 ? 0.f : gld(GO_DPD + 4 * R0), pd1 = C2 ? 0.f : gld(GO_DPD + 4 * R1);
                tmem_ld_16x16_async2(tacc + GT_DR + 16 * h2, acc);
                ld_half(tr + moff[h2], rv);
                ld_half(tk + moff[h2], kv);
                ld_half(t_rh + moff[h2], hat);
                tmem_ld_done();
                // (two-lane fp32 arithmetic on the pairs of neighbouring columns)
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    const int nn = 2 * h2 + n;
                    const float2 u2 = C2 ? make_float2(0.f, 0.f) : ldsf2(sbase + GS_U + 4 * (cb + 8 * nn));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float2 pd = h ? make_float2(pd1, pd1) : make_float2(pd0, pd0);
                        const float2 ac = make_float2(acc[n][2 * h], acc[n][2 * h + 1]), kk = make_float2(kv[n][2 * h], kv[n][2 * h + 1]);
                        const float2 sr = ex2_2(sub2(make_float2(a[nn][2 * h], a[nn][2 * h + 1]), make_float2(lw2[nn][2 * h], lw2[nn][2 * h + 1])));
                        const float2 oo = C2 ? mul2(ac, sr) : fma2(mul2(u2, kk), pd, mul2(ac, sr));
                        const float2 qq = mul2(ac, make_float2(hat[n][2 * h], hat[n][2 * h + 1]));
                        o[n][2 * h] = oo.x; o[n][2 * h + 1] = oo.y;
                        qv[nn][2 * h] = qq.x; qv[nn][2 * h + 1] = qq.y;
                        if (!C2) {
                            const float2 dd = fma2(mul2(make_float2(rv[n][2 * h], rv[n][2 * h + 1]), kk), pd, make_float2(du_acc[nn][0], du_acc[nn][1]));
                            du_acc[nn][0] = dd.x; du_acc[nn][1] = dd.y;
                        }
                    }
                }
                tmem_ld_16x16_async2(tacc + GT_DK + 16 * h2, acc);
                ld_half(t_kh + moff[h2], hat);
                tmem_ld_done();
                st_half(o_dr + moff[h2], o);
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    const int nn = 2 * h2 + n;
                    const float2 u2 = C2 ? make_float2(0.f, 0.f) : ldsf2(sbase + GS_U + 4 * (cb + 8 * nn));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const float2 pd = h ? make_float2(pd1, pd1) : make_float2(pd0, pd0);
                        const float2 ac = make_float2(acc[n][2 * h], acc[n][2 * h + 1]);
                        const float2 sk = make_float2(ex2(-a[nn][2 * h]), ex2(-a[nn][2 * h + 1]));
                        float2 oo = C2 ? mul2(ac, sk) : fma2(mul2(u2, make_float2(rv[n][2 * h], rv[n][2 * h + 1])), pd, mul2(ac, sk));
                        const float2 zz = sub2(make_float2(qv[nn][2 * h], qv[nn][2 * h + 1]), mul2(ac, make_float2(hat[n][2 * h], hat[n][2 * h + 1])));
                        z[nn][2 * h] = zz.x; z[nn][2 * h + 1] = zz.y;
                        if (C2) {
                            // oo is the gradient of k (1 - w): the key gets (1 - w) of it, and the decay logit its
                            // share through the key factor, folded into the term that leaves the suffix sums
                            const float2 omw = make_float2(one_minus_ex2(lw2[nn][2 * h]), one_minus_ex2(lw2[nn][2 * h + 1]));
                            const float2 qq = fma2(mul2(oo, make_float2(kv[n][2 * h], kv[n][2 * h + 1])), sub2(make_float2(1.f, 1.f), omw),
                                                   make_float2(qv[nn][2 * h], qv[nn][2 * h + 1]));
                            qv[nn][2 * h] = qq.x; qv[nn][2 * h + 1] = qq.y;
                            oo = mul2(oo, omw);
                        }
                        o[n][2 * h] = oo.x; o[n][2 * h + 1] = oo.y;
                    }
                }
                st_half(o_dk + moff[h2], o);
            }
            // dV: every product of the chunk has completed, so x, v, dy can take the group's next chunk
            if (!mbar_wait(gb(GB_MV), mph, abort_flag)) ok = false;
            mph ^= 1;
            tc_fence_after();
            if (gt == 0 && it + 2 < nit) issue_loads_a(it + 2);
            {
                float acc[G_NB][4];
#pragma unroll
                for (int h2 = 0; h2 < G_H2; ++h2) tmem_ld_16x16_async2(tacc + GT_DV + 16 * h2, reinterpret_cast<float (&)[2][4]>(acc[2 * h2]));
                tmem_ld_done();
                st_tile(o_dv, moff, acc);
            }
            tc_fence_before();
            ok = scan_rows<true>(z, gbase + GO_TOT, grp, sp, cb, lane, ok);
            if (!ok) { alive = false; break; }
            if (gt == 0 && it + 2 < nit) issue_loads_b(it + 2);      // (r, k were last read before the barrier of the sums)
#pragma unroll
            for (int n = 0; n < G_NB; ++n) {
                float E0 = 0.f, E1 = 0.f;
#pragma unroll
                for (int o = 0; o < G_NSLAB; ++o) { const float2 ev = ldsf2(gbase + GO_EP + 4 * (o * 64 + cb + 8 * n)); E0 += ev.x; E1 += ev.y; }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float2 dl = sub2(add2(make_float2(E0, E1), make_float2(z[n][2 * h], z[n][2 * h + 1])), make_float2(qv[n][2 * h], qv[n][2 * h + 1]));
                    const float2 dx2 = mul2(dl, mul2(make_float2(lw2[n][2 * h], lw2[n][2 * h + 1]), make_float2(LN2, LN2)));
                    z[n][2 * h] = dx2.x; z[n][2 * h + 1] = dx2.y;
                }
            }
            st_tile(o_dx, moff, z);
        }
        // ---- the chunk's four gradient tiles leave: TMA for a whole chunk, plain stores for a ragged one
        fence_proxy_async();
        gbar(grp);
        if (valid < L) {
            __nv_bfloat16* outs[4] = {p.dr, p.dx, p.dv, p.dk};       // in the order of the staging tiles in shared memory
            for (int i = gt; i < 4 * valid * 8; i += G_GT) {
                const int tile = i / (valid * 8), rem = i % (valid * 8), t = rem >> 3, blk = rem & 7;
                uint32_t w[4];
                lds_v4(t_sb + tile * TILE + swz(t, blk << 4), w);
                *reinterpret_cast<uint4*>(outs[tile] + (size_t)(row0 + (long long)c * L + t) * C + col0 + 8 * blk) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            // every thread has read the staging tiles: the first of them takes the next chunk's start state by TMA at
            // the top of the group's next iteration, issued by one thread that would otherwise not wait for the others
            gbar(grp);
        }
        if (gt == 0) {
            if (valid == L) {
                const int row = (int)(row0 + (long long)c * L);
                tma_store_2d(&tm_dr, col0, row, o_dr);
                tma_store_2d(&tm_dk, col0, row, o_dk);
                tma_store_2d(&tm_dv, col0, row, o_dv);
                tma_store_2d(&tm_dx, col0, row, o_dx);
                bulk_commit();
            }
            if (unsafe && it + 2 < nit) { issue_loads_a(it + 2); issue_loads_b(it + 2); }      // (the other path has issued them)
        }
    }

    if (PACKED && GSUM && nit == 0 && grp == 0) {
        // a segment past its sequence's end: the identity summary (the decay product is stored below)
        float Z[G_NB][4];
#pragma unroll
        for (int n = 0; n < G_NB; ++n) Z[n][0] = Z[n][1] = Z[n][2] = Z[n][3] = 0.f;
        store_f32_block(p.gsum_out + ((size_t)unit * (p.nseg - 1) + (seg - 1)) * GSUM_FLOATS + 64, Z);
    }
    if (PACKED && !GSUM && nit == 0 && seg == 0 && grp == 0 && p.dstate_in) {
        // a sequence without tokens hands the state's gradient through
        float G[G_NB][4];
        if (p.dstate_out) load_f32_block(p.dstate_out + (size_t)unit * 4096, G);
        else {
#pragma unroll
            for (int n = 0; n < G_NB; ++n) G[n][0] = G[n][1] = G[n][2] = G[n][3] = 0.f;
        }
        store_f32_block(p.dstate_in + (size_t)unit * 4096, G);
    }
    // ---- the bonus gradient of this unit: over the lanes' rows, the row groups and the two groups, in a fixed order
    if (!alive && gt == 0) sts32(abort_flag, 1u);    // (the other group's waits see it)
    if (GSUM && cx == 0 && q == 0) { stsf(gbase + GO_REDV + 4 * R0, dprod_lo); stsf(gbase + GO_REDV + 4 * R1, dprod_hi); }
    if (!C2 && !GSUM) {
#pragma unroll
        for (int d = 4; d < 32; d <<= 1)
#pragma unroll
            for (int n = 0; n < G_NB; ++n)
#pragma unroll
                for (int e = 0; e < 2; ++e) du_acc[n][e] += __shfl_xor_sync(0xffffffffu, du_acc[n][e], d);
        if (g == 0) {
#pragma unroll
            for (int n = 0; n < G_NB; ++n)
#pragma unroll
                for (int e = 0; e < 2; ++e) gsm(GO_REDV)[sp * 64 + cb + 8 * n + e] = du_acc[n][e];
        }
    }
    if (gt == 0) {
        bulk_wait<0>();                              // the gradient tiles have reached memory
        // no copy into shared memory may stay in flight
        if (last_a >= 0) mbar_wait(gb(GB_INA), (last_a >> 1) & 1, abort_flag, false);
        if (last_b >= 0) mbar_wait(gb(GB_INB), (last_b >> 1) & 1, abort_flag, false);
        if (last_s >= 0) mbar_wait(gb(GB_S0), (last_s >> 1) & 1, abort_flag, false);
    }
    tc_fence_before();
    __syncthreads();
    if (GSUM && tid < 64 && !lds32(abort_flag))       // the segment's decay: the product over both groups' chunks
        p.gsum_out[((size_t)unit * (p.nseg - 1) + (seg - 1)) * GSUM_FLOATS + tid] =
            ldsf(sbase + GO_REDV + 4 * tid) * ldsf(sbase + GO_BYTES + GO_REDV + 4 * tid);
    if (!C2 && !GSUM && tid < 64 && !lds32(abort_flag)) {
        float s = 0.f;
#pragma unroll
        for (int gg = 0; gg < 2; ++gg) {
            const float* rv4 = reinterpret_cast<const float*>(smem + gg * GO_BYTES + GO_REDV);
            const float* fb = reinterpret_cast<const float*>(smem + gg * GO_BYTES + GO_DUFB);
            s += ((rv4[tid] + rv4[64 + tid]) + (rv4[128 + tid] + rv4[192 + tid])) + fb[tid];
        }
        p.du_part[((size_t)unit * p.nseg + seg) * 64 + tid] = s;
    }
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(lds32(sbase + GS_TMEM), GT_COLS);
    }
}

// du[h][i] = sum over the batch of the units' partial sums: eight strided partial sums in batch order, added in a
// fixed order (deterministic; many sequences do not serialise on one thread)
__global__ void __launch_bounds__(512)
wkv6_backward_chunked_du_kernel(const float* __restrict__ du_part, int B, int H, int nseg, float* __restrict__ du)
{
    __shared__ float part[8][64];
    const int h = blockIdx.x, i = threadIdx.x & 63, grp = threadIdx.x >> 6;
    float acc = 0.f;
    for (int b = grp; b < B; b += 8)
        for (int sg = 0; sg < nseg; ++sg) acc += du_part[(((size_t)b * H + h) * nseg + sg) * 64 + i];
    part[grp][i] = acc;
    __syncthreads();
    if (grp == 0)
        du[h * 64 + i] = ((part[0][i] + part[1][i]) + (part[2][i] + part[3][i])) + ((part[4][i] + part[5][i]) + (part[6][i] + part[7][i]));
}

}  // namespace bc


// The sequence split of a gradient call: as for the forward pass (choose_split), calls with fewer units than half the
// SMs cut every sequence into up to 8 segments of at least 8 chunks.
inline int backward_split(long long units, int T, int n_sm, int* seg_chunks)
{
    size_t unused = 0;
    return choose_split(units, T, n_sm, seg_chunks, &unused);
}

// Workspace of the chunked gradient: checkpoints, bonus gradients per unit and segment, the adjoint's segment
// summaries, the token-by-token path's scratch (one slot of 64 states per SM and group of warps).
inline size_t chunked_backward_workspace_bytes(long long units, int T, int n_sm)
{
    const size_t nck = (size_t)((T + ck::L - 1) / ck::L) + 1;
    int seg_chunks = 0;
    const int nseg = backward_split(units, T, n_sm, &seg_chunks);
    return ((size_t)units * nck * bc::CKPT_FLOATS + (size_t)units * nseg * 64 + (size_t)units * (nseg - 1) * bc::GSUM_FLOATS +
            (size_t)2 * n_sm * bc::FB_SLOT_FLOATS) * sizeof(float);
}

// The same for packed sequences: checkpoints in the packed layout, [H][total_rows / 64 + 2 S] states.
inline size_t backward_order_floats(long long n_seq)       // a counter's 64 bytes and the sequence order, in floats, 16-byte granular
{
    return (size_t)((ORDER_OFFSET / 4 + n_seq + 3) / 4 * 4);
}
// (the most segments a packed call of this many units may be cut into, whatever its longest sequence: the workspace is
// sized for that, so that its size does not depend on max_seqlen)
inline int packed_split_max(long long units, int n_sm)
{
    if (units <= 0 || n_sm <= 0 || units * 2 > n_sm) return 1;
    const long long want = n_sm / units;
    return want > 8 ? 8 : (int)want;
}
inline size_t chunked_backward_varlen_workspace_bytes(long long n_seq, long long total_rows, int H, int n_sm)
{
    const size_t slots = (size_t)(total_rows / ck::L + 2 * n_seq);
    const size_t units = (size_t)n_seq * H, nmax = (size_t)packed_split_max((long long)units, n_sm);
    return ((size_t)H * slots * bc::CKPT_FLOATS + units * nmax * 64 + units * (nmax - 1) * bc::GSUM_FLOATS +
            backward_order_floats(n_seq) + (size_t)2 * n_sm * bc::FB_SLOT_FLOATS) * sizeof(float);
}

// The part of the gradient's workspace that a training step's forward pass may use as its split scratch (the
// token-by-token path's slots: idle until the gradient call).
inline float* backward_workspace_forward_scratch(float* ws, long long units, int T, int n_sm, size_t* bytes)
{
    const size_t nck = (size_t)((T + ck::L - 1) / ck::L) + 1;
    int seg_chunks = 0;
    const int nseg = backward_split(units, T, n_sm, &seg_chunks);
    *bytes = (size_t)2 * n_sm * bc::FB_SLOT_FLOATS * sizeof(float);
    return ws + (size_t)units * nck * bc::CKPT_FLOATS + (size_t)units * nseg * 64 + (size_t)units * (nseg - 1) * bc::GSUM_FLOATS;
}

inline gf_status_t chunked_backward(const __nv_bfloat16* r, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                    const __nv_bfloat16* x, const float* u, const float* state_in,
                                    const __nv_bfloat16* dy, const float* dstate_out, __nv_bfloat16* dr,
                                    __nv_bfloat16* dk, __nv_bfloat16* dv, __nv_bfloat16* dx, float* du, float* dstate_in,
                                    int B, int T, int H, float* ws, cudaStream_t st, std::atomic<uint64_t>* launches,
                                    bool c2 = false, bool ckpt_saved = false, const int32_t* cu = nullptr,
                                    long long packed_rows = 0)
{
    // packed sequences: cu = device cu_seqlens of B sequences over packed_rows rows, T = max_seqlen (the split is cut by it)
    const long long units = (long long)B * H, rows = cu ? packed_rows : (long long)B * T;
    const int n_sm = sm_count();
    if (n_sm <= 0) return GF_ERR_CUDA;
    static PerDeviceFlag attr_set;
    const int dev = current_device();
    if (dev < 0) return GF_ERR_CUDA;
    if (!attr_set.is_set(dev)) {
        if (cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess ||
            cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess ||
            cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess ||
            cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess ||
            cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess ||
            cudaFuncSetAttribute(bc::wkv6_backward_chunked_kernel<false, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, bc::G_SMEM_ALLOC) != cudaSuccess)
            return GF_ERR_CUDA;
        attr_set.set(dev);
    }
    const size_t nck = (size_t)((T + ck::L - 1) / ck::L) + 1;
    int seg_chunks = 0;
    int nseg = backward_split(units, T, n_sm, &seg_chunks);
    if (units * nseg > 0x7fffffffLL) nseg = 1;
    const int nalloc = cu ? packed_split_max(units, n_sm) : nseg;      // (packed: the workspace is laid out for the widest split)
    const long long ckpt_slots = cu ? rows / ck::L + 2LL * B : 0;
    float* ckpt = ws;
    const size_t n_ckpt = cu ? (size_t)H * ckpt_slots : (size_t)units * nck;       // checkpoints: bf16 [64][64] tiles
    if (n_ckpt * 64 >= (1ull << 31)) return GF_ERR_UNSUPPORTED;                    // (32-bit TMA row coordinates)
    float* du_part = ckpt + n_ckpt * bc::CKPT_FLOATS;
    float* gsum = du_part + (size_t)units * nalloc * 64;
    float* fb = gsum + (size_t)units * (nalloc - 1) * bc::GSUM_FLOATS;
    const int32_t* order = nullptr;
    if (cu) {
        // packed: the sequences longest first (the order array lies between the bonus partial sums and the scratch slots)
        unsigned int* counter = reinterpret_cast<unsigned int*>(fb);
        if (B <= ORDER_MAX_SEQ) {
            int32_t* ord = reinterpret_cast<int32_t*>(reinterpret_cast<char*>(fb) + ORDER_OFFSET);
            wkv6_order_kernel<<<1, 1024, 0, st>>>(cu, B, counter, ord);
            launches->fetch_add(1, std::memory_order_relaxed);
            if (cudaGetLastError() != cudaSuccess) return GF_ERR_CUDA;
            order = ord;
        }
        fb += backward_order_floats(B);
    }
    if (!ckpt_saved) {                               // (else the forward pass of the training step left them there)
        // (split calls: the forward summaries borrow the buffer of the adjoint's, which are written after them)
        const gf_status_t s = chunked_checkpoints(k, v, x, state_in, ckpt, B, T, H, st, launches, c2 ? 1 : 0, gsum, nseg, seg_chunks, cu, rows);
        if (s != GF_OK) return s;
    }
    const long long C = (long long)H * 64;
    CUtensorMap tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck;
    if (!ck::make_map(&tck, ckpt, (long long)n_ckpt * 64, 64, 64)) return GF_ERR_CUDA;
    if (!ck::make_map(&tx, x, rows, C, 64) || !ck::make_map(&tr, r, rows, C, 64) || !ck::make_map(&tk, k, rows, C, 64) ||
        !ck::make_map(&tv, v, rows, C, 64) || !ck::make_map(&tdy, dy, rows, C, 64) || !ck::make_map(&tdr, dr, rows, C, 64) ||
        !ck::make_map(&tdk, dk, rows, C, 64) || !ck::make_map(&tdv, dv, rows, C, 64) || !ck::make_map(&tdx, dx, rows, C, 64))
        return GF_ERR_CUDA;
    bc::BParams p{u, dstate_out, dstate_in, reinterpret_cast<const __nv_bfloat16*>(ckpt), du_part, fb, dr, dk, dv, dx, T, H, 2 * n_sm,
                  wait_limit_us().load(std::memory_order_relaxed), gsum, gsum, nseg, seg_chunks};
    const bc::BParamsPacked pp{p, cu, ckpt_slots, order};
    if (nseg > 1) {
        // the adjoint's summaries of every segment but the first (they need no state: the order of the two first launches is free)
        if (cu) bc::wkv6_backward_chunked_kernel<false, true, true><<<(unsigned)(units * (nseg - 1)), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, pp);
        else bc::wkv6_backward_chunked_kernel<false, true><<<(unsigned)(units * (nseg - 1)), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, p);
        launches->fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return GF_ERR_CUDA;
    }
    if (cu && c2) bc::wkv6_backward_chunked_kernel<true, false, true><<<(unsigned)(units * nseg), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, pp);
    else if (cu) bc::wkv6_backward_chunked_kernel<false, false, true><<<(unsigned)(units * nseg), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, pp);
    else if (c2) bc::wkv6_backward_chunked_kernel<true><<<(unsigned)(units * nseg), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, p);
    else bc::wkv6_backward_chunked_kernel<false><<<(unsigned)(units * nseg), bc::G_THREADS, bc::G_SMEM_ALLOC, st>>>(tx, tr, tk, tv, tdy, tdr, tdk, tdv, tdx, tck, p);
    launches->fetch_add(1, std::memory_order_relaxed);
    if (cudaGetLastError() != cudaSuccess) return GF_ERR_CUDA;
    if (c2) return GF_OK;                            // no bonus, no bonus gradient
    bc::wkv6_backward_chunked_du_kernel<<<(unsigned)H, 512, 0, st>>>(du_part, B, H, nseg, du);
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
