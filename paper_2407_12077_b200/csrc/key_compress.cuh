// GOLD key compression for sm_100a: c_t = x_t W^{KD}, the product that ends linear pre-fill in GoldFinch
// (the output of the Finch-C2 layers times the learned D x D/16 matrix gives every token's entry of the
// compressed key cache).  x: [rows][D] bf16, w: [D][Dc] bf16 row-major, c: [rows][Dc] bf16, fp32 accumulate.
//
// With Dc = D/16 the product does 2*Dc = 256 flops per 2-byte element of x it reads (D = 2048): it sits at
// the crossing of the HBM and tensor rooflines, so x is read exactly once and W (D*Dc*2 bytes, L2-resident)
// as rarely as tensor memory allows.  One persistent CTA per SM walks row tiles of MBLK*128 tokens; a tile's
// MBLK x NB accumulators (128 rows x 64 fp32 columns each, NB = ceil(Dc/64)) take, up to Dc = 128, at most 256
// of the 512 columns of tensor memory, so there are two sets: the products of the next tile run while the
// epilogue drains this one (wider outputs fill all 512 columns with one set).  Every 64-row slice of W that
// enters shared memory serves MBLK*128 tokens.
//   warp 0      TMA producer: per 64 input channels, 2*MBLK tiles of x and NB tiles of W into a ring stage
//   warp 1      tensor-memory allocation; an elected lane issues the MBLK*NB*4 tcgen05.mma (128x64x16) of a stage
//   warps 2-5   epilogue: the 32 accumulator rows of the own sub-partition -> bf16 slab -> TMA store (32-row
//               boxes; rows past the end of the tensor are clipped by the store, rows read past it are zero)
// Operands are 128-byte swizzled as TMA delivers them: two stacked 64-token x tiles form the 128-row K-major
// A operand (8-row groups 1024 bytes apart throughout), a W tile is the MN-major B operand of the prefill
// kernel's R^ S_0 product.
// Every wait is bounded (status flag and abort as in the prefill kernel).
#pragma once
#include "wkv6_chunked.cuh"

namespace gf {
namespace kc {

using namespace ck;                                   // PTX wrappers, descriptors, TILE, bounded waits

constexpr int KC_THREADS = 192;
constexpr int KC_RING = 24 * TILE;                    // ring of x and W tiles: 4 stages of up to 6 tiles or 3 of up to 8
constexpr int KC_MAX_NS = 4;
constexpr int KC_OFF_SLAB = KC_RING;                  // [4 warps][32 rows x 128 B]
constexpr int KC_OFF_MISC = KC_OFF_SLAB + 4 * 4096;   // abort word, tensor-memory address, barriers
constexpr int KC_SMEM = KC_OFF_MISC + 256 + 1024;     // + slack for manual 1024-byte alignment
enum { KC_FULL = 0, KC_EMPTY = KC_MAX_NS, KC_ACC_FULL = 2 * KC_MAX_NS, KC_ACC_EMPTY = KC_ACC_FULL + 2, KC_BAR_COUNT = KC_ACC_EMPTY + 2 };
static_assert(16 + 8 * KC_BAR_COUNT <= 256, "barrier block");
// instruction descriptor: fp32 accumulator, bf16 A (K-major) and B (MN-major), M = 128, N = 64
constexpr uint32_t KC_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

struct KcParams {
    long long rows;
    int ksteps;                                       // ceil(D / 64)
};

// One accumulator row per lane: 32 consecutive fp32 columns of the lane's row in this warp's sub-partition.
__device__ __forceinline__ void tmem_ld_row32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}

template <int MBLK, int NB>
__global__ void __launch_bounds__(KC_THREADS, 1)
key_compress_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_c32, const KcParams p)
{
    constexpr int STAGE_TILES = 2 * MBLK + NB;       // x tiles + W tiles per stage
    constexpr int KC_NS = STAGE_TILES <= 6 ? 4 : 3;  // ring stages
    constexpr int KC_STAGE = STAGE_TILES * TILE;
    static_assert(KC_NS * KC_STAGE <= KC_RING && MBLK * NB * 64 <= 512, "tile shape");
    // a tile's accumulators in up to 256 columns: two sets, the epilogue of one tile overlaps the products of the
    // next; in 512 columns: one set
    constexpr int NSETS = MBLK * NB * 64 <= 256 ? 2 : 1;
    constexpr int ACC_COLS = 512 / NSETS;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t abort_flag = sbase + KC_OFF_MISC;
    auto bar = [&](int i) { return sbase + KC_OFF_MISC + 16 + 8 * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tile_rows = (long long)MBLK * 128;
    const long long n_tiles = (p.rows + tile_rows - 1) / tile_rows;

    if (tid == 0) {
        for (int i = 0; i < KC_NS; ++i) {
            mbar_init(bar(KC_FULL + i), 1);
            mbar_init(bar(KC_EMPTY + i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(KC_ACC_FULL + i), 1);
            mbar_init(bar(KC_ACC_EMPTY + i), 4);
        }
        sts32(abort_flag, 0u);
        sts32(abort_flag + 4, ck::WAIT_LIMIT_US);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(sbase + KC_OFF_MISC + 8, 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = lds32(sbase + KC_OFF_MISC + 8);

    if (warp == 0) {
        // ============================== TMA producer ==============================
        int it = 0, issued = 0;
        bool alive = true;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x) {
            const int row0 = (int)(t * tile_rows);
            for (int ks = 0; ks < p.ksteps; ++ks, ++it) {
                const int s = it % KC_NS;
                if (it >= KC_NS && !mbar_wait_warp(bar(KC_EMPTY + s), ((it / KC_NS) + 1) & 1, abort_flag)) { alive = false; break; }
                const uint32_t dst = sbase + s * KC_STAGE;
                if (elect_one()) {
                    mbar_expect_tx(bar(KC_FULL + s), (2 * MBLK + NB) * TILE);
#pragma unroll
                    for (int mb = 0; mb < 2 * MBLK; ++mb) tma_load_2d(dst + mb * TILE, &tm_x, ks * 64, row0 + 64 * mb, bar(KC_FULL + s));
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb) tma_load_2d(dst + (2 * MBLK + nb) * TILE, &tm_w, nb * 64, ks * 64, bar(KC_FULL + s));
                }
                __syncwarp();
                issued = it + 1;
            }
        }
        // do not leave while copies into this CTA's shared memory may still be in flight
        for (int c = max(0, issued - KC_NS); c < issued; ++c)
            mbar_wait_warp(bar(KC_FULL + c % KC_NS), (c / KC_NS) & 1, abort_flag, false);
    } else if (warp == 1) {
        // ============================== MMA issuer ==============================
        int it = 0, ti = 0;
        bool alive = true;
        for (long long t = blockIdx.x; t < n_tiles && alive; t += gridDim.x, ++ti) {
            const int ab = NSETS == 2 ? (ti & 1) : 0, use = NSETS == 2 ? (ti >> 1) : ti;   // accumulator set and its use count
            // the epilogue has read this set's previous tile out of tensor memory
            if (use >= 1 && !mbar_wait_warp(bar(KC_ACC_EMPTY + ab), (use + 1) & 1, abort_flag)) break;
            tc_fence_after();
            for (int ks = 0; ks < p.ksteps; ++ks, ++it) {
                const int s = it % KC_NS;
                if (!mbar_wait_warp(bar(KC_FULL + s), (it / KC_NS) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t st = sbase + s * KC_STAGE;
#pragma unroll
                    for (int mb = 0; mb < MBLK; ++mb) {
                        const uint64_t da = smem_desc(st + 2 * mb * TILE);       // 128 rows: two stacked x tiles
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {
                            const uint64_t db = smem_desc(st + (2 * MBLK + nb) * TILE);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                tc_mma(tmem + ACC_COLS * ab + 64 * (mb * NB + nb), da + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk),
                                       KC_IDESC, (ks > 0 || kk > 0) ? 1u : 0u);
                        }
                    }
                    tc_commit(bar(KC_EMPTY + s));                    // the stage is free once these products are done
                    if (ks == p.ksteps - 1) tc_commit(bar(KC_ACC_FULL + ab));
                }
                __syncwarp();
            }
        }
    } else {
        // ============================== epilogue warps ==============================
        const int sp = warp & 3;                     // tensor-memory sub-partition: accumulator rows 32*sp .. 32*sp+31
        const uint32_t slab = sbase + KC_OFF_SLAB + (warp - 2) * 4096;
        int ti = 0;
        for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x, ++ti) {
            const int ab = NSETS == 2 ? (ti & 1) : 0, use = NSETS == 2 ? (ti >> 1) : ti;
            if (!mbar_wait(bar(KC_ACC_FULL + ab), use & 1, abort_flag)) break;
            tc_fence_after();
            const long long row0 = t * tile_rows;
#pragma unroll
            for (int mb = 0; mb < MBLK; ++mb) {
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    const uint32_t ta = tmem + ((uint32_t)(32 * sp) << 16) + ACC_COLS * ab + 64 * (mb * NB + nb);
                    if (lane == 0) bulk_wait_read<0>();          // this warp's previous store has finished reading the slab
                    __syncwarp();
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t v[32];
                        tmem_ld_row32(ta + 32 * half, v);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {            // 8 columns = one 16-byte unit of this lane's row
                            const uint32_t w0 = pack_bf16(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1]));
                            const uint32_t w1 = pack_bf16(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3]));
                            const uint32_t w2 = pack_bf16(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5]));
                            const uint32_t w3 = pack_bf16(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]));
                            asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};"
                                         ::"r"(slab + swz(lane, (4 * half + q) << 4)), "r"(w0), "r"(w1), "r"(w2), "r"(w3) : "memory");
                        }
                    }
                    fence_proxy_async();
                    __syncwarp();
                    const long long grow = row0 + 128 * mb + 32 * sp;
                    if (lane == 0 && grow < p.rows) {
                        tma_store_2d(&tm_c32, nb * 64, (int)grow, slab);
                        bulk_commit();
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            mbar_arrive_if(bar(KC_ACC_EMPTY + ab), lane == 0);
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

}  // namespace kc

// c[rows][Dc] = x[rows][D] w[D][Dc]; D and Dc multiples of 8 (16-byte rows for TMA), Dc <= 256.  Widths that are not
// multiples of 64 ride on TMA's bounds handling: the missing input channels and output columns are read as zeros
// and the store clips the columns past Dc.
inline gf_status_t key_compress(const __nv_bfloat16* x, const __nv_bfloat16* w, __nv_bfloat16* c, long long rows, int D, int Dc,
                                cudaStream_t st, std::atomic<uint64_t>* launches)
{
    if (rows <= 0 || rows >= (1LL << 31) - 256 || D <= 0 || (D & 7) || Dc <= 0 || (Dc & 7) || Dc > 256) return GF_ERR_INVALID_ARG;
    const int n_sm = sm_count();
    const int dev = current_device();
    if (n_sm <= 0 || dev < 0) return GF_ERR_CUDA;
    static PerDeviceFlag attr_set;
    if (!attr_set.is_set(dev)) {
        if (cudaFuncSetAttribute(kc::key_compress_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<1, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<1, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess)
            return GF_ERR_CUDA;
        attr_set.set(dev);
    }
    CUtensorMap tx, tw, tc;
    if (!ck::make_map(&tx, x, rows, D, 64) || !ck::make_map(&tw, w, D, Dc, 64) || !ck::make_map(&tc, c, rows, Dc, 32)) return GF_ERR_CUDA;
    // 256-row tiles halve the re-reads of W but need enough rows to give every SM a tile
    const int nb = (Dc + 63) / 64, mblk = rows >= 256LL * n_sm ? 2 : 1;
    const long long n_tiles = (rows + 128LL * mblk - 1) / (128LL * mblk);
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);
    kc::KcParams p{rows, (D + 63) / 64};
    if (mblk == 2) {
        switch (nb) {
        case 1: kc::key_compress_kernel<2, 1><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        case 2: kc::key_compress_kernel<2, 2><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        case 3: kc::key_compress_kernel<2, 3><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        default: kc::key_compress_kernel<2, 4><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        }
    } else {
        switch (nb) {
        case 1: kc::key_compress_kernel<1, 1><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        case 2: kc::key_compress_kernel<1, 2><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        case 3: kc::key_compress_kernel<1, 3><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        default: kc::key_compress_kernel<1, 4><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
        }
    }
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
