// GOLD key compression for sm_100a: c_t = x_t W^{KD}, the product that ends linear pre-fill in GoldFinch
// (the output of the Finch-C2 layers times the learned D x D/16 matrix gives every token's entry of the
// compressed key cache).  x: [rows][D] bf16, w: [D][Dc] bf16 row-major, c: [rows][Dc] bf16, fp32 accumulate.
//
// With Dc = D/16 the product does 2*Dc = 256 flops per 2-byte element of x it reads (D = 2048): it sits at
// the crossing of the HBM and tensor rooflines, so x is read exactly once and W (D*Dc*2 bytes, L2-resident)
// as rarely as tensor memory allows.  One persistent CTA per SM walks row tiles of MB*64 tokens; a tile's
// MB x NB accumulators of 64 x 64 fp32 (NB = Dc/64) fill the 512 columns of tensor memory, so every 64-row
// slice of W that enters shared memory serves MB*64 tokens.
//   warp 0      TMA producer: per 64 input channels, MB tiles of x and NB tiles of W into a ring stage
//   warp 1      tensor-memory allocation; an elected lane issues the MB*NB*4 tcgen05.mma (64x64x16) of a stage
//   warps 2-5   epilogue: accumulator rows of the own sub-partition -> bf16 slab -> TMA store (16-row boxes;
//               rows past the end of the tensor are clipped by the store, rows read past it are zero filled)
// Operand tiles and descriptors are those of the prefill kernel's R^ S_0 product: x tile K-major (tokens x
// channels), W tile MN-major (channels x outputs), both 128-byte swizzled as TMA delivers them.
// Every wait is bounded (status flag and abort as in the prefill kernel).
#pragma once
#include "wkv6_chunked.cuh"

namespace gf {
namespace kc {

using namespace ck;                                   // PTX wrappers, descriptors, TILE, bounded waits

constexpr int KC_THREADS = 192;
constexpr int KC_NS = 4;                              // ring stages
constexpr int KC_MAX_TILES = 6;                       // x tiles + W tiles per stage (48 KB)
constexpr int KC_STAGE = KC_MAX_TILES * TILE;
constexpr int KC_OFF_SLAB = KC_NS * KC_STAGE;         // [4 warps][16 rows x 128 B]
constexpr int KC_OFF_MISC = KC_OFF_SLAB + 4 * 2048;   // abort word, tensor-memory address, barriers
constexpr int KC_SMEM = KC_OFF_MISC + 256 + 1024;     // + slack for manual 1024-byte alignment
enum { KC_FULL = 0, KC_EMPTY = KC_NS, KC_ACC_FULL = 2 * KC_NS, KC_ACC_EMPTY, KC_BAR_COUNT };
static_assert(16 + 8 * KC_BAR_COUNT <= 256, "barrier block");

struct KcParams {
    long long rows;
    int ksteps;                                       // D / 64
};

template <int MB, int NB>
__global__ void __launch_bounds__(KC_THREADS, 1)
key_compress_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_c16, const KcParams p)
{
    static_assert(MB + NB <= KC_MAX_TILES && MB * NB <= 8, "tile shape");
    constexpr uint32_t TM_COLS_KC = MB * NB * 64 <= 256 ? 256 : 512;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t abort_flag = sbase + KC_OFF_MISC;
    auto bar = [&](int i) { return sbase + KC_OFF_MISC + 16 + 8 * i; };
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long tile_rows = (long long)MB * 64;
    const long long n_tiles = (p.rows + tile_rows - 1) / tile_rows;

    if (tid == 0) {
        for (int i = 0; i < KC_NS; ++i) {
            mbar_init(bar(KC_FULL + i), 1);
            mbar_init(bar(KC_EMPTY + i), 1);
        }
        mbar_init(bar(KC_ACC_FULL), 1);
        mbar_init(bar(KC_ACC_EMPTY), 4);
        sts32(abort_flag, 0u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(sbase + KC_OFF_MISC + 8, TM_COLS_KC);
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
                    mbar_expect_tx(bar(KC_FULL + s), (MB + NB) * TILE);
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb) tma_load_2d(dst + mb * TILE, &tm_x, ks * 64, row0 + 64 * mb, bar(KC_FULL + s));
#pragma unroll
                    for (int nb = 0; nb < NB; ++nb) tma_load_2d(dst + (MB + nb) * TILE, &tm_w, nb * 64, ks * 64, bar(KC_FULL + s));
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
            // the epilogue has read the previous tile's accumulators out of tensor memory
            if (ti >= 1 && !mbar_wait_warp(bar(KC_ACC_EMPTY), (ti - 1) & 1, abort_flag)) break;
            tc_fence_after();
            for (int ks = 0; ks < p.ksteps; ++ks, ++it) {
                const int s = it % KC_NS;
                if (!mbar_wait_warp(bar(KC_FULL + s), (it / KC_NS) & 1, abort_flag)) { alive = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t st = sbase + s * KC_STAGE;
#pragma unroll
                    for (int mb = 0; mb < MB; ++mb) {
                        const uint64_t da = smem_desc(st + mb * TILE);
#pragma unroll
                        for (int nb = 0; nb < NB; ++nb) {
                            const uint64_t db = smem_desc(st + (MB + nb) * TILE);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                tc_mma(tmem + 64 * (mb * NB + nb), da + (uint64_t)(2 * kk), db + (uint64_t)(128 * kk), IDESC_K_MN,
                                       (ks > 0 || kk > 0) ? 1u : 0u);
                        }
                    }
                    tc_commit(bar(KC_EMPTY + s));                    // the stage is free once these products are done
                    if (ks == p.ksteps - 1) tc_commit(bar(KC_ACC_FULL));
                }
                __syncwarp();
            }
        }
    } else {
        // ============================== epilogue warps ==============================
        const int sp = warp & 3;                     // tensor-memory sub-partition: accumulator rows 16*sp .. 16*sp+15
        const uint32_t slab = sbase + KC_OFF_SLAB + (warp - 2) * 2048;
        int ti = 0;
        for (long long t = blockIdx.x; t < n_tiles; t += gridDim.x, ++ti) {
            if (!mbar_wait(bar(KC_ACC_FULL), ti & 1, abort_flag)) break;
            tc_fence_after();
            const long long row0 = t * tile_rows;
#pragma unroll
            for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
                for (int nb = 0; nb < NB; ++nb) {
                    const uint32_t ta = tmem + ((uint32_t)(32 * sp) << 16) + 64 * (mb * NB + nb);
                    float acc[4][4];
                    if (lane == 0) bulk_wait_read<0>();          // this warp's previous store has finished reading the slab
                    __syncwarp();
                    tmem_ld_16x32(ta, acc);
                    store_half_bf16<0>(slab, 0, acc, lane);
                    tmem_ld_16x32(ta + 32, acc);
                    store_half_bf16<1>(slab, 0, acc, lane);
                    fence_proxy_async();
                    __syncwarp();
                    const long long grow = row0 + 64 * mb + 16 * sp;
                    if (lane == 0 && grow < p.rows) {
                        tma_store_2d(&tm_c16, nb * 64, (int)grow, slab);
                        bulk_commit();
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            mbar_arrive_if(bar(KC_ACC_EMPTY), lane == 0);
        }
        if (lane == 0) bulk_wait<0>();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem, TM_COLS_KC);
    }
}

}  // namespace kc

// c[rows][Dc] = x[rows][D] w[D][Dc]; D a multiple of 64, Dc in {64, 128, 192, 256}.
inline gf_status_t key_compress(const __nv_bfloat16* x, const __nv_bfloat16* w, __nv_bfloat16* c, long long rows, int D, int Dc,
                                cudaStream_t st, std::atomic<uint64_t>* launches)
{
    if (rows <= 0 || rows >= (1LL << 31) - 256 || D <= 0 || (D & 63) || Dc <= 0 || (Dc & 63) || Dc > 256) return GF_ERR_INVALID_ARG;
    const int n_sm = sm_count();
    const int dev = current_device();
    if (n_sm <= 0 || dev < 0) return GF_ERR_CUDA;
    static PerDeviceFlag attr_set;
    if (!attr_set.is_set(dev)) {
        if (cudaFuncSetAttribute(kc::key_compress_kernel<4, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess ||
            cudaFuncSetAttribute(kc::key_compress_kernel<2, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kc::KC_SMEM) != cudaSuccess)
            return GF_ERR_CUDA;
        attr_set.set(dev);
    }
    CUtensorMap tx, tw, tc;
    if (!ck::make_map(&tx, x, rows, D, 64) || !ck::make_map(&tw, w, D, Dc, 64) || !ck::make_map(&tc, c, rows, Dc, 16)) return GF_ERR_CUDA;
    const int nb = Dc / 64, mb = nb <= 2 ? 4 : 2;
    const long long n_tiles = (rows + 64LL * mb - 1) / (64LL * mb);
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);
    kc::KcParams p{rows, D / 64};
    switch (nb) {
    case 1: kc::key_compress_kernel<4, 1><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
    case 2: kc::key_compress_kernel<4, 2><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
    case 3: kc::key_compress_kernel<2, 3><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
    default: kc::key_compress_kernel<2, 4><<<grid, kc::KC_THREADS, kc::KC_SMEM, st>>>(tx, tw, tc, p); break;
    }
    launches->fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

}  // namespace gf
