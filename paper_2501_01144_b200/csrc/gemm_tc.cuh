// Tensor-core GEMM for sm_100a: Y[M,N] = A[M,K] * B[N,K]^T with one power-of-two
// scale per 32 elements of K on each operand (Sec. 3.3: products inside a block
// share the exponent sum eA + eB; here the block-scaled MMA applies it in hardware).
//
// Operands arrive as plain [rows][K] byte matrices holding the E4M3 encoding of
// 0.5 * value (exact: every DialectFP4 magnitude has at most four significant bits)
// and as scale atoms (bd_common.cuh) holding e + 127 as UE8M0.  TMA loads 128-byte
// swizzled K-major tiles and the scale atoms into a ring of shared-memory stages;
// one thread issues tcgen05.cp (scales -> TMEM) and tcgen05.mma.kind::mxf8f6f4
// .block_scale (K = 32 per instruction = one block) into a TMEM accumulator; four
// epilogue warps read the accumulator with tcgen05.ld and store fp32 or bf16.
//
// Every wait on an mbarrier is bounded: when the limit is reached the kernel
// records kStatusTimeout, stops waiting everywhere, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <stdlib.h>
#include <cuda_bf16.h>

#include "bd_common.cuh"
#include "ptx_sm100.cuh"
#include "quantize.cuh"

#ifndef BD_FUSED_EXP
#define BD_FUSED_EXP 0
#endif

namespace bd {
namespace tc {

constexpr int BM = 128;            // rows of A per tile = MMA M = TMEM lanes
constexpr int BK = 128;            // bytes of K per stage = one 128-byte swizzle row = 4 blocks
constexpr int kThreads = 192;      // warp 0: TMA, warp 1: MMA + TMEM, warps 2..5: epilogue

template <int BN>
struct Config {
    static constexpr int kStages = BN == 256 ? 4 : 6;
    static constexpr int kATile = BM * BK;                       // 16 KiB
    static constexpr int kBTile = BN * BK;
    static constexpr int kSfA = kScaleAtomBytes;
    static constexpr int kSfB = (BN / 128) * kScaleAtomBytes;
    static constexpr int kStageBytes = kATile + kBTile + kSfA + kSfB;
    static constexpr int kSmemBytes = kStages * kStageBytes + 1024 /* alignment slack */ + 256 /* barriers */;
    static constexpr int kAccCols = BN;
    static constexpr int kSfaCol = BN;
    static constexpr int kSfbCol = BN + 4;
    static constexpr int kTmemCols = BN == 256 ? 512 : 256;      // power of two >= BN + 4 + 4 * BN / 128
};

__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_cp_32x128b_warpx4(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tcgen05_mma_mxf8(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                 uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
}
__device__ __forceinline__ void tcgen05_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tcgen05_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bit): start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1, swizzle mode in bits 61..63.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((addr >> 4) & 0x3fffu) | (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16 |
           (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32 | (uint64_t)1 << 46 | (uint64_t)layout << 61;
}
constexpr uint32_t kLayoutSwizzle128 = 2, kLayoutNone = 0;
// The same descriptor split in two words, so that the issuing thread only adds to the low one:
// low = (addr >> 4) | (lbo >> 4) << 16, high = (sbo >> 4) | version 1 << 14 | layout << 29.
__device__ __forceinline__ uint32_t desc_hi(uint32_t sbo_bytes, uint32_t layout) {
    return ((sbo_bytes >> 4) & 0x3fffu) | 1u << 14 | layout << 29;
}
__device__ __forceinline__ uint64_t desc_join(uint32_t lo, uint32_t hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}

// Instruction descriptor of the block-scaled MMA: E4M3 x E4M3 (format 0), both K-major,
// UE8M0 scales, N >> 3 at bit 17, M >> 4 at bit 24, scale byte selectors at bits 4 (B) and 29 (A).
template <int BN>
__device__ __forceinline__ uint32_t instr_desc(uint32_t sf_id) {
    return (uint32_t)(BN >> 3) << 17 | 1u << 23 | (uint32_t)(BM >> 4) << 24 | sf_id << 4 | sf_id << 29;
}

template <int BN, int MODE = 0>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               const uint8_t *__restrict__ sfA, const uint8_t *__restrict__ sfB, int M, int N, int K,
               int row_tiles_a, int row_tiles_b, void *__restrict__ Y, int64_t ldy, int out_bf16) {
    using C = Config<BN>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    // all A tiles, then all B tiles (both 1024-byte aligned for the 128-byte swizzle), then the scale atoms
    auto a_tile = [&](int s) { return base + (uint32_t)s * C::kATile; };
    auto b_tile = [&](int s) { return base + (uint32_t)C::kStages * C::kATile + (uint32_t)s * C::kBTile; };
    auto sfa_tile = [&](int s) { return base + (uint32_t)C::kStages * (C::kATile + C::kBTile) + (uint32_t)s * C::kSfA; };
    auto sfb_tile = [&](int s) {
        return base + (uint32_t)C::kStages * (C::kATile + C::kBTile + C::kSfA) + (uint32_t)s * C::kSfB;
    };
    const uint32_t bars = base + C::kStages * C::kStageBytes;              // full[S], empty[S], tmem_full
    volatile uint32_t *const shared_words = (volatile uint32_t *)(base_ptr + C::kStages * C::kStageBytes + 128);
    volatile uint32_t *const tmem_slot = shared_words;                     // TMEM base address
    volatile uint32_t *const abort_flag = shared_words + 1;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
    const int k_tiles = (K + BK - 1) / BK;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (C::kStages + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * C::kStages);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < C::kStages; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void *)tmem_slot)), "r"((uint32_t)C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer ----
            const int atoms_b = min(BN / 128, row_tiles_b - blockIdx.x * (BN / 128));
            const uint32_t tx = C::kATile + C::kBTile + C::kSfA + (uint32_t)atoms_b * kScaleAtomBytes;
            int issued = 0;
            for (int kt = 0; kt < k_tiles; kt++) {
                const int s = kt % C::kStages;
                if ((MODE & 8) && kt >= C::kStages) break;
                mbar_wait(empty_bar(s), ((kt / C::kStages) & 1) ^ 1, abort_flag);
                if (*abort_flag) break;
                if ((MODE & 1) && kt >= C::kStages) {               // experiment: no loads after the ring is filled
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full_bar(s)) : "memory");
                    issued = kt + 1;
                    continue;
                }
                mbar_expect_tx(full_bar(s), tx);
                tma_load_2d(a_tile(s), &mapA, kt * BK, m0, full_bar(s));
                tma_load_2d(b_tile(s), &mapB, kt * BK, n0, full_bar(s));
                bulk_load(sfa_tile(s), sfA + ((int64_t)kt * row_tiles_a + blockIdx.y) * kScaleAtomBytes,
                          kScaleAtomBytes, full_bar(s));
                bulk_load(sfb_tile(s), sfB + ((int64_t)kt * row_tiles_b + blockIdx.x * (BN / 128)) * kScaleAtomBytes,
                          (uint32_t)atoms_b * kScaleAtomBytes, full_bar(s));
                issued = kt + 1;
            }
            if (*abort_flag) {
                // bounded wait for this thread's own copies still in flight before the CTA may exit
                for (int kt = max(0, issued - C::kStages); kt < issued; kt++)
                    for (uint32_t spin = 0; spin < (1u << 20); spin++)
                        if (mbar_try_wait(full_bar(kt % C::kStages), (kt / C::kStages) & 1)) break;
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer ----
            for (int kt = 0; kt < k_tiles; kt++) {
                const int s = kt % C::kStages;
                if (!(MODE & 8) || kt < C::kStages) mbar_wait(full_bar(s), (kt / C::kStages) & 1, abort_flag);
                if (*abort_flag) break;
                tcgen05_fence_after();
                const uint32_t sfa_s = sfa_tile(s), sfb_s = sfb_tile(s);
                if (!(MODE & 4) || kt == 0)
                tcgen05_cp_32x128b_warpx4(tmem + C::kSfaCol, smem_desc(sfa_s, 0, 128, kLayoutNone));
                if (!(MODE & 4) || kt == 0)
#pragma unroll
                for (int j = 0; j < BN / 128; j++)
                    tcgen05_cp_32x128b_warpx4(tmem + C::kSfbCol + 4 * j,
                                              smem_desc(sfb_s + j * kScaleAtomBytes, 0, 128, kLayoutNone));
#pragma unroll
                for (int k = 0; k < ((MODE & 2) ? 0 : BK / 32); k++) {
                    const uint64_t da = smem_desc(a_tile(s) + 32 * k, 16, 1024, kLayoutSwizzle128);
                    const uint64_t db = smem_desc(b_tile(s) + 32 * k, 16, 1024, kLayoutSwizzle128);
                    if (MODE & 16) {                               // experiment: plain (unscaled) FP8 kind, timing only
                        const uint32_t idesc = 1u << 4 | (uint32_t)(BN >> 3) << 17 | (uint32_t)(BM >> 4) << 24;
                        asm volatile(
                            "{\n\t.reg .pred p;\n\t"
                            "setp.ne.b32 p, %4, 0;\n\t"
                            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
                            ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"((uint32_t)((kt | k) != 0)) : "memory");
                    } else
                    tcgen05_mma_mxf8(tmem, da, db, instr_desc<BN>(k), tmem + C::kSfaCol, tmem + C::kSfbCol,
                                     (kt | k) != 0);
                }
                tcgen05_commit(empty_bar(s));                      // stage free once these MMAs have read it
            }
            tcgen05_commit(tmem_full_bar);                         // accumulator complete
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 * (w % 4) .. + 31 ----
        mbar_wait(tmem_full_bar, 0, abort_flag, 256);
        tcgen05_fence_after();
        const int quad = warp % 4;
        const int row = m0 + quad * 32 + lane;
        const bool vec_ok = (ldy % 8 == 0) && (((uintptr_t)Y & 15u) == 0);
#pragma unroll 1
        for (int c = 0; c < BN / 32; c++) {
            uint32_t r[32];
            tcgen05_ld_32x32b_x32(tmem + ((uint32_t)(quad * 32) << 16) + c * 32, r);
            tcgen05_wait_ld();
            const int col = n0 + c * 32;
            if (row >= M || col >= N || *abort_flag) continue;
            if (out_bf16) {
                __nv_bfloat16 *dst = (__nv_bfloat16 *)Y + (int64_t)row * ldy + col;
                if (vec_ok && col + 32 <= N) {
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        uint32_t p[4];
#pragma unroll
                        for (int j = 0; j < 4; j++) {
                            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * i + 2 * j]),
                                                                     __uint_as_float(r[8 * i + 2 * j + 1]));
                            p[j] = *(uint32_t *)&h;
                        }
                        ((uint4 *)dst)[i] = make_uint4(p[0], p[1], p[2], p[3]);
                    }
                } else {
                    for (int i = 0; i < 32 && col + i < N; i++) dst[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
                }
            } else {
                float *dst = (float *)Y + (int64_t)row * ldy + col;
                if (vec_ok && col + 32 <= N) {
#pragma unroll
                    for (int i = 0; i < 8; i++)
                        ((uint4 *)dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
                } else {
                    for (int i = 0; i < 32 && col + i < N; i++) dst[i] = __uint_as_float(r[i]);
                }
            }
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)C::kTmemCols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------
// Two-CTA variant: a cluster of two CTAs on neighbouring SMs computes a 256 x 256 tile
// with tcgen05.mma.cta_group::2.  CTA r of the pair loads rows [128 r, 128 r + 128) of
// the A tile and of the B tile, so each SM reads half as much B from shared memory per
// MMA as the one-CTA kernel; the leader (rank 0) issues the scale copies and the MMAs
// for both; each CTA owns the accumulator rows of its own A half and stores them.
// All loads complete on the leader's "full" barrier; the leader's commit frees the
// stage in both CTAs.
// ---------------------------------------------------------------------------
constexpr int kStages2 = 6;
constexpr int kHalfTile = 128 * BK;                               // 16 KiB: A half or B half
constexpr int kStage2Bytes = 2 * kHalfTile + kScaleAtomBytes + 2 * kScaleAtomBytes;
constexpr int kSmem2Bytes = kStages2 * kStage2Bytes + 1024 + 256;

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tcgen05_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tcgen05_cp_pair(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tcgen05_mma_mxf8_pair(uint32_t d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                                      uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
}

// Store one 32-column chunk of an accumulator row (fp32 registers) as fp32 or bf16.
__device__ __forceinline__ void store_chunk(const uint32_t (&r)[32], void *Y, int64_t ldy, int row, int col, int N,
                                            int out_bf16, bool vec_ok) {
    if (out_bf16) {
        __nv_bfloat16 *dst = (__nv_bfloat16 *)Y + (int64_t)row * ldy + col;
        if (vec_ok && col + 32 <= N) {
#pragma unroll
            for (int i = 0; i < 4; i++) {
                uint32_t p[4];
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[8 * i + 2 * j]),
                                                             __uint_as_float(r[8 * i + 2 * j + 1]));
                    p[j] = *(uint32_t *)&h;
                }
                ((uint4 *)dst)[i] = make_uint4(p[0], p[1], p[2], p[3]);
            }
        } else {
            for (int i = 0; i < 32 && col + i < N; i++) dst[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
        }
    } else {
        float *dst = (float *)Y + (int64_t)row * ldy + col;
        if (vec_ok && col + 32 <= N) {
#pragma unroll
            for (int i = 0; i < 8; i++) ((uint4 *)dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
        } else {
            for (int i = 0; i < 32 && col + i < N; i++) dst[i] = __uint_as_float(r[i]);
        }
    }
}

template <int MODE = 0>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const __grid_constant__ CUtensorMap mapSfA, const __grid_constant__ CUtensorMap mapSfB, int M, int N,
                int K, int row_tiles_a, int row_tiles_b, void *__restrict__ Y, int64_t ldy, int out_bf16) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto a_tile = [&](int s) { return base + (uint32_t)s * kHalfTile; };
    auto b_tile = [&](int s) { return base + (uint32_t)(kStages2 + s) * kHalfTile; };
    auto sfa_tile = [&](int s) { return base + (uint32_t)(2 * kStages2) * kHalfTile + (uint32_t)s * kScaleAtomBytes; };
    auto sfb_tile = [&](int s) {
        return base + (uint32_t)(2 * kStages2) * kHalfTile + (uint32_t)(kStages2 + 2 * s) * kScaleAtomBytes;
    };
    const uint32_t bars = base + kStages2 * kStage2Bytes;
    volatile uint32_t *const shared_words = (volatile uint32_t *)(base_ptr + kStages2 * kStage2Bytes + 128);
    volatile uint32_t *const tmem_slot = shared_words;
    volatile uint32_t *const abort_flag = shared_words + 1;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kStages2 + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * kStages2);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();                      // 0 = leader
    const int pair = blockIdx.x / 2;
    const int m0 = pair * 256 + (int)rank * 128;                  // this CTA's accumulator rows
    const int n0 = blockIdx.y * 256;
    const int k_tiles = (K + BK - 1) / BK;
    constexpr int kAccCols = 256, kSfaCol = 256, kSfbCol = 260, kTmemCols = 512;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages2; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void *)tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                           // both CTAs: barriers initialised, TMEM allocated
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer (both CTAs); every copy completes on the leader's full barrier ----
            constexpr uint32_t tx_pair = 2u * (2u * kHalfTile + 3u * kScaleAtomBytes);
            int issued = 0;
            for (int kt = 0; kt < k_tiles; kt++) {
                const int s = kt % kStages2;
                if ((MODE & 8) && kt >= kStages2) break;
                mbar_wait(empty_bar(s), ((kt / kStages2) & 1) ^ 1, abort_flag);
                if (*abort_flag) break;
                const uint32_t fb = map_to_cta(full_bar(s), 0);
                if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
                tma_load_2d_pair(a_tile(s), &mapA, kt * BK, m0, fb);
                tma_load_2d_pair(b_tile(s), &mapB, kt * BK, n0 + (int)rank * 128, fb);
                tma_load_2d_pair(sfa_tile(s), &mapSfA, 0, kt * row_tiles_a + pair * 2 + (int)rank, fb);
                tma_load_2d_pair(sfb_tile(s), &mapSfB, 0, kt * row_tiles_b + blockIdx.y * 2, fb);
                issued = kt + 1;
            }
            (void)issued;
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            // ---- MMA issuer (leader only) ----
            for (int kt = 0; kt < k_tiles; kt++) {
                const int s = kt % kStages2;
                if (!(MODE & 8) || kt < kStages2) mbar_wait(full_bar(s), (kt / kStages2) & 1, abort_flag);
                if (*abort_flag) break;
                tcgen05_fence_after();
                if (!(MODE & 4) || kt == 0) {
                tcgen05_cp_pair(tmem + kSfaCol, smem_desc(sfa_tile(s), 0, 128, kLayoutNone));
                tcgen05_cp_pair(tmem + kSfbCol, smem_desc(sfb_tile(s), 0, 128, kLayoutNone));
                tcgen05_cp_pair(tmem + kSfbCol + 4, smem_desc(sfb_tile(s) + kScaleAtomBytes, 0, 128, kLayoutNone));
                }
#pragma unroll
                for (int k = 0; k < BK / 32; k++) {
                    const uint64_t da = smem_desc(a_tile(s) + 32 * k, 16, 1024, kLayoutSwizzle128);
                    const uint64_t db = smem_desc(b_tile(s) + 32 * k, 16, 1024, kLayoutSwizzle128);
                    const uint32_t idesc = (uint32_t)(256 >> 3) << 17 | 1u << 23 | (uint32_t)(256 >> 4) << 24 |
                                           (uint32_t)k << 4 | (uint32_t)k << 29;
                    tcgen05_mma_mxf8_pair(tmem, da, db, idesc, tmem + kSfaCol, tmem + kSfbCol, (kt | k) != 0);
                }
                tcgen05_commit_pair(empty_bar(s));
            }
            tcgen05_commit_pair(tmem_full_bar);
        }
    } else {
        mbar_wait(tmem_full_bar, 0, abort_flag, 256);
        tcgen05_fence_after();
        const int quad = warp % 4;
        const int row = m0 + quad * 32 + lane;
        const bool vec_ok = (ldy % 8 == 0) && (((uintptr_t)Y & 15u) == 0);
#pragma unroll 1
        for (int c = 0; c < kAccCols / 32; c++) {
            uint32_t r[32];
            tcgen05_ld_32x32b_x32(tmem + ((uint32_t)(quad * 32) << 16) + c * 32, r);
            tcgen05_wait_ld();
            const int col = n0 + c * 32;
            if (row >= M || col >= N || *abort_flag) continue;
            store_chunk(r, Y, ldy, row, col, N, out_bf16, vec_ok);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                           // the peer may still signal our barriers until here
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------
// Two-CTA kernel with the weight decode fused in: the B operand stays in its packed
// 4-bit form in HBM and in the shared-memory stages (64 bytes of codes per row and
// k-step, loaded by TMA with the 64-byte swizzle, plus the 256-byte id atom); four
// decode warps per CTA expand each stage's codes through the dialect byte tables into a
// small ring of operand buffers in the 128-byte-swizzled K-major layout the MMA reads;
// a proxy fence and an mbarrier hand each buffer to the MMA issuer of the leader CTA.
// A arrives as operand bytes (from the quantizer or the decode kernel) exactly as in
// gemm_tc2_kernel.  Freed resources come back through tcgen05.commit to both CTAs.
// ---------------------------------------------------------------------------
constexpr int kStagesF = 6;           // raw stages: A tile + packed B codes + ids + scale atoms
constexpr int kDecBufs = 4;           // decoded-B operand buffers
constexpr int kCodeTile = 128 * 64;   // 8 KiB: 128 rows x 64 bytes of codes
constexpr int kDecodeGroups = 4;
constexpr int kDecodeWarps = 4 * kDecodeGroups;
constexpr int kFusedThreads = 32 * (2 + kDecodeWarps + 4);   // warp 0 TMA, warp 1 MMA, the decode warps, 4 epilogue warps
struct FusedSmem {
    static constexpr int a = 0;
    static constexpr int codes = a + kStagesF * kHalfTile;
    static constexpr int dec = codes + kStagesF * kCodeTile;
    static constexpr int sfa = dec + kDecBufs * kHalfTile;
    static constexpr int sfb = sfa + kStagesF * kScaleAtomBytes;
    static constexpr int ids = sfb + kStagesF * 2 * kScaleAtomBytes;
    static constexpr int bars = ids + kStagesF * kIdAtomBytes;
    static constexpr int words = bars + 256;
    static constexpr int luts = words + 64;
    static constexpr int total = luts + 128 + 1024 /* alignment slack */;
};

// One lane of a converged warp (the same lane every time).  Loops that issue TMA / tcgen05
// instructions run with the whole warp converged and only predicate the instruction on this,
// so that addresses and descriptors stay in uniform registers instead of being moved per instruction.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kFusedThreads, 1)
gemm_tc2f_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapCodes,
                 const __grid_constant__ CUtensorMap mapSfA, const __grid_constant__ CUtensorMap mapSfB,
                 const uint8_t *__restrict__ idsB, int M, int N, int K, int row_tiles_a, int row_tiles_b,
                 void *__restrict__ Y, int64_t ldy, int out_bf16) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto a_tile = [&](int s) { return base + FusedSmem::a + (uint32_t)s * kHalfTile; };
    auto code_tile = [&](int s) { return base + FusedSmem::codes + (uint32_t)s * kCodeTile; };
    auto dec_tile = [&](int d) { return base + FusedSmem::dec + (uint32_t)d * kHalfTile; };
    auto sfa_tile = [&](int s) { return base + FusedSmem::sfa + (uint32_t)s * kScaleAtomBytes; };
    auto sfb_tile = [&](int s) { return base + FusedSmem::sfb + (uint32_t)s * 2 * kScaleAtomBytes; };
    auto id_tile = [&](int s) { return base + FusedSmem::ids + (uint32_t)s * kIdAtomBytes; };
    const uint32_t bars = base + FusedSmem::bars;
    auto full_bar = [&](int s) { return bars + 8u * s; };                         // leader: A + scales of both CTAs
    auto empty_bar = [&](int s) { return bars + 8u * (kStagesF + s); };           // both: stage s consumed
    auto raw_bar = [&](int s) { return bars + 8u * (2 * kStagesF + s); };         // local: codes + ids landed
    auto dec_full_bar = [&](int d) { return bars + 8u * (3 * kStagesF + d); };    // leader: buffer d decoded in both CTAs
    auto dec_empty_bar = [&](int d) { return bars + 8u * (3 * kStagesF + kDecBufs + d); };   // both: buffer d consumed
    const uint32_t tmem_full_bar = bars + 8u * (3 * kStagesF + 2 * kDecBufs);
    volatile uint32_t *const shared_words = (volatile uint32_t *)(base_ptr + FusedSmem::words);
    volatile uint32_t *const tmem_slot = shared_words;
    volatile uint32_t *const abort_flag = shared_words + 1;
    uint32_t *const luts = (uint32_t *)(base_ptr + FusedSmem::luts);              // e4m3_lo[16], e4m3_hi[16]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x / 2;
    const int m0 = pair * 256 + (int)rank * 128;
    const int n0 = blockIdx.y * 256;
    const int k_tiles = (K + BK - 1) / BK;
    constexpr int kAccCols = 256, kSfaCol = 256, kSfbCol = 260, kTmemCols = 512;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStagesF; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(raw_bar(s), 1);
        }
        for (int d = 0; d < kDecBufs; d++) {
            mbar_init(dec_full_bar(d), 2);                        // one arrival per CTA of the pair
            mbar_init(dec_empty_bar(d), 1);
        }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32) {
        luts[threadIdx.x] = threadIdx.x < 16 ? c_tables.e4m3_lo[threadIdx.x] : c_tables.e4m3_hi[threadIdx.x - 16];
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void *)tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ---- TMA producer (whole warp converged, one elected lane issues) ----
        constexpr uint32_t tx_pair = 2u * (kHalfTile + 3u * kScaleAtomBytes);
        const int my_row_tile = blockIdx.y * 2 + (int)rank;                       // this CTA's 128 rows of B
        const bool have_ids = my_row_tile < row_tiles_b;
        int s = 0;
        uint32_t ph = 1;
        for (int kt = 0; kt < k_tiles; kt++) {
            mbar_wait(empty_bar(s), ph, abort_flag);
            if (*abort_flag) break;
            const uint32_t fb = map_to_cta(full_bar(s), 0);
            if (elect_one()) {
                mbar_expect_tx(raw_bar(s), kCodeTile + (have_ids ? kIdAtomBytes : 0));
                tma_load_2d(code_tile(s), &mapCodes, kt * (BK / 2), n0 + (int)rank * 128, raw_bar(s));
                if (have_ids)
                    bulk_load(id_tile(s), idsB + ((int64_t)kt * row_tiles_b + my_row_tile) * kIdAtomBytes, kIdAtomBytes,
                              raw_bar(s));
                if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
                tma_load_2d_pair(a_tile(s), &mapA, kt * BK, m0, fb);
                tma_load_2d_pair(sfa_tile(s), &mapSfA, 0, kt * row_tiles_a + pair * 2 + (int)rank, fb);
                tma_load_2d_pair(sfb_tile(s), &mapSfB, 0, kt * row_tiles_b + blockIdx.y * 2, fb);
            }
            __syncwarp();
            if (++s == kStagesF) { s = 0; ph ^= 1u; }
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---- MMA issuer (leader CTA; whole warp converged, one elected lane issues) ----
            // Everything that does not depend on the k-step is computed once: descriptor high words,
            // the four instruction descriptors (one per scale byte), TMEM addresses.
            const uint32_t hi_op = desc_hi(1024, kLayoutSwizzle128), hi_sf = desc_hi(128, kLayoutNone);
            const uint32_t lo_a0 = (a_tile(0) >> 4) | 1u << 16, lo_b0 = (dec_tile(0) >> 4) | 1u << 16;
            const uint32_t lo_sfa0 = sfa_tile(0) >> 4, lo_sfb0 = sfb_tile(0) >> 4;
            const uint32_t idesc0 = (uint32_t)(256 >> 3) << 17 | 1u << 23 | (uint32_t)(256 >> 4) << 24;
            const uint32_t t_sfa = tmem + kSfaCol, t_sfb = tmem + kSfbCol;
            int s = 0, d = 0;
            uint32_t ph_s = 0, ph_d = 0;
            for (int kt = 0; kt < k_tiles; kt++) {
                mbar_wait(full_bar(s), ph_s, abort_flag);
                mbar_wait(dec_full_bar(d), ph_d, abort_flag);
                if (*abort_flag) break;
                tcgen05_fence_after();
                const uint32_t lo_sfa = lo_sfa0 + (uint32_t)s * (kScaleAtomBytes >> 4);
                const uint32_t lo_sfb = lo_sfb0 + (uint32_t)s * (2 * kScaleAtomBytes >> 4);
                const uint32_t lo_a = lo_a0 + (uint32_t)s * (kHalfTile >> 4), lo_b = lo_b0 + (uint32_t)d * (kHalfTile >> 4);
                if (elect_one()) {
                    tcgen05_cp_pair(t_sfa, desc_join(lo_sfa, hi_sf));
                    tcgen05_cp_pair(t_sfb, desc_join(lo_sfb, hi_sf));
                    tcgen05_cp_pair(t_sfb + 4, desc_join(lo_sfb + (kScaleAtomBytes >> 4), hi_sf));
#pragma unroll
                    for (int k = 0; k < BK / 32; k++)
                        tcgen05_mma_mxf8_pair(tmem, desc_join(lo_a + 2 * k, hi_op), desc_join(lo_b + 2 * k, hi_op),
                                              idesc0 | (uint32_t)k << 4 | (uint32_t)k << 29, t_sfa, t_sfb, (kt | k) != 0);
                    tcgen05_commit_pair(empty_bar(s));
                    tcgen05_commit_pair(dec_empty_bar(d));
                }
                __syncwarp();
                if (++s == kStagesF) { s = 0; ph_s ^= 1u; }
                if (++d == kDecBufs) { d = 0; ph_d ^= 1u; }
            }
            if (elect_one()) tcgen05_commit_pair(tmem_full_bar);
            __syncwarp();
        }
    } else if (warp < 2 + kDecodeWarps) {
        // ---- decode warps, in kDecodeGroups groups of four: group g takes the k-steps kt = g (mod groups),
        // so that consecutive k-steps are decoded concurrently; thread j of a group expands row j ----
        const int group = (warp - 2) / 4;
        const int j = ((warp - 2) % 4) * 32 + lane;
        const uint32_t swz64 = (uint32_t)(j >> 1) & 3u, swz128 = (uint32_t)j & 7u;
        const uint32_t dec_full_leader = map_to_cta(dec_full_bar(0), 0);
        for (int kt = group; kt < k_tiles; kt += kDecodeGroups) {
            const int s = kt % kStagesF, d = kt % kDecBufs;
            mbar_wait(raw_bar(s), (kt / kStagesF) & 1, abort_flag);
            mbar_wait(dec_empty_bar(d), ((kt / kDecBufs) & 1) ^ 1, abort_flag);
            if (*abort_flag) break;
            const uint8_t *codes = base_ptr + FusedSmem::codes + s * kCodeTile + j * 64;
            const uint32_t ids16 = *(const uint16_t *)(base_ptr + FusedSmem::ids + s * kIdAtomBytes + j * 2);
            uint8_t *dst = base_ptr + FusedSmem::dec + d * kHalfTile + j * 128;
            uint4 w[4];
#pragma unroll
            for (int c = 0; c < 4; c++) w[c] = *(const uint4 *)(codes + 16 * (c ^ swz64));
#pragma unroll
            for (int c = 0; c < 4; c++) {
                const uint32_t id = (ids16 >> (4 * c)) & 15u;
                const uint32_t lo = luts[id], hi = luts[16 + id];
                uint32_t o[8];
                decode_word(w[c].x, lo, hi, o[0], o[1]);
                decode_word(w[c].y, lo, hi, o[2], o[3]);
                decode_word(w[c].z, lo, hi, o[4], o[5]);
                decode_word(w[c].w, lo, hi, o[6], o[7]);
                *(uint4 *)(dst + 16 * ((2 * c) ^ swz128)) = make_uint4(o[0], o[1], o[2], o[3]);
                *(uint4 *)(dst + 16 * ((2 * c + 1) ^ swz128)) = make_uint4(o[4], o[5], o[6], o[7]);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
            asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory"); // the four warps of this group are done
            if (j == 0) mbar_arrive_cluster(dec_full_leader + 8u * d);
        }
    } else {
        // ---- epilogue ----
        mbar_wait(tmem_full_bar, 0, abort_flag, 256);
        tcgen05_fence_after();
        const int quad = warp % 4;
        const int row = m0 + quad * 32 + lane;
        const bool vec_ok = (ldy % 8 == 0) && (((uintptr_t)Y & 15u) == 0);
#pragma unroll 1
        for (int c = 0; c < kAccCols / 32; c++) {
            uint32_t r[32];
            tcgen05_ld_32x32b_x32(tmem + ((uint32_t)(quad * 32) << 16) + c * 32, r);
            tcgen05_wait_ld();
            const int col = n0 + c * 32;
            if (row >= M || col >= N || *abort_flag) continue;
            store_chunk(r, Y, ldy, row, col, N, out_bf16, vec_ok);
        }
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols)
                     : "memory");
    }
}

// ---- host side --------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// Tensor map of a [rows][K] byte matrix, box = 128 bytes of K x box_rows rows, 128-byte swizzle, zero fill.
inline bool make_operand_map(CUtensorMap *map, const uint8_t *ptr, int64_t rows, int64_t K, int box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)K};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void *)ptr, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

// Tensor map over the scale atoms: [atoms][128 x uint32], box = `atoms_per_box` whole atoms, zero fill.
inline bool make_scale_map(CUtensorMap *map, const uint8_t *ptr, int64_t atoms, int atoms_per_box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {128, (cuuint64_t)atoms};
    cuuint64_t strides[1] = {(cuuint64_t)kScaleAtomBytes};
    cuuint32_t box[2] = {128, (cuuint32_t)atoms_per_box};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT32, 2, (void *)ptr, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

template <int MODE = 0>
inline cudaError_t launch_pair(const uint8_t *a8, const uint8_t *sfa, int64_t M, const uint8_t *b8, const uint8_t *sfb,
                               int64_t N, int64_t K, void *Y, bool out_bf16, int64_t ldy, cudaStream_t st) {
    CUtensorMap mapA, mapB, mapSfA, mapSfB;
    const int64_t rta = row_tiles(M), rtb = row_tiles(N), kg = k_groups(K);
    if (!make_operand_map(&mapA, a8, M, K, 128) || !make_operand_map(&mapB, b8, N, K, 128) ||
        !make_scale_map(&mapSfA, sfa, rta * kg, 1) || !make_scale_map(&mapSfB, sfb, rtb * kg, 2))
        return cudaErrorInvalidValue;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc2_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem2Bytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((unsigned)(2 * ((M + 255) / 256)), (unsigned)((N + 255) / 256));
    gemm_tc2_kernel<MODE><<<grid, kThreads, kSmem2Bytes, st>>>(mapA, mapB, mapSfA, mapSfB, (int)M, (int)N, (int)K, (int)rta,
                                                        (int)rtb, Y, ldy, out_bf16 ? 1 : 0);
    return cudaGetLastError();
}

// Tensor map of packed codes [rows][K/2] bytes: box = 64 bytes x 128 rows, 64-byte swizzle, zero fill.
inline bool make_codes_map(CUtensorMap *map, const uint8_t *ptr, int64_t rows, int64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)(K / 2), (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)(K / 2)};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void *)ptr, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
           CUDA_SUCCESS;
}

// A as operand bytes + scale atoms, B as a packed operand (codes, ids, scale atoms).
inline cudaError_t launch_fused(const uint8_t *a8, const uint8_t *sfa, int64_t M, const QView &B, int64_t K, void *Y,
                                bool out_bf16, int64_t ldy, cudaStream_t st) {
    CUtensorMap mapA, mapCodes, mapSfA, mapSfB;
    const int64_t N = B.rows, rta = row_tiles(M), rtb = row_tiles(N), kg = k_groups(K);
    if (!make_operand_map(&mapA, a8, M, K, 128) || !make_codes_map(&mapCodes, B.codes, N, K) ||
        !make_scale_map(&mapSfA, sfa, rta * kg, 1) || !make_scale_map(&mapSfB, B.scales, rtb * kg, 2))
        return cudaErrorInvalidValue;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc2f_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FusedSmem::total);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((unsigned)(2 * ((M + 255) / 256)), (unsigned)((N + 255) / 256));
    gemm_tc2f_kernel<<<grid, kFusedThreads, FusedSmem::total, st>>>(mapA, mapCodes, mapSfA, mapSfB, B.ids, (int)M, (int)N,
                                                                   (int)K, (int)rta, (int)rtb, Y, ldy, out_bf16 ? 1 : 0);
    return cudaGetLastError();
}

template <int BN, int MODE = 0>
inline cudaError_t launch(const uint8_t *a8, const uint8_t *sfa, int64_t M, const uint8_t *b8, const uint8_t *sfb,
                          int64_t N, int64_t K, void *Y, bool out_bf16, int64_t ldy, cudaStream_t st) {
    using C = Config<BN>;
    CUtensorMap mapA, mapB;
    if (!make_operand_map(&mapA, a8, M, K, BM) || !make_operand_map(&mapB, b8, N, K, BN)) return cudaErrorInvalidValue;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    dim3 grid((unsigned)((N + BN - 1) / BN), (unsigned)((M + BM - 1) / BM));
    gemm_tc_kernel<BN, MODE><<<grid, kThreads, C::kSmemBytes, st>>>(mapA, mapB, sfa, sfb, (int)M, (int)N, (int)K,
                                                             (int)row_tiles(M), (int)row_tiles(N), Y, ldy, out_bf16 ? 1 : 0);
    return cudaGetLastError();
}

}  // namespace tc

inline bool tc_supported(int64_t M, int64_t N, int64_t K) {
    return K % kBlock == 0 && M >= 1 && N >= 1 && M < (1ll << 31) && N < (1ll << 31) && K < (1ll << 31);
}
inline size_t tc_operand_bytes(int64_t rows, int64_t K) { return ((size_t)rows * (size_t)K + 255) & ~(size_t)255; }
inline size_t tc_gemm_workspace(int64_t M, int64_t N, int64_t K) { return tc_operand_bytes(M, K) + tc_operand_bytes(N, K); }

inline int tc_variant() {
    static int variant = -1;
    if (variant < 0) { const char *v = getenv("BD_TC_VARIANT"); variant = v ? atoi(v) : 0; }
    return variant;
}
// true: B is consumed in packed form by the fused kernel (no decoded copy of B needed)
inline bool tc_fused_b() { return tc_variant() == 0; }

inline cudaError_t tc_gemm_fused(const uint8_t *a8, const uint8_t *sfa, int64_t M, const QView &B, int64_t K, void *Y,
                                 bool out_bf16, int64_t ldy, cudaStream_t st) {
    return tc::launch_fused(a8, sfa, M, B, K, Y, out_bf16, ldy, st);
}

inline cudaError_t tc_gemm(const uint8_t *a8, const uint8_t *sfa, int64_t M, const uint8_t *b8, const uint8_t *sfb,
                           int64_t N, int64_t K, void *Y, bool out_bf16, int64_t ldy, cudaStream_t st) {
    const int variant = tc_variant();
    if (variant == 1) return tc::launch<128>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 3) return tc::launch<256, 1>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 4) return tc::launch<256, 2>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 28) return tc::launch_pair<12>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 20) return tc::launch_pair<0>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 11) return tc::launch<256, 29>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 10) return cudaSuccess;                        // experiment: decode kernels only
    if (variant == 7) return tc::launch<256, 5>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 8) return tc::launch<256, 13>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 9) return tc::launch<256, 9>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 5) return tc::launch<128, 1>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (variant == 6) return tc::launch<128, 2>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    if (N > 128) return tc::launch<256>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
    return tc::launch<128>(a8, sfa, M, b8, sfb, N, K, Y, out_bf16, ldy, st);
}

}  // namespace bd
