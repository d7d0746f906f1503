// Tensor-core GEMM for sm_100a: Y[M,N] = A[M,K] * dq(B)[N,K]^T with one power-of-two
// scale per 32 elements of K on each operand (Sec. 3.3: the products of a block share
// the exponent sum eA + eB; the block-scaled MMA applies it in hardware).
//
// A arrives as a plain [M][K] byte matrix holding the E4M3 encoding of 0.5 * value
// (exact: every DialectFP4 magnitude has at most four significant bits) plus its scale
// atoms; B stays packed (4-bit codes, 4-bit ids, scale atoms) all the way into shared
// memory and is expanded there by decode warps.
//
// One persistent kernel.  A cluster of two CTAs on neighbouring SMs owns 256 x 256
// output tiles and computes them with tcgen05.mma.cta_group::2 (kind::mxf8f6f4
// .block_scale, K = 32 per instruction = one block, UE8M0 scales in TMEM, fp32
// accumulator in TMEM).  Per CTA:
//   warp 0        TMA producer: A tile (128-byte swizzle), packed B codes (64-byte swizzle),
//                 id atom, scale atoms, into a ring of stages;
//   warp 1        MMA issuer (leader CTA only): tcgen05.cp scales -> TMEM, four MMAs per stage;
//   warps 2..17   decode, in four groups that take alternate k-steps: codes -> operand bytes
//                 through the dialect byte tables, written in the 128-byte-swizzled K-major
//                 layout, handed over with a proxy fence and an mbarrier;
//   warps 18..25  epilogue (two warps per TMEM lane quadrant, each taking half of the columns).
// Loops that issue TMA / tcgen05 instructions run with the whole warp converged and one
// elected lane, so that addresses and descriptors stay in uniform registers.
//
// Scheduling: the grid is one cluster per SM pair; cluster c takes tiles c, c + C, ... in an
// order that keeps the clusters running at the same time on neighbouring rows of the same
// weight columns.  The ring of stages runs across tile boundaries, so the loads of the next
// tile are in flight while the epilogue drains the accumulator.
//
// Epilogue: each of the eight warps moves its 32 rows x 128 columns through a private
// 4 KiB staging buffer (tcgen05.ld -> convert -> st.shared, 128-byte swizzle) and writes it
// with TMA tensor stores, 128 bytes per row, so the accumulator is released after about a
// microsecond and the global writes are full lines.
//
// Every wait is bounded: when the limit is reached the kernel records
// kStatusTimeout, stops waiting everywhere, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "bd_common.cuh"
#include "ptx_sm100.cuh"
#include "quantize.cuh"

namespace bd {
namespace tc {

constexpr int BK = 128;                 // bytes of K per stage = one 128-byte swizzle row = 4 blocks
constexpr int kStages = 5;              // raw stages: A tile + packed B codes + ids + scale atoms
constexpr int kDecBufs = 4;             // decoded-B operand buffers
constexpr int kHalfTile = 128 * BK;     // 16 KiB: 128 rows of operand bytes
constexpr int kCodeTile = 128 * 64;     // 8 KiB: 128 rows x 64 bytes of codes
#ifndef BD_TC_DECODE_GROUPS
#define BD_TC_DECODE_GROUPS 4
#endif
constexpr int kDecodeWarps = 16;
constexpr int kDecodeGroups = BD_TC_DECODE_GROUPS;   // groups take alternate k-steps; 16 / groups warps share one k-step
constexpr int kEpilogueWarp0 = 2 + kDecodeWarps;
constexpr int kEpilogueWarps = 8;        // two per TMEM lane quadrant, each taking half of the columns
constexpr int kThreads = 32 * (kEpilogueWarp0 + kEpilogueWarps);
constexpr int kStageOutBytes = 32 * 128;  // per epilogue warp: 32 rows x 128 bytes

struct Smem {
    static constexpr int a = 0;
    static constexpr int codes = a + kStages * kHalfTile;
    static constexpr int dec = codes + kStages * kCodeTile;
    static constexpr int sfa = dec + kDecBufs * kHalfTile;
    static constexpr int sfb = sfa + kStages * kScaleAtomBytes;
    static constexpr int ids = sfb + kStages * 2 * kScaleAtomBytes;
    static constexpr int bars = ids + kStages * kIdAtomBytes;
    static constexpr int words = bars + 256;
    static constexpr int luts = words + 256;
    static constexpr int out = ((luts + 128 + 1023) / 1024) * 1024;          // epilogue staging, 1 KiB aligned
    static constexpr int total = out + kEpilogueWarps * kStageOutBytes + 1024 /* alignment slack */;
};
static_assert((3 * kStages + 2 * kDecBufs + 2) * 8 <= 256, "barrier area too small");
static_assert(Smem::total <= 227 * 1024, "shared memory budget");

// Work of one launch, identical for every cluster: cluster c takes tiles c, c + clusters, ...
struct Schedule {
    int m_pairs, n_tiles, k_tiles;      // tile grid (256 x 256 tiles, k-steps of 128)
    int clusters;
};
struct Item {
    int tile;
};
__device__ __forceinline__ bool get_item(const Schedule &sc, int c, int i, Item &it) {
    it.tile = i * sc.clusters + c;
    return it.tile < sc.m_pairs * sc.n_tiles;
}

#ifdef BD_TC_PROFILE
__device__ unsigned long long g_prof[32];
#define PROF_DECL long long prof_t0 = 0; long long prof_acc[4] = {0, 0, 0, 0}; (void)prof_t0; (void)prof_acc
#define PROF_T0 prof_t0 = clock64()
#define PROF_ADD(i) prof_acc[i] += clock64() - prof_t0
#define PROF_OUT(i, slot) if (cluster == 0 && rank == 0 && lane == 0) atomicAdd(&g_prof[slot], (unsigned long long)prof_acc[i])
#else
#define PROF_DECL
#define PROF_T0
#define PROF_ADD(i)
#define PROF_OUT(i, slot)
#endif

// ---- PTX wrappers (cluster pair) ---------------------------------------------
__device__ __forceinline__ void tcgen05_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tcgen05_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
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
// One lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load whose completion is counted on a barrier of the pair's leader CTA.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Arrives on the barrier at the same offset in both CTAs once all earlier MMAs have completed.
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
__device__ __forceinline__ void tcgen05_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tcgen05_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (64 bit), split in two words so that the issuing warp only
// adds to the low one: low = (addr >> 4) | (leading byte offset >> 4) << 16,
// high = (stride byte offset >> 4) | descriptor version 1 << 14 | swizzle mode << 29.
constexpr uint32_t kLayoutSwizzle128 = 2, kLayoutNone = 0;
__device__ __forceinline__ uint32_t desc_hi(uint32_t sbo_bytes, uint32_t layout) {
    return ((sbo_bytes >> 4) & 0x3fffu) | 1u << 14 | layout << 29;
}
__device__ __forceinline__ uint64_t desc_join(uint32_t lo, uint32_t hi) {
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
    return d;
}

// Store one 16-column chunk of an accumulator row (fp32 registers) as fp32 or bf16.
__device__ __forceinline__ void store_chunk(const uint32_t (&r)[16], void *Y, int64_t ldy, int row, int col, int N,
                                            int out_bf16, bool vec_ok) {
    if (out_bf16) {
        __nv_bfloat16 *dst = (__nv_bfloat16 *)Y + (int64_t)row * ldy + col;
        if (vec_ok && col + 16 <= N) {
#pragma unroll
            for (int i = 0; i < 2; i++) {
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
            for (int i = 0; i < 16 && col + i < N; i++) dst[i] = __float2bfloat16_rn(__uint_as_float(r[i]));
        }
    } else {
        float *dst = (float *)Y + (int64_t)row * ldy + col;
        if (vec_ok && col + 16 <= N) {
#pragma unroll
            for (int i = 0; i < 4; i++) ((uint4 *)dst)[i] = make_uint4(r[4 * i], r[4 * i + 1], r[4 * i + 2], r[4 * i + 3]);
        } else {
            for (int i = 0; i < 16 && col + i < N; i++) dst[i] = __uint_as_float(r[i]);
        }
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapCodes,
                 const __grid_constant__ CUtensorMap mapSfA, const __grid_constant__ CUtensorMap mapSfB,
                 const uint8_t *__restrict__ idsB, const Schedule sc, int M, int N, int row_tiles_a, int row_tiles_b,
                 void *__restrict__ Y, int64_t ldy, int out_bf16, const __grid_constant__ CUtensorMap mapY, int use_tma_store) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto a_tile = [&](int s) { return base + Smem::a + (uint32_t)s * kHalfTile; };
    auto code_tile = [&](int s) { return base + Smem::codes + (uint32_t)s * kCodeTile; };
    auto dec_tile = [&](int d) { return base + Smem::dec + (uint32_t)d * kHalfTile; };
    auto sfa_tile = [&](int s) { return base + Smem::sfa + (uint32_t)s * kScaleAtomBytes; };
    auto sfb_tile = [&](int s) { return base + Smem::sfb + (uint32_t)s * 2 * kScaleAtomBytes; };
    auto id_tile = [&](int s) { return base + Smem::ids + (uint32_t)s * kIdAtomBytes; };
    const uint32_t bars = base + Smem::bars;
    auto full_bar = [&](int s) { return bars + 8u * s; };                         // leader: A + scales of both CTAs
    auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };            // both: stage s consumed
    auto raw_bar = [&](int s) { return bars + 8u * (2 * kStages + s); };          // local: codes + ids landed
    auto dec_full_bar = [&](int d) { return bars + 8u * (3 * kStages + d); };     // leader: buffer d decoded in both CTAs
    auto dec_empty_bar = [&](int d) { return bars + 8u * (3 * kStages + kDecBufs + d); };   // both: buffer d consumed
    const uint32_t tmem_full_bar = bars + 8u * (3 * kStages + 2 * kDecBufs);      // both: accumulator complete
    const uint32_t tmem_empty_bar = tmem_full_bar + 8u;                           // leader: accumulator read out
    volatile uint32_t *const shared_words = (volatile uint32_t *)(base_ptr + Smem::words);
    volatile uint32_t *const tmem_slot = shared_words;
    volatile uint32_t *const abort_flag = shared_words + 1;
    uint32_t *const luts = (uint32_t *)(base_ptr + Smem::luts);                   // e4m3_lo[16], e4m3_hi[16]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();
    const int cluster = blockIdx.x / 2;
    constexpr int kSfaCol = 256, kSfbCol = 260, kTmemCols = 512;

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < kStages; s++) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(raw_bar(s), 1);
        }
        for (int d = 0; d < kDecBufs; d++) {
            mbar_init(dec_full_bar(d), 2);                        // one arrival per CTA of the pair
            mbar_init(dec_empty_bar(d), 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 2 * kEpilogueWarps);            // the epilogue warps of both CTAs
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32)
        luts[threadIdx.x] = threadIdx.x < 16 ? c_tables.e4m3_lo[threadIdx.x] : c_tables.e4m3_hi[threadIdx.x - 16];
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
    // programmatic dependent launch: everything above overlapped the tail of the previous kernel in the
    // stream; its results (the operand bytes the quantizer wrote) are read only after this point
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        // ---- TMA producer (whole warp converged, one elected lane issues) ----
        constexpr uint32_t tx_pair = 2u * (kHalfTile + 3u * kScaleAtomBytes);
        int s = 0;
        uint32_t ph = 1;
        Item it;
        PROF_DECL;
        for (int i = 0; get_item(sc, cluster, i, it); i++) {
            const int m_pair = it.tile % sc.m_pairs, n_tile = it.tile / sc.m_pairs;
            const int m0 = m_pair * 256 + (int)rank * 128, n0 = n_tile * 256 + (int)rank * 128;
            const int my_row_tile = n_tile * 2 + (int)rank;                       // this CTA's 128 rows of B
            const bool have_ids = my_row_tile < row_tiles_b;
            for (int kt = 0; kt < sc.k_tiles; kt++) {
                PROF_T0;
                mbar_wait(empty_bar(s), ph, abort_flag);
                PROF_ADD(0);
#ifdef BD_TC_PROFILE
                if (cluster == 0 && rank == 0 && lane == 0 && (i > 0 || kt >= kStages))
                    atomicAdd(&g_prof[18], (unsigned long long)((uint32_t)clock64() - shared_words[8 + s]));
#endif
                if (*abort_flag) break;
                const uint32_t fb = map_to_cta(full_bar(s), 0);
                if (elect_one()) {
#ifdef BD_TC_PROFILE
                    shared_words[2 + s] = (uint32_t)clock64();
#endif
                    mbar_expect_tx(raw_bar(s), kCodeTile + (have_ids ? kIdAtomBytes : 0));
                    tma_load_2d(code_tile(s), &mapCodes, kt * (BK / 2), n0, raw_bar(s));
                    if (have_ids)
                        bulk_load(id_tile(s), idsB + ((int64_t)kt * row_tiles_b + my_row_tile) * kIdAtomBytes,
                                  kIdAtomBytes, raw_bar(s));
                    if (rank == 0) mbar_expect_tx(full_bar(s), tx_pair);
                    tma_load_2d_pair(a_tile(s), &mapA, kt * BK, m0, fb);
                    tma_load_2d_pair(sfa_tile(s), &mapSfA, 0, kt * row_tiles_a + m_pair * 2 + (int)rank, fb);
                    tma_load_2d_pair(sfb_tile(s), &mapSfB, 0, kt * row_tiles_b + n_tile * 2, fb);
                }
                __syncwarp();
                if (++s == kStages) { s = 0; ph ^= 1u; }
            }
            if (*abort_flag) break;
        }
        PROF_OUT(0, 0);
    } else if (warp == 1) {
        if (rank == 0) {
            // ---- MMA issuer (leader CTA; whole warp converged, one elected lane issues) ----
            const uint32_t hi_op = desc_hi(1024, kLayoutSwizzle128), hi_sf = desc_hi(128, kLayoutNone);
            const uint32_t lo_a0 = (a_tile(0) >> 4) | 1u << 16, lo_b0 = (dec_tile(0) >> 4) | 1u << 16;
            const uint32_t lo_sfa0 = sfa_tile(0) >> 4, lo_sfb0 = sfb_tile(0) >> 4;
            // block-scaled E4M3 x E4M3 (formats 0), both K-major, UE8M0 scales (bit 23), N >> 3 at bit 17,
            // M >> 4 at bit 24 (M = 256 across the pair); the scale byte selectors go to bits 4 (B) and 29 (A)
            const uint32_t idesc0 = (uint32_t)(256 >> 3) << 17 | 1u << 23 | (uint32_t)(256 >> 4) << 24;
            const uint32_t t_sfa = tmem + kSfaCol, t_sfb = tmem + kSfbCol;
            int s = 0, d = 0;
            uint32_t ph_s = 0, ph_d = 0;
            bool ready = false;
            Item it;
            PROF_DECL;
#ifdef BD_TC_PROFILE
            const long long prof_start = clock64();
#endif
            for (int i = 0; get_item(sc, cluster, i, it); i++) {
                PROF_T0;
                if (i > 0) mbar_wait(tmem_empty_bar, (uint32_t)(i - 1) & 1u, abort_flag);
                PROF_ADD(2);
                tcgen05_fence_after();
                for (int kt = 0; kt < sc.k_tiles; kt++) {
                    if (!ready) {
                        // slow path: the probe at the end of the previous k-step found a barrier open
                        PROF_T0;
                        mbar_wait(full_bar(s), ph_s, abort_flag);
                        PROF_ADD(0);
                        PROF_T0;
                        mbar_wait(dec_full_bar(d), ph_d, abort_flag);
                        PROF_ADD(1);
                        if (*abort_flag) break;
                    }
#ifdef BD_TC_PROFILE
                    const uint32_t prof_iss0 = (uint32_t)clock64();
                    if (cluster == 0 && lane == 0) atomicAdd(&g_prof[16], (unsigned long long)(prof_iss0 - shared_words[16 + d]));
#endif
                    tcgen05_fence_after();
                    const uint32_t lo_sfa = lo_sfa0 + (uint32_t)s * (kScaleAtomBytes >> 4);
                    const uint32_t lo_sfb = lo_sfb0 + (uint32_t)s * (2 * kScaleAtomBytes >> 4);
                    const uint32_t lo_a = lo_a0 + (uint32_t)s * (kHalfTile >> 4), lo_b = lo_b0 + (uint32_t)d * (kHalfTile >> 4);
                    const uint32_t first = kt == 0 ? 0u : 1u;
                    if (elect_one()) {
                        tcgen05_cp_pair(t_sfa, desc_join(lo_sfa, hi_sf));
                        tcgen05_cp_pair(t_sfb, desc_join(lo_sfb, hi_sf));
                        tcgen05_cp_pair(t_sfb + 4, desc_join(lo_sfb + (kScaleAtomBytes >> 4), hi_sf));
#pragma unroll
                        for (int k = 0; k < BK / 32; k++)
                            tcgen05_mma_mxf8_pair(tmem, desc_join(lo_a + 2 * k, hi_op), desc_join(lo_b + 2 * k, hi_op),
                                                  idesc0 | (uint32_t)k << 4 | (uint32_t)k << 29, t_sfa, t_sfb,
                                                  k == 0 ? first : 1u);
                        tcgen05_commit_pair(empty_bar(s));
                        tcgen05_commit_pair(dec_empty_bar(d));
#ifdef BD_TC_PROFILE
                        shared_words[8 + s] = (uint32_t)clock64();
                        if (cluster == 0) atomicAdd(&g_prof[17], (unsigned long long)((uint32_t)clock64() - prof_iss0));
#endif
                    }
                    __syncwarp();
                    if (++s == kStages) { s = 0; ph_s ^= 1u; }
                    if (++d == kDecBufs) { d = 0; ph_d ^= 1u; }
                    // probe the next k-step's barriers now (the rings run across tiles): their shared-memory
                    // round trip overlaps the instruction issue above instead of opening the next iteration
                    const bool full_ok = mbar_test_wait(full_bar(s), ph_s), dec_ok = mbar_test_wait(dec_full_bar(d), ph_d);
                    ready = full_ok && dec_ok;
#ifdef BD_TC_PROFILE
                    if (cluster == 0 && lane == 0 && ready) atomicAdd(&g_prof[19], 1ull);
#endif
                }
                if (elect_one()) tcgen05_commit_pair(tmem_full_bar);
                __syncwarp();
                if (*abort_flag) break;
            }
            PROF_OUT(0, 1);
            PROF_OUT(1, 2);
            PROF_OUT(2, 3);
#ifdef BD_TC_PROFILE
            prof_acc[3] = clock64() - prof_start;
#endif
            PROF_OUT(3, 4);
        }
    } else if (warp < kEpilogueWarp0) {
        // ---- decode warps, in groups of four: group g takes this CTA's k-steps g, g + groups, ...;
        // thread j of a group expands row j of the CTA's 128 B rows ----
        constexpr int kGroupWarps = kDecodeWarps / kDecodeGroups, kGroupThreads = 32 * kGroupWarps;
        constexpr int kPerRow = kGroupThreads / 128, kBlocksPerThread = 4 / kPerRow;   // threads per B row, blocks per thread
        const int group = (warp - 2) / kGroupWarps;
        const int tg = ((warp - 2) % kGroupWarps) * 32 + lane;
        const int j = tg / kPerRow, c0 = (tg % kPerRow) * kBlocksPerThread;
        const uint32_t swz64 = (uint32_t)(j >> 1) & 3u, swz128 = (uint32_t)j & 7u;
        const uint32_t dec_full_leader = map_to_cta(dec_full_bar(0), 0);
        int total_k = 0;
        {
            Item it;
            for (int i = 0; get_item(sc, cluster, i, it); i++) total_k += sc.k_tiles;
        }
        PROF_DECL;
#ifdef BD_TC_PROFILE
        const long long prof_start = clock64();
#endif
        for (int g = group; g < total_k; g += kDecodeGroups) {
            const int s = g % kStages, d = g % kDecBufs;
            PROF_T0;
            mbar_wait(raw_bar(s), (uint32_t)(g / kStages) & 1u, abort_flag);
            PROF_ADD(0);
#ifdef BD_TC_PROFILE
            if (cluster == 0 && rank == 0 && tg == 0) {
                atomicAdd(&g_prof[14], (unsigned long long)((uint32_t)clock64() - shared_words[2 + s]));
                atomicAdd(&g_prof[15], 1ull);
            }
#endif
            PROF_T0;
            mbar_wait(dec_empty_bar(d), ((uint32_t)(g / kDecBufs) & 1u) ^ 1u, abort_flag);
            PROF_ADD(1);
            if (*abort_flag) break;
#ifdef BD_TC_PROFILE
            const long long pt0 = clock64();
#endif
            const uint8_t *codes = base_ptr + Smem::codes + s * kCodeTile + j * 64;
            const uint32_t ids16 = *(const uint16_t *)(base_ptr + Smem::ids + s * kIdAtomBytes + (j % 32) * 8 + (j / 32) * 2);
            uint8_t *dst = base_ptr + Smem::dec + d * kHalfTile + j * 128;
            uint4 w[kBlocksPerThread];
#pragma unroll
            for (int i = 0; i < kBlocksPerThread; i++) w[i] = *(const uint4 *)(codes + 16 * ((c0 + i) ^ swz64));
#pragma unroll
            for (int i = 0; i < kBlocksPerThread; i++) {
                const int c = c0 + i;
                const uint32_t id = (ids16 >> (4 * c)) & 15u;
                const uint32_t lo = luts[id], hi = luts[16 + id];
                uint32_t o[8];
                decode_word(w[i].x, lo, hi, o[0], o[1]);
                decode_word(w[i].y, lo, hi, o[2], o[3]);
                decode_word(w[i].z, lo, hi, o[4], o[5]);
                decode_word(w[i].w, lo, hi, o[6], o[7]);
                *(uint4 *)(dst + 16 * ((2 * c) ^ swz128)) = make_uint4(o[0], o[1], o[2], o[3]);
                *(uint4 *)(dst + 16 * ((2 * c + 1) ^ swz128)) = make_uint4(o[4], o[5], o[6], o[7]);
            }
#ifdef BD_TC_PROFILE
            const long long pt1 = clock64();
#endif
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
#ifdef BD_TC_PROFILE
            const long long pt2 = clock64();
#endif
            asm volatile("bar.sync %0, %1;" ::"r"(1 + group), "n"(kGroupThreads) : "memory");   // this group's warps are done
#ifdef BD_TC_PROFILE
            const long long pt3 = clock64();
#endif
            if (tg == 0) mbar_arrive_cluster(dec_full_leader + 8u * d);
#ifdef BD_TC_PROFILE
            if (tg == 0) shared_words[16 + d] = (uint32_t)pt3;
            if (cluster == 0 && rank == 0 && tg == 0) {
                atomicAdd(&g_prof[10], (unsigned long long)(pt1 - pt0));
                atomicAdd(&g_prof[11], (unsigned long long)(pt2 - pt1));
                atomicAdd(&g_prof[12], (unsigned long long)(pt3 - pt2));
                atomicAdd(&g_prof[13], (unsigned long long)(clock64() - pt3));
            }
#endif
        }
        if (warp == 2) {
            PROF_OUT(0, 5);
            PROF_OUT(1, 6);
#ifdef BD_TC_PROFILE
            prof_acc[2] = clock64() - prof_start;
#endif
            PROF_OUT(2, 7);
        }
    } else {
        // ---- epilogue: warp w reads TMEM lanes 32 * (w % 4) .. + 31 of this CTA's accumulator half,
        // columns [128 * half, + 128) ----
        const int quad = warp % 4, ew = warp - kEpilogueWarp0, half = ew / 4;
        const bool vec_ok = (ldy % 8 == 0) && (((uintptr_t)Y & 15u) == 0);
        const uint32_t tmem_empty_leader = map_to_cta(tmem_empty_bar, 0);
        const int local_row = quad * 32 + lane;
        const uint32_t stage_out = base + Smem::out + (uint32_t)ew * kStageOutBytes;
        uint8_t *const stage_ptr = base_ptr + Smem::out + ew * kStageOutBytes + lane * 128;
        const uint32_t lane_swz = (uint32_t)lane & 7u;
        const int cols_per_pass = out_bf16 ? 64 : 32;                 // 128 bytes per row and pass
        Item it;
        PROF_DECL;
        for (int i = 0; get_item(sc, cluster, i, it); i++) {
            const int m_pair = it.tile % sc.m_pairs, n_tile = it.tile / sc.m_pairs;
            const int row0 = m_pair * 256 + (int)rank * 128 + quad * 32;
            const int n0 = n_tile * 256 + half * 128;
            PROF_T0;
            mbar_wait(tmem_full_bar, (uint32_t)i & 1u, abort_flag, 256);
            PROF_ADD(0);
            PROF_T0;
            tcgen05_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(quad * 32) << 16) + half * 128;
            if (use_tma_store) {
                for (int pass = 0; pass < 128 / cols_per_pass; pass++) {
                    // the previous pass's tensor store must have finished reading the staging buffer
                    if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();
                    if (out_bf16) {
                        // 64 columns: four loads in flight, one wait
                        uint32_t r[4][16];
#pragma unroll
                        for (int c = 0; c < 4; c++) tcgen05_ld_32x32b_x16(t_base + pass * 64 + c * 16, r[c]);
                        tcgen05_wait_ld();
#pragma unroll
                        for (int c = 0; c < 4; c++) {                 // 16 columns -> 32 bytes = chunks 2c, 2c + 1
                            uint32_t p[8];
#pragma unroll
                            for (int j = 0; j < 8; j++) {
                                __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[c][2 * j]), __uint_as_float(r[c][2 * j + 1]));
                                p[j] = *(uint32_t *)&h;
                            }
                            *(uint4 *)(stage_ptr + 16 * ((2 * c) ^ lane_swz)) = make_uint4(p[0], p[1], p[2], p[3]);
                            *(uint4 *)(stage_ptr + 16 * ((2 * c + 1) ^ lane_swz)) = make_uint4(p[4], p[5], p[6], p[7]);
                        }
                    } else {
                        uint32_t r[2][16];
#pragma unroll
                        for (int c = 0; c < 2; c++) tcgen05_ld_32x32b_x16(t_base + pass * 32 + c * 16, r[c]);
                        tcgen05_wait_ld();
#pragma unroll
                        for (int c = 0; c < 2; c++)                   // 16 columns -> 64 bytes = chunks 4c .. 4c + 3
#pragma unroll
                            for (int q = 0; q < 4; q++)
                                *(uint4 *)(stage_ptr + 16 * ((4 * c + q) ^ lane_swz)) =
                                    make_uint4(r[c][4 * q], r[c][4 * q + 1], r[c][4 * q + 2], r[c][4 * q + 3]);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && !*abort_flag) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&mapY), "r"(n0 + pass * cols_per_pass), "r"(row0), "r"(stage_out) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            } else {
                const int row = row0 + lane;
#pragma unroll 1
                for (int c = 0; c < 8; c++) {
                    uint32_t r[16];
                    tcgen05_ld_32x32b_x16(t_base + c * 16, r);
                    tcgen05_wait_ld();
                    const int col = n0 + c * 16;
                    if (row < M && col < N && !*abort_flag) store_chunk(r, Y, ldy, row, col, N, out_bf16, vec_ok);
                }
            }
            // accumulator read out: the MMA issuer may start the next tile
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
            PROF_ADD(1);
        }
        if (ew == 0) {
            PROF_OUT(0, 8);
            PROF_OUT(1, 9);
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");    // staging buffers must outlive the stores
        __syncwarp();
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

inline bool make_map_2d(CUtensorMap *map, CUtensorMapDataType type, const void *ptr, uint64_t inner, uint64_t outer,
                        uint64_t stride_bytes, uint32_t box_inner, uint32_t box_outer, CUtensorMapSwizzle swizzle) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {stride_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t elem[2] = {1, 1};
    return fn(map, type, 2, (void *)ptr, dims, strides, box, elem, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Number of two-CTA clusters of this kernel that can be resident at once (cached).
inline int max_resident_clusters() {
    static int cached = 0;
    if (cached) return cached;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 128);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Smem::total;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_pair_kernel, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, 0);
        n = sms / 2;
    }
    cached = n;
    return cached;
}

// A as operand bytes + scale atoms, B as a packed operand.
inline cudaError_t launch(const uint8_t *a8, const uint8_t *sfa, int64_t M, const QView &B, int64_t K, void *Y,
                          bool out_bf16, int64_t ldy, cudaStream_t st) {
    CUtensorMap mapA, mapCodes, mapSfA, mapSfB, mapY;
    const int64_t N = B.rows, rta = row_tiles(M), rtb = row_tiles(N), kg = k_groups(K);
    if (!make_map_2d(&mapA, CU_TENSOR_MAP_DATA_TYPE_UINT8, a8, K, M, K, BK, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mapCodes, CU_TENSOR_MAP_DATA_TYPE_UINT8, B.codes, K / 2, N, K / 2, 64, 128, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map_2d(&mapSfA, CU_TENSOR_MAP_DATA_TYPE_UINT32, sfa, 128, rta * kg, kScaleAtomBytes, 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&mapSfB, CU_TENSOR_MAP_DATA_TYPE_UINT32, B.scales, 128, rtb * kg, kScaleAtomBytes, 128, 2, CU_TENSOR_MAP_SWIZZLE_NONE))
        return cudaErrorInvalidValue;
    // output through TMA tensor stores (32 rows x 128 bytes per box) when Y is 16-byte aligned with a
    // row pitch that is a multiple of 16 bytes; otherwise plain stores
    const int esz = out_bf16 ? 2 : 4;
    int use_tma_store = (((uintptr_t)Y & 15u) == 0 && (ldy * esz) % 16 == 0) ? 1 : 0;
    if (use_tma_store &&
        !make_map_2d(&mapY, out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Y, N, M,
                     (uint64_t)ldy * esz, 128 / esz, 32, CU_TENSOR_MAP_SWIZZLE_128B))
        use_tma_store = 0;
    if (!use_tma_store) mapY = mapA;                                   // unused, but must be a valid object
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(gemm_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::total);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    Schedule sc;
    sc.m_pairs = (int)((M + 255) / 256);
    sc.n_tiles = (int)((N + 255) / 256);
    sc.k_tiles = (int)((K + BK - 1) / BK);
    const int tiles = sc.m_pairs * sc.n_tiles;
    const int resident = max_resident_clusters();
    sc.clusters = tiles < resident ? tiles : resident;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * sc.clusters);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Smem::total;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the previous kernel drains
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_pair_kernel, mapA, mapCodes, mapSfA, mapSfB, (const uint8_t *)B.ids, sc, (int)M,
                              (int)N, (int)rta, (int)rtb, Y, ldy, out_bf16 ? 1 : 0, mapY, use_tma_store);
}

}  // namespace tc

inline bool tc_supported(int64_t M, int64_t N, int64_t K) {
    return K % kBlock == 0 && M >= 1 && N >= 1 && M < (1ll << 31) && N < (1ll << 31) && K < (1ll << 31);
}
inline size_t tc_operand_bytes(int64_t rows, int64_t K) { return ((size_t)rows * (size_t)K + 255) & ~(size_t)255; }
// workspace of the tensor-core path given A as a packed operand: its operand bytes
inline size_t tc_gemm_workspace(int64_t M, int64_t, int64_t K) { return tc_operand_bytes(M, K); }

}  // namespace bd
