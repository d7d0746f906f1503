// Tensor-core GEMM for sm_100a with the decoded weights in tensor memory:
//   Y[M,N] = X[M,K] * dq(W)[N,K]^T,  computed as D = dq(W) * X^T tile by tile
// (Sec. 3.3: one power-of-two scale per 32 elements of K on each operand, applied by the
// block-scaled MMA).
//
// Why this orientation: tcgen05.mma takes its A operand either from shared memory or from tensor
// memory.  With the weights as A, the decode warps expand the packed codes straight into TMEM
// (tcgen05.st) and the MMA reads them from there, so the only shared-memory traffic of the main
// loop is the activation tile (written by TMA, read once by the MMA) and the packed codes.  In the
// shared-memory variant of this kernel every byte the decode warps loaded or stored through the
// load/store unit took its turn on the same shared-memory pipe the MMA reads its operands through.
//
// A cluster of two CTAs owns a tile of 256 weight rows x 256 tokens:
//   tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale, M = 256 (128 weight rows per CTA, A in
//   TMEM), N = 256 tokens (each CTA holds 128 of them in shared memory, K-major, 128-byte swizzle),
//   K = 32 per instruction = one block; UE8M0 scales in TMEM; fp32 accumulator in TMEM with
//   lanes = weight rows and columns = tokens.
// Warps of a CTA:
//   0        TMA producer: activation tile and the scale atoms of both operands (ring of stages);
//   1        MMA issuer (leader CTA);
//   2        TMA producer: packed codes and ids of this CTA's 128 weight rows (its own ring);
//   3..14    decode, three groups of four warps taking k-steps in turn; thread = weight row =
//            TMEM lane: codes -> 128 operand bytes -> tcgen05.st into one of the A buffers;
//   15..22   epilogue: TMEM -> registers (the accumulator is handed back here) -> transposed
//            staging tile -> TMA tensor store.
// Measured on B200: the main loop issues one k-step (256 x 256 x 128) per ~540 cycles, 95 % of the
// tensor pipe's 512; under the 1000 W cap the clock, not the schedule, then sets the time, so what
// is left to gain is energy per k-step (mostly the activation bytes that cross from L2).
// Every wait is bounded (see mbar_wait): on a timeout the kernel records kStatusTimeout, stops
// waiting everywhere, frees its TMEM and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdlib.h>

#include "bd_common.cuh"
#include "ptx_sm100.cuh"
#include "quantize.cuh"

namespace bd {
namespace tc {

constexpr int BK = 128;                      // bytes of K per k-step = one 128-byte swizzle row = 4 blocks
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

constexpr int kXStages = 6;                  // activation tile + scale atoms
constexpr int kCodeStages = 6;               // packed codes + ids
constexpr int kABufs = 5;                    // decoded weight k-steps in tensor memory (32 columns each)
constexpr int kXTile = 128 * BK;             // 16 KiB: 128 tokens x 128 operand bytes
constexpr int kCodeTile = 128 * 64;          // 8 KiB: 128 weight rows x 64 bytes of codes
constexpr int kDecodeWarp0 = 3, kDecodeGroups = 3, kDecodeWarps = 4 * kDecodeGroups;
constexpr int kEpilogueWarp0 = kDecodeWarp0 + kDecodeWarps, kEpilogueWarps = 8;
constexpr int kThreads = 32 * (kEpilogueWarp0 + kEpilogueWarps);
constexpr int kStageOut = 2048;            // one staging buffer: 32 tokens x 32 bf16 or 16 tokens x 32 fp32
constexpr int kStageBufs = 2;               // per epilogue warp, used in turn: a store reads one while the next is filled

// tensor-memory columns
constexpr int kColD = 0;                     // accumulator: 256 token columns
constexpr int kColA = 256;                   // kABufs x 32 columns of operand bytes
constexpr int kColSfW = kColA + 32 * kABufs; // weight scales (4 columns)
constexpr int kColSfX = kColSfW + 4;         // activation scales (8 columns)
static_assert(kColSfX + 8 <= 512, "tensor memory budget");

struct Smem {
    static constexpr int x = 0;
    static constexpr int codes = x + kXStages * kXTile;
    static constexpr int sfw = codes + kCodeStages * kCodeTile;
    static constexpr int sfx = sfw + kXStages * kScaleAtomBytes;
    static constexpr int ids = sfx + kXStages * 2 * kScaleAtomBytes;
    static constexpr int bars = ids + kCodeStages * kIdAtomBytes;
    static constexpr int words = bars + 512;
    static constexpr int luts = words + 64;
    static constexpr int qtab = luts + 128;                      // the quantizer's tables (requantising epilogue)
    static constexpr int idx = qtab + (int)sizeof(SmemTables);   // dialect ids traded between the four warps of an epilogue half
    static constexpr int out = ((idx + 512 + 1023) / 1024) * 1024;
    static constexpr int total = out + kEpilogueWarps * kStageBufs * kStageOut + 1024 /* alignment slack */;
};
static_assert((2 * kXStages + 2 * kCodeStages + 2 * kABufs + 2) * 8 <= 512, "barrier area too small");
static_assert(Smem::total <= 227 * 1024, "shared memory budget");

// Work items of a launch, identical for every cluster: cluster c takes items c, c + clusters, ...
// Tiles are numbered with the token tile running fastest (token tile = tile % t_tiles, weight-row pair =
// tile / t_tiles), so the clusters that run at the same time share weight rows and differ in their tokens.
// Items [0, split_from) are whole tiles of 256 tokens.  Each later tile is cut into `parts` items of
// `part_tokens` tokens: two of 128, which lets a last, sparsely filled wave of tiles spread over twice as
// many clusters; or, when the whole problem has at most 128 tokens, one item of just those tokens (rounded up
// to the MMA's step of 16), so that a decode-sized call does not pay for 256 columns per k-step.
// A call of at most 128 tokens has few tiles (one per 256 weight rows); with k_splits > 1 each is further cut
// along K into k_splits items of k_per k-steps, so that more SMs pull weights; their fp32 partial sums go to
// scratch memory and a second kernel (splitk_reduce_kernel) adds them in split order.
struct Schedule {
    int w_pairs, t_tiles, k_tiles, clusters, split_from, parts, part_tokens, k_splits, k_per;
};
struct Tile {
    int w_pair;      // weight rows [256 * w_pair, + 256)
    int t_start;     // first token
    int tokens;      // the N of the MMA: 256, or the schedule's part_tokens
    int k_begin, k_end, split;   // k-steps of this item; which split of its tile it is
};
__device__ __forceinline__ bool next_tile(const Schedule &sc, int c, int i, Tile &t) {
    int item = i * sc.clusters + c;
    const int tiles = sc.w_pairs * sc.t_tiles;
    t.k_begin = 0;
    t.k_end = sc.k_tiles;
    t.split = 0;
    if (sc.k_splits > 1) {                                        // every tile is k_splits consecutive items
        t.split = item % sc.k_splits;
        item /= sc.k_splits;
        t.k_begin = t.split * sc.k_per;
        t.k_end = min(sc.k_tiles, t.k_begin + sc.k_per);
    }
    int tile = item, part = 0;
    t.tokens = 256;
    if (item >= sc.split_from) {
        tile = sc.split_from + (item - sc.split_from) / sc.parts;
        part = (item - sc.split_from) % sc.parts;
        t.tokens = sc.part_tokens;
    }
    t.w_pair = tile / sc.t_tiles;
    t.t_start = (tile % sc.t_tiles) * 256 + part * 128;
    return tile < tiles;
}

// Split K: at most kMaxKSplits items per tile, each of at least kMinKPerSplit k-steps, for calls of at most
// kSplitMaxTokens tokens.  (An earlier version let the last warp to arrive add the partial sums inside the
// GEMM; a second kernel whose threads each own four outputs is faster at every size: 16.7 vs 21.1 us at 16
// tokens, K = 11008, N = 4096.)
constexpr int kMaxKSplits = 4, kMinKPerSplit = 8, kSplitMaxTokens = 128;

__device__ __forceinline__ void tcgen05_mma_mxf8_pair_atmem(uint32_t d, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc,
                                                            uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], [%1], %2, %3, [%5], [%6], p;\n\t}"
        ::"r"(d), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb) : "memory");
}
__device__ __forceinline__ void tcgen05_st_32x32b_x8(uint32_t taddr, const uint32_t (&r)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tcgen05_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// bf16 epilogue of one warp: its 32 * CHUNKS token columns go to registers first, packed as bf16 pairs of
// neighbouring tokens (16 * CHUNKS registers), so the accumulator is free again after CHUNKS TMEM round trips;
// then, 32 tokens at a time, lanes 2m and 2m + 1 trade halves so that each writes one 32-bit word of two
// neighbouring output columns (the even lane the row of token t, the odd lane the row of token t + 1) into one
// of the warp's two staging buffers, which a TMA tensor store writes out as 32 rows x 32 columns while the
// other buffer is filled.
template <int CHUNKS, typename Release, typename StagingFree>
__device__ __forceinline__ void epilogue_bf16(uint32_t t_base, uint8_t *stage_ptr, uint32_t stage_out, const CUtensorMap *mapY,
                                              int n0, int t0, int lane, volatile uint32_t *abort_flag, Release release_accumulator,
                                              StagingFree staging_free) {
    uint32_t p[16 * CHUNKS];
#pragma unroll
    for (int c = 0; c < CHUNKS; c++) {
        uint32_t r[32];
        tcgen05_ld_32x32b_x32(t_base + c * 32, r);
        tcgen05_wait_ld();
#pragma unroll
        for (int q = 0; q < 16; q++) {
            __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(r[2 * q]), __uint_as_float(r[2 * q + 1]));
            p[c * 16 + q] = *(uint32_t *)&h;                      // tokens 32 c + 2 q and + 1 of my column
        }
    }
    release_accumulator();
#pragma unroll
    for (int pass = 0; pass < CHUNKS; pass++) {                   // 32 tokens per pass
        const uint32_t sb = staging_free();                       // offset of the staging buffer whose turn it is
        // the exchanges of eight registers go out together, so that their latencies overlap
#pragma unroll
        for (int q0 = 0; q0 < 16; q0 += 8) {
            uint32_t other[8];
#pragma unroll
            for (int u = 0; u < 8; u++) other[u] = __shfl_xor_sync(0xffffffffu, p[16 * pass + q0 + u], 1);
#pragma unroll
            for (int u = 0; u < 8; u++) {
                const int q = q0 + u;
                const uint32_t mine = p[16 * pass + q];
                const uint32_t word = (lane & 1) ? prmt_b32(other[u], mine, 0x7632u)   // (col - 1, col) of token t + 1
                                                 : prmt_b32(mine, other[u], 0x5410u);  // (col, col + 1) of token t
                *(uint32_t *)(stage_ptr + sb + (2 * q + (lane & 1)) * 64 + (lane >> 1) * 4) = word;
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0 && !*abort_flag) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(mapY), "r"(n0), "r"(t0 + pass * 32), "r"(stage_out + sb) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
    }
}

// REQUANT: the instantiation whose epilogue requantises the result (its quantizer arithmetic costs registers that the
// plain instantiation keeps for the main loop).
template <bool REQUANT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
gemm_wtmem_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapXpart,
                  const __grid_constant__ CUtensorMap mapCodes,
                  const __grid_constant__ CUtensorMap mapSfW, const __grid_constant__ CUtensorMap mapSfX,
                  const uint8_t *__restrict__ idsW, const Schedule sc, int M, int N, int row_tiles_x, int row_tiles_w,
                  void *__restrict__ Y, int64_t ldy, int out_bf16, const __grid_constant__ CUtensorMap mapY, int use_tma_store,
                  float *__restrict__ partials, const QView yq) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *const base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto x_tile = [&](int s) { return base + Smem::x + (uint32_t)s * kXTile; };
    auto code_tile = [&](int s) { return base + Smem::codes + (uint32_t)s * kCodeTile; };
    auto sfw_tile = [&](int s) { return base + Smem::sfw + (uint32_t)s * kScaleAtomBytes; };
    auto sfx_tile = [&](int s) { return base + Smem::sfx + (uint32_t)s * 2 * kScaleAtomBytes; };
    auto id_tile = [&](int s) { return base + Smem::ids + (uint32_t)s * kIdAtomBytes; };
    const uint32_t bars = base + Smem::bars;
    auto x_full = [&](int s) { return bars + 8u * s; };                                   // leader: tile + scales of both CTAs
    auto x_empty = [&](int s) { return bars + 8u * (kXStages + s); };                     // both: stage consumed by the MMA
    auto c_full = [&](int s) { return bars + 8u * (2 * kXStages + s); };                  // local: codes + ids landed
    auto c_empty = [&](int s) { return bars + 8u * (2 * kXStages + kCodeStages + s); };   // local: codes read by the decode group
    auto a_full = [&](int b) { return bars + 8u * (2 * kXStages + 2 * kCodeStages + b); };            // leader: buffer written in both CTAs
    auto a_empty = [&](int b) { return bars + 8u * (2 * kXStages + 2 * kCodeStages + kABufs + b); };  // both: buffer consumed
    const uint32_t tmem_full_bar = bars + 8u * (2 * kXStages + 2 * kCodeStages + 2 * kABufs);         // both: accumulator complete
    const uint32_t tmem_empty_bar = tmem_full_bar + 8u;                                               // leader: accumulator read out
    volatile uint32_t *const shared_words = (volatile uint32_t *)(base_ptr + Smem::words);
    volatile uint32_t *const tmem_slot = shared_words;
    volatile uint32_t *const abort_flag = shared_words + 1;
    uint32_t *const luts = (uint32_t *)(base_ptr + Smem::luts);                         // e4m3_lo[16], e4m3_hi[16]

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = cluster_ctarank();
    const int cluster = blockIdx.x / 2;

    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        abort_flag[1] = 0;                                        // set once the previous kernel has completed
        abort_flag[2] = g_debug_spin_limit ? g_debug_spin_limit : kSpinLimit;
        for (int s = 0; s < kXStages; s++) {
            mbar_init(x_full(s), 1);
            mbar_init(x_empty(s), 1);
        }
        for (int s = 0; s < kCodeStages; s++) {
            mbar_init(c_full(s), 1);
            mbar_init(c_empty(s), 4);                             // one arrival per warp of the decode group
        }
        for (int b = 0; b < kABufs; b++) {
            mbar_init(a_full(b), 2);                              // one arrival per CTA of the pair
            mbar_init(a_empty(b), 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 2 * kEpilogueWarps);          // the epilogue warps of both CTAs
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x < 32)
        luts[threadIdx.x] = threadIdx.x < 16 ? c_tables.e4m3_lo[threadIdx.x] : c_tables.e4m3_hi[threadIdx.x - 16];
    SmemTables &qtab = *(SmemTables *)(base_ptr + Smem::qtab);
    if (REQUANT) load_tables(qtab);                               // (ends with __syncthreads())
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(smem_u32((const void *)tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                           // both CTAs: barriers initialised, TMEM allocated
    tcgen05_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ---- TMA producer of the activation tile and the scale atoms (one elected lane issues) ----
        // Programmatic dependent launch: the previous kernel of the stream is the one that wrote the activation
        // operand, and only this warp reads it, so only this warp waits for that kernel.  The weights are older
        // than that kernel (it started its own dependents only after everything before it had completed), so
        // the code producer and the decode warps fill their rings while it drains.  Every store of this kernel
        // follows an MMA that consumed a tile loaded here, i.e. follows the wait.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        if (lane == 0) abort_flag[1] = 1;                         // from here on every bounded wait counts its polls
        int s = 0;
        uint32_t ph = 1;
        const uint32_t x_full_leader = map_to_cta(x_full(0), 0);
        Tile t;
        for (int i = 0; next_tile(sc, cluster, i, t); i++) {
            // each CTA holds half of the item's tokens; smaller items load their rows through a tensor map of their own
            const int per_cta = t.tokens / 2, t0 = t.t_start + (int)rank * per_cta;
            const CUtensorMap *map = t.tokens == 256 ? &mapX : &mapXpart;
            const uint32_t tx_pair = 2u * ((uint32_t)per_cta * BK + 3u * kScaleAtomBytes);
            for (int kt = t.k_begin; kt < t.k_end; kt++) {
                if (!mbar_wait(x_empty(s), ph, abort_flag)) break;
                const uint32_t fb = x_full_leader + 8u * (uint32_t)s;
                if (elect_one()) {
                    if (rank == 0) mbar_expect_tx(x_full(s), tx_pair);
                    tma_load_2d_pair(x_tile(s), map, kt * BK, t0, fb);
                    tma_load_2d_pair(sfw_tile(s), &mapSfW, 0, kt * row_tiles_w + t.w_pair * 2 + (int)rank, fb);
                    // two scale atoms = 256 tokens from the item's first token (a smaller item uses the first)
                    tma_load_2d_pair(sfx_tile(s), &mapSfX, 0, kt * row_tiles_x + t.t_start / 128, fb);
                }
                __syncwarp();
                if (++s == kXStages) { s = 0; ph ^= 1u; }
            }
            if (*abort_flag) break;
        }
    } else if (warp == 2) {
        // ---- TMA producer of this CTA's packed codes and ids ----
        int s = 0;
        uint32_t ph = 1;
        const bool skip_first = g_debug_skip_first_code_stage != 0;   // test hook: see bd_debug_fault
        Tile t;
        for (int i = 0; next_tile(sc, cluster, i, t); i++) {
            const int w0 = t.w_pair * 256 + (int)rank * 128;
            const int my_row_tile = t.w_pair * 2 + (int)rank;
            const bool have_ids = my_row_tile < row_tiles_w;
            for (int kt = t.k_begin; kt < t.k_end; kt++) {
                if (!mbar_wait(c_empty(s), ph, abort_flag)) break;
                if (elect_one() && !(skip_first && i == 0 && kt == t.k_begin)) {
                    mbar_expect_tx(c_full(s), kCodeTile + (have_ids ? kIdAtomBytes : 0));
                    tma_load_2d(code_tile(s), &mapCodes, kt * (BK / 2), w0, c_full(s));
                    if (have_ids)
                        bulk_load(id_tile(s), idsW + ((int64_t)kt * row_tiles_w + my_row_tile) * kIdAtomBytes, kIdAtomBytes,
                                  c_full(s));
                }
                __syncwarp();
                if (++s == kCodeStages) { s = 0; ph ^= 1u; }
            }
            if (*abort_flag) break;
        }
    } else if (warp == 1) {
        if (rank == 0) {
            // ---- MMA issuer (leader CTA; whole warp converged, one elected lane issues) ----
            const uint32_t hi_op = desc_hi(1024, kLayoutSwizzle128), hi_sf = desc_hi(128, kLayoutNone);
            const uint32_t lo_x0 = (x_tile(0) >> 4) | 1u << 16;
            const uint32_t lo_sfw0 = sfw_tile(0) >> 4, lo_sfx0 = sfx_tile(0) >> 4;
            // block-scaled E4M3 x E4M3 (formats 0), B K-major, UE8M0 scales (bit 23), N >> 3 at bit 17 (256 tokens),
            // M >> 4 at bit 24 (256 weight rows across the pair); scale byte selectors at bits 4 (B) and 29 (A)
            const uint32_t idesc_m = 1u << 23 | (uint32_t)(256 >> 4) << 24;
            const uint32_t t_d = tmem + kColD, t_sfw = tmem + kColSfW, t_sfx = tmem + kColSfX;
            int s = 0, b = 0;
            uint32_t ph_s = 0, ph_b = 0;
            bool ready = false;
            Tile t;
            for (int i = 0; next_tile(sc, cluster, i, t); i++) {
                const uint32_t idesc0 = idesc_m | (uint32_t)(t.tokens >> 3) << 17;
                if (i > 0) mbar_wait(tmem_empty_bar, (uint32_t)(i - 1) & 1u, abort_flag);
                tcgen05_fence_after();
                for (int kt = t.k_begin; kt < t.k_end; kt++) {
                    if (!ready) {
                        // slow path: the probe at the end of the previous k-step found a barrier open
                        if (!mbar_wait(x_full(s), ph_s, abort_flag) || !mbar_wait(a_full(b), ph_b, abort_flag)) break;
                    }
                    tcgen05_fence_after();
                    const uint32_t lo_sfw = lo_sfw0 + (uint32_t)s * (kScaleAtomBytes >> 4);
                    const uint32_t lo_sfx = lo_sfx0 + (uint32_t)s * (2 * kScaleAtomBytes >> 4);
                    const uint32_t lo_x = lo_x0 + (uint32_t)s * (kXTile >> 4);
                    const uint32_t t_a = tmem + kColA + 32u * (uint32_t)b;
                    const uint32_t first = kt == t.k_begin ? 0u : 1u;
                    if (elect_one()) {
                        tcgen05_cp_pair(t_sfw, desc_join(lo_sfw, hi_sf));
                        tcgen05_cp_pair(t_sfx, desc_join(lo_sfx, hi_sf));
                        tcgen05_cp_pair(t_sfx + 4, desc_join(lo_sfx + (kScaleAtomBytes >> 4), hi_sf));
#pragma unroll
                        for (int k = 0; k < BK / 32; k++)
                            tcgen05_mma_mxf8_pair_atmem(t_d, t_a + 8u * k, desc_join(lo_x + 2 * k, hi_op),
                                                        idesc0 | (uint32_t)k << 4 | (uint32_t)k << 29, t_sfw, t_sfx,
                                                        k == 0 ? first : 1u);
                        tcgen05_commit_pair(x_empty(s));
                        tcgen05_commit_pair(a_empty(b));
                    }
                    __syncwarp();
                    if (++s == kXStages) { s = 0; ph_s ^= 1u; }
                    if (++b == kABufs) { b = 0; ph_b ^= 1u; }
                    // probe the next k-step's barriers now (the rings run across tiles): the shared-memory
                    // round trip overlaps the instruction issue above instead of opening the next iteration
                    const bool x_ok = mbar_test_wait(x_full(s), ph_s), a_ok = mbar_test_wait(a_full(b), ph_b);
                    ready = x_ok && a_ok;
                }
                if (*abort_flag && elect_one()) {
                    // this CTA is aborting: tell the peer before its epilogue warps are woken by the commit below,
                    // so that they too skip their stores
                    asm volatile("st.shared::cluster.u32 [%0], %1;\n\tfence.acq_rel.cluster;"
                                 ::"r"(map_to_cta(smem_u32((const void *)abort_flag), 1)), "r"(1u) : "memory");
                }
                __syncwarp();
                if (elect_one()) tcgen05_commit_pair(tmem_full_bar);
                __syncwarp();
                if (*abort_flag) break;
            }
        }
    } else if (warp < kEpilogueWarp0) {
        // ---- decode warps: group g takes this CTA's k-steps g, g + groups, ... (counted across tiles);
        // a warp may only touch the TMEM lanes 32 * (warp % 4) .. + 31, so thread `lane` of warp w owns
        // weight row (and TMEM lane) j = 32 * (w % 4) + lane; the four warps of a group cover all 128 ----
        const int group = (warp - kDecodeWarp0) / 4, quad = warp % 4;
        const int j = quad * 32 + lane;
        const bool group_leader = (warp - kDecodeWarp0) % 4 == 0 && lane == 0;
        const uint32_t swz64 = (uint32_t)(j >> 1) & 3u;
        const uint32_t a_full_leader = map_to_cta(a_full(0), 0);
        const uint32_t t_row = tmem + ((uint32_t)(quad * 32) << 16) + kColA;
        int total_k = 0;
        {
            Tile t;
            for (int i = 0; next_tile(sc, cluster, i, t); i++) total_k += t.k_end - t.k_begin;
        }
        // ring positions of this group's k-step, kept by increments (the step, the number of groups, is smaller
        // than either ring): code stage s with the parity to wait for, operand buffer b likewise
        int s = group % kCodeStages, b = group % kABufs;
        uint32_t s_par = 0, b_par = 1;
        static_assert(kDecodeGroups <= kCodeStages && kDecodeGroups <= kABufs, "one wrap per step at most");
        // A warp whose wait ran out (or that saw the abort word) is `dead`: it stops waiting and working but keeps
        // meeting its group at the named barrier of every remaining k-step.  The four warps wait on the same
        // barriers, yet one may see the abort word where another still sees its barrier complete; a warp that left
        // the loop would then leave the other at the named barrier for good.
        bool dead = false;
        for (int g = group; g < total_k; g += kDecodeGroups) {
            uint4 w[4];
            uint32_t ids16 = 0;
            if (!dead) dead = !mbar_wait(c_full(s), s_par, abort_flag);
            if (!dead) {
                const uint8_t *codes = base_ptr + Smem::codes + s * kCodeTile + j * 64;
                ids16 = *(const uint16_t *)(base_ptr + Smem::ids + s * kIdAtomBytes + (j % 32) * 8 + (j / 32) * 2);
#pragma unroll
                for (int c = 0; c < 4; c++) w[c] = *(const uint4 *)(codes + 16 * (c ^ swz64));
                // the codes are in registers: hand the stage back to its producer
                __syncwarp();
                if (lane == 0) mbar_arrive_local(c_empty(s));
                dead = !mbar_wait(a_empty(b), b_par, abort_flag);
            }
            if (!dead) {
                tcgen05_fence_after();                            // the MMAs that read this buffer have completed
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    const uint32_t id = (ids16 >> (4 * c)) & 15u;
                    const uint32_t lo = luts[id], hi = luts[16 + id];
                    uint32_t o[8];
                    decode_word(w[c].x, lo, hi, o[0], o[1]);
                    decode_word(w[c].y, lo, hi, o[2], o[3]);
                    decode_word(w[c].z, lo, hi, o[4], o[5]);
                    decode_word(w[c].w, lo, hi, o[6], o[7]);
                    tcgen05_st_32x32b_x8(t_row + 32u * (uint32_t)b + 8u * (uint32_t)c, o);   // block c = columns 8c .. 8c + 7
                }
                tcgen05_wait_st();
                tcgen05_fence_before();
            }
            asm volatile("bar.sync %0, 128;" ::"r"(1 + group) : "memory");   // the four warps of this group are done
            if (group_leader && !dead) mbar_arrive_cluster(a_full_leader + 8u * b);
            s += kDecodeGroups;
            if (s >= kCodeStages) { s -= kCodeStages; s_par ^= 1u; }
            b += kDecodeGroups;
            if (b >= kABufs) { b -= kABufs; b_par ^= 1u; }
        }
    } else {
        // ---- epilogue: warp w reads the TMEM lanes 32 * (w % 4) .. + 31 (weight rows) of this CTA's
        // accumulator, token columns [128 * half, + 128), and writes them transposed: Y[token][weight row] ----
        const int quad = warp % 4, ew = warp - kEpilogueWarp0, half = ew / 4;
        const uint32_t tmem_empty_leader = map_to_cta(tmem_empty_bar, 0);
        const uint32_t stage_out = base + Smem::out + (uint32_t)ew * (kStageBufs * kStageOut);
        uint8_t *const stage_ptr = base_ptr + Smem::out + ew * (kStageBufs * kStageOut);
        // 4 KiB of staging per warp, two buffers: 32 tokens x 32 bf16 or 16 tokens x 32 fp32 per tensor store
        // accumulator read out (all of this warp's columns are in registers): the MMA issuer may start the next tile
        auto release_accumulator = [&]() {
            tcgen05_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(tmem_empty_leader);
        };
        // the two staging buffers take turns: before one is filled again, the tensor store issued two passes ago
        // (the one that read it) must have finished reading; the latest store may still be in flight
        uint32_t stage_turn = 0;
        auto staging_free = [&]() -> uint32_t {
            if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
            __syncwarp();
            stage_turn ^= 1u;
            return stage_turn * kStageOut;
        };
        Tile t;
        for (int i = 0; next_tile(sc, cluster, i, t); i++) {
            // token columns of this warp: the two warps of a quadrant share items of 128 tokens or more; a smaller
            // item goes to the first of them, rounded up to whole passes of 64 tokens (the columns past the item
            // hold stale sums of tokens that do not exist, and the stores clip them)
            const int cols = t.tokens >= 128 ? t.tokens / 2 : (half == 0 ? (t.tokens + 63) / 64 * 64 : 0);
            const int n0 = t.w_pair * 256 + (int)rank * 128 + quad * 32;    // this warp's 32 output columns
            const int t0 = t.t_start + half * cols;                         // and its first output row
            mbar_wait(tmem_full_bar, (uint32_t)i & 1u, abort_flag, 256);
            tcgen05_fence_after();
            const uint32_t t_base = tmem + ((uint32_t)(quad * 32) << 16) + kColD + half * cols;
            if (cols == 0) {
                release_accumulator();
            } else if (sc.k_splits > 1) {
                // split along K: this item's sums are partial.  Each warp writes its 32 weight rows x tokens to
                // partials[split][token][weight row]; the reduce kernel behind this launch adds the splits
                const int n = n0 + lane, np = sc.w_pairs * 256, toks = sc.part_tokens;
                const int tok0 = t.tokens >= 128 ? half * cols : 0;          // this warp's first token
                float *mine = partials + ((size_t)t.split * toks + tok0) * np + n;
#pragma unroll 1
                for (int c = 0; c * 16 < cols; c++) {
                    uint32_t r[16];
                    tcgen05_ld_32x32b_x16(t_base + c * 16, r);
                    tcgen05_wait_ld();
#pragma unroll
                    for (int q = 0; q < 16; q++)
                        if (tok0 + c * 16 + q < toks && !*abort_flag) __stcg(mine + (size_t)(c * 16 + q) * np, __uint_as_float(r[q]));
                }
                release_accumulator();
            } else if (REQUANT) {
                // Requantising epilogue (Sec. 3.3, last paragraph: the accumulated result is "requantized into 4-bit
                // DialectFP4 format for the next matrix multiplication").  The result row of a token is the next
                // product's operand row, cut into blocks of 32 along N; this warp's 32 weight rows are one such
                // block (number n0 / 32) of every token.  32 tokens per pass: each lane stores its row's fp32 sums
                // into a 32 x 32 staging tile (element (token q, row n) at q * 32 + (n ^ q): both the row-wise
                // stores and the token-wise loads touch 32 banks), then lane q owns token q's block and runs the
                // two-stage rule of Sec. 3.2 on it, exactly as the standalone quantizer does on fp32 sources.
                // Codes and scale bytes go out per lane; the four dialect ids of a token's four blocks (the four
                // warps of this epilogue half) share two bytes of the id atom, so they meet in shared memory and
                // the first warp stores them.
                uint32_t *const tile = (uint32_t *)stage_ptr;     // 4 KiB: both staging buffers of this warp
                const int b = n0 / kBlock, nb_out = (int)(yq.K / kBlock);
                const int atoms_rows = (int)row_tiles(yq.rows) * kRowTile, atoms_blocks = (int)k_groups(yq.K) * kBlocksPerAtom;
                for (int pass = 0; pass * 32 < cols; pass++) {
                    uint32_t r[32];
                    tcgen05_ld_32x32b_x32(t_base + pass * 32, r);
                    tcgen05_wait_ld();
                    if ((pass + 1) * 32 >= cols) release_accumulator();
                    __syncwarp();                                 // the previous pass's loads of the tile are done
#pragma unroll
                    for (int q = 0; q < 32; q++) tile[q * 32 + (lane ^ q)] = r[q];
                    __syncwarp();
                    uint32_t bits[32];
#pragma unroll
                    for (int k = 0; k < 32; k++) bits[k] = tile[lane * 32 + (k ^ lane)];
                    const int tok = t0 + pass * 32 + lane;
                    const bool valid = tok < M && b < nb_out;
                    BlockResult res;
                    res.id = 0; res.scale = 0;
                    if (valid) {
                        bool nonfinite;
                        uint32_t unused[8];
                        quantize_two_stage_f32<false>(bits, qtab, res, unused, nonfinite);
                        if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
                        if (!*abort_flag)
                            *(uint4 *)(yq.codes + (int64_t)tok * yq.ldc + (int64_t)b * 16) =
                                make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
                    }
                    // scale bytes and ids of the atoms' padding (tokens past M, blocks past N / 32) are written as zeros
                    const bool in_atoms = tok < atoms_rows && b < atoms_blocks;
                    if (in_atoms && !*abort_flag) yq.scales[scale_offset(yq.rows, tok, b)] = (uint8_t)res.scale;
                    uint8_t *const trade = base_ptr + Smem::idx + (half * 2 + (pass & 1)) * 128;
                    trade[quad * 32 + lane] = (uint8_t)res.id;
                    asm volatile("bar.sync %0, 128;" ::"r"(4 + half) : "memory");   // the four warps of this half
                    if (quad == 0 && in_atoms && !*abort_flag) {
                        const uint32_t id16 = trade[lane] | trade[32 + lane] << 4 | trade[64 + lane] << 8 | trade[96 + lane] << 12;
                        *(uint16_t *)(yq.ids + id_byte_offset(yq.rows, tok, b)) = (uint16_t)id16;
                    }
                }
            } else if (use_tma_store && out_bf16) {
                if (cols == 128) epilogue_bf16<4>(t_base, stage_ptr, stage_out, &mapY, n0, t0, lane, abort_flag, release_accumulator, staging_free);
                else epilogue_bf16<2>(t_base, stage_ptr, stage_out, &mapY, n0, t0, lane, abort_flag, release_accumulator, staging_free);
            } else if (use_tma_store) {
                for (int pass = 0; pass * 16 < cols; pass++) {        // fp32: 16 tokens x 32 columns per pass
                    uint32_t r[16];
                    tcgen05_ld_32x32b_x16(t_base + pass * 16, r);
                    tcgen05_wait_ld();
                    if ((pass + 1) * 16 >= cols) release_accumulator();
                    const uint32_t sb = staging_free();
#pragma unroll
                    for (int q = 0; q < 16; q++) *(uint32_t *)(stage_ptr + sb + q * 128 + lane * 4) = r[q];
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && !*abort_flag) {
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&mapY), "r"(n0), "r"(t0 + pass * 16), "r"(stage_out + sb) : "memory");
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
            } else {
                // plain stores: for one token the 32 lanes write 32 neighbouring output columns
                const int n = n0 + lane;
#pragma unroll 1
                for (int c = 0; c * 16 < cols; c++) {
                    uint32_t r[16];
                    tcgen05_ld_32x32b_x16(t_base + c * 16, r);
                    tcgen05_wait_ld();
                    if (n < N && !*abort_flag) {
#pragma unroll
                        for (int q = 0; q < 16; q++) {
                            const int tok = t0 + c * 16 + q;
                            if (tok < M) {
                                if (out_bf16) ((__nv_bfloat16 *)Y)[(int64_t)tok * ldy + n] = __float2bfloat16_rn(__uint_as_float(r[q]));
                                else ((float *)Y)[(int64_t)tok * ldy + n] = __uint_as_float(r[q]);
                            }
                        }
                    }
                }
                release_accumulator();
            }
        }
        // the staging buffers must outlive the stores' reads of them; the writes themselves complete with the grid
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
    }

    tcgen05_fence_before();
    __syncthreads();
    cluster_sync_all();                                           // the peer may still signal our barriers until here
    if (warp == 1) {
        tcgen05_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// Adds the k_splits partial sums of a launch in split order and writes Y: thread = four neighbouring outputs of
// one token.  partials is [k_splits][toks][np] fp32 (np a multiple of 256).
template <typename OutT>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float *__restrict__ partials, int k_splits, int toks, int np,
                                                            int M, int N, OutT *__restrict__ Y, int64_t ldy) {
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the GEMM's partial sums
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int quads = np / 4;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)M * quads) return;
    const int tok = (int)(i / quads), n = (int)(i - (int64_t)tok * quads) * 4;
    if (n >= N) return;
    float4 v[kMaxKSplits];
#pragma unroll
    for (int sp = 0; sp < kMaxKSplits; sp++)
        v[sp] = sp < k_splits ? __ldcg((const float4 *)(partials + ((size_t)sp * toks + tok) * np + n)) : make_float4(0, 0, 0, 0);
    float4 sum = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
    for (int sp = 0; sp < kMaxKSplits; sp++) {                    // fixed order: split 0, 1, ...
        sum.x += v[sp].x; sum.y += v[sp].y; sum.z += v[sp].z; sum.w += v[sp].w;
    }
    const float out[4] = {sum.x, sum.y, sum.z, sum.w};
    OutT *dst = Y + (int64_t)tok * ldy + n;
#pragma unroll
    for (int e = 0; e < 4; e++)
        if (n + e < N) {
            if (sizeof(OutT) == 2) ((__nv_bfloat16 *)dst)[e] = __float2bfloat16_rn(out[e]);
            else ((float *)dst)[e] = out[e];
        }
}

// ---- host side --------------------------------------------------------------
// Per-device state of the launcher (one process may drive several devices).
constexpr int kMaxDevices = 64;
inline int current_device() {
    int dev = 0;
    cudaGetDevice(&dev);
    return dev >= 0 && dev < kMaxDevices ? dev : 0;
}

inline int max_resident_clusters() {
    static int cached[kMaxDevices] = {};
    const int dev = current_device();
    if (cached[dev]) return cached[dev];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * 128);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = Smem::total;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_wtmem_kernel<false>, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        n = sms / 2;
    }
    cached[dev] = n;
    return n;
}

// X as operand bytes + scale atoms (the quantizer's second output form), W as a packed operand.
// Scratch a short call (M <= 128) can use to split K over more clusters: bytes of fp32 partial sums.
inline size_t splitk_workspace(int64_t M, int64_t N, int64_t K) {
    if (M > kSplitMaxTokens) return 0;
    const int64_t toks = (M + 15) / 16 * 16, np = (N + 255) / 256 * 256;
    // the split is only taken when at most half of the clusters would have a tile (74 clusters on the GPUs this
    // was written for; a launch that finds less scratch than it needs does not split)
    if (np / 256 > 37) return 0;
    return (size_t)kMaxKSplits * toks * np * sizeof(float);
}

// `scratch` (optional): splitk_workspace bytes, 256-byte aligned.
// `kernels` (optional) receives the number of kernels launched: one, or two when K was split.
// `requant` (optional; more than 128 tokens, N a multiple of 32): instead of writing Y, the epilogue quantises each
// token's result row along N with the two-stage rule and writes it as the packed operand [M, N] given here.
inline cudaError_t launch(const uint8_t *x8, const uint8_t *sfx, int64_t M, const QView &W, int64_t K, void *Y,
                          bool out_bf16, int64_t ldy, cudaStream_t st, void *scratch = nullptr, size_t scratch_bytes = 0,
                          int *kernels = nullptr, const QView *requant = nullptr) {
    if (kernels) *kernels = 1;
    CUtensorMap mapX, mapXpart, mapCodes, mapSfW, mapSfX, mapY;
    const int64_t N = W.rows, rtx = row_tiles(M), rtw = row_tiles(N), kg = k_groups(K);
    // items smaller than a whole tile: the whole problem when it has at most 128 tokens, else halves of 128
    const int part_tokens = M <= 128 ? (int)((M + 15) / 16 * 16) : 128;
    if (!make_map_2d(&mapX, CU_TENSOR_MAP_DATA_TYPE_UINT8, x8, K, M, K, BK, 128, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mapXpart, CU_TENSOR_MAP_DATA_TYPE_UINT8, x8, K, M, K, BK, part_tokens / 2, CU_TENSOR_MAP_SWIZZLE_128B) ||
        !make_map_2d(&mapCodes, CU_TENSOR_MAP_DATA_TYPE_UINT8, W.codes, K / 2, N, (uint64_t)W.ldc, 64, 128, CU_TENSOR_MAP_SWIZZLE_64B) ||
        !make_map_2d(&mapSfW, CU_TENSOR_MAP_DATA_TYPE_UINT32, W.scales, 128, rtw * kg, kScaleAtomBytes, 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !make_map_2d(&mapSfX, CU_TENSOR_MAP_DATA_TYPE_UINT32, sfx, 128, rtx * kg, kScaleAtomBytes, 128, 2, CU_TENSOR_MAP_SWIZZLE_NONE))
        return cudaErrorInvalidValue;
    // output through TMA tensor stores (32 columns x 32 or 16 rows per box) when Y is 16-byte aligned with a
    // row pitch that is a multiple of 16 bytes; otherwise plain stores
    const int esz = out_bf16 ? 2 : 4;
    int use_tma_store = (!requant && ((uintptr_t)Y & 15u) == 0 && (ldy * esz) % 16 == 0) ? 1 : 0;
    if (use_tma_store &&
        !make_map_2d(&mapY, out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Y, N, M,
                     (uint64_t)ldy * esz, 32, out_bf16 ? 32 : 16, CU_TENSOR_MAP_SWIZZLE_NONE))
        use_tma_store = 0;
    if (!use_tma_store) mapY = mapX;                                   // unused, but must be a valid object
    static bool configured[kMaxDevices] = {};
    const int dev = current_device();
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_wtmem_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::total);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(gemm_wtmem_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::total);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    Schedule sc;
    sc.w_pairs = (int)((N + 255) / 256);
    sc.t_tiles = (int)((M + 255) / 256);
    sc.k_tiles = (int)((K + BK - 1) / BK);
    const int tiles = sc.w_pairs * sc.t_tiles;
    const int resident = max_resident_clusters();
    sc.split_from = tiles;
    sc.parts = 2;
    sc.part_tokens = part_tokens;
    sc.k_splits = 1;
    sc.k_per = sc.k_tiles;
    if (M <= 128) {
        // one token tile: every item is the whole (short) token range
        sc.split_from = 0;
        sc.parts = 1;
        // few tiles: cut K so that about all clusters have an item of at least kMinKPerSplit k-steps
        int want = resident / tiles;
        if (want > kMaxKSplits) want = kMaxKSplits;
        if (want > sc.k_tiles / kMinKPerSplit) want = sc.k_tiles / kMinKPerSplit;
        if (want > 1 && M <= kSplitMaxTokens && scratch && scratch_bytes >= (size_t)want * part_tokens * sc.w_pairs * 256 * sizeof(float)) {
            sc.k_per = (sc.k_tiles + want - 1) / want;
            sc.k_splits = (sc.k_tiles + sc.k_per - 1) / sc.k_per;      // no empty split
        }
    } else {
        // a last wave (one tile per cluster) that fills at most half of the clusters is cut into 128-token items (twice as many, half
        // as long), unless the second half of the last token tile would be empty
        const int rest = tiles % resident, m_tail = (int)(M % 256);
        if (rest > 0 && 2 * rest <= resident && (m_tail == 0 || m_tail > 128)) sc.split_from = tiles - rest;
    }
    const int items = (sc.split_from + (tiles - sc.split_from) * sc.parts) * sc.k_splits;
    sc.clusters = items < resident ? items : resident;
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
    const QView none{nullptr, nullptr, nullptr, 0, 0, 0};
    cudaError_t e = requant
        ? cudaLaunchKernelEx(&cfg, gemm_wtmem_kernel<true>, mapX, mapXpart, mapCodes, mapSfW, mapSfX, (const uint8_t *)W.ids, sc,
                             (int)M, (int)N, (int)rtx, (int)rtw, Y, ldy, 0, mapY, use_tma_store, (float *)scratch, *requant)
        : cudaLaunchKernelEx(&cfg, gemm_wtmem_kernel<false>, mapX, mapXpart, mapCodes, mapSfW, mapSfX, (const uint8_t *)W.ids, sc,
                             (int)M, (int)N, (int)rtx, (int)rtw, Y, ldy, out_bf16 ? 1 : 0, mapY, use_tma_store, (float *)scratch, none);
    if (e != cudaSuccess || sc.k_splits == 1) return e;
    if (kernels) *kernels = 2;
    const int np = sc.w_pairs * 256;
    cfg.gridDim = dim3((unsigned)(((int64_t)M * (np / 4) + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.dynamicSmemBytes = 0;
    if (out_bf16)
        return cudaLaunchKernelEx(&cfg, splitk_reduce_kernel<__nv_bfloat16>, (const float *)scratch, sc.k_splits, sc.part_tokens, np,
                                  (int)M, (int)N, (__nv_bfloat16 *)Y, ldy);
    return cudaLaunchKernelEx(&cfg, splitk_reduce_kernel<float>, (const float *)scratch, sc.k_splits, sc.part_tokens, np, (int)M, (int)N,
                              (float *)Y, ldy);
}

}  // namespace tc

inline bool tc_supported(int64_t M, int64_t N, int64_t K) {
    return K % kBlock == 0 && M >= 1 && N >= 1 && M < (1ll << 31) && N < (1ll << 31) && K < (1ll << 31);
}
inline size_t tc_operand_bytes(int64_t rows, int64_t K) { return ((size_t)rows * (size_t)K + 255) & ~(size_t)255; }
// workspace of the tensor-core path given A as a packed operand: its operand bytes, then (short calls) the
// split-K scratch
inline size_t tc_gemm_workspace(int64_t M, int64_t N, int64_t K) { return tc_operand_bytes(M, K) + tc::splitk_workspace(M, N, K); }

}  // namespace bd
