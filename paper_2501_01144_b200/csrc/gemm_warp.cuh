// Linear layer for calls of at most 16 tokens (the decode phase): a warp-level kernel that streams the packed
// weights once and does nothing else that scales with them.
//
// The tensor-core kernel of gemm_tc.cuh is built for wide tiles: tensor memory, barrier rings and two-CTA
// hand-overs cost a call several microseconds before the first product, which a call of a few tokens never
// earns back.  Here a warp owns 16 weight rows and a share of K; there are no hand-overs between warps:
//   * the packed codes, scale bytes and id nibbles of 16 rows x 128 elements of K (one "unit") travel from
//     global to the warp's own shared-memory ring with cp.async, several units ahead, and start before the
//     kernel waits for the activations (the weights do not depend on the previous kernel);
//   * every lane takes the code word (8 elements) of its row and k-slot from shared memory and expands it to eight
//     fp16 values with three kinds of byte permutes: the dialect's table of half-unit integers h = 0..15 gives the
//     magnitudes, and the pattern (sign << 15 | h) IS an fp16 number, the subnormal h * 2^-24, so no conversion
//     instruction is needed (warp-level E4M3 MMAs are emulated through fp16 on this architecture, with a
//     conversion per pair of elements; measured, they cost more than everything else in the loop together);
//   * two mma.sync m16n8k16 (fp16 x fp16, fp32 accumulation) per block of 32: A = 16 weight rows, B = the block of
//     8 tokens as fp16 integers, so the pair yields the exact in-block sums of Sec. 3.3 for 16 x 8 outputs (sums of
//     32 products of two 4-bit integers, far inside fp32's 24 bits);
//   * the block's two power-of-two scales are applied to those sums in fp32 and the blocks are added in fp32;
//   * the warps of a CTA hold different shares of K of the same 16 rows and add their sums through shared
//     memory: no partial sums in global memory, no second kernel.
// The activations come from a small kernel in front (quantize_records_kernel) which quantises the at most 16
// token rows with the two-stage rule and writes, per block of K and group of 8 tokens, a record of the values as
// fp16 integers (signed half-units) in the order the MMA's B fragment wants them, plus the block scales as fp32
// factors (which also carry the 2^22 that undoes the subnormal encoding of the weights and the half-units).
//
// Order of K inside a block: lane t of a quad feeds its elements 8t..8t+3 to the first MMA (k-slots 2t, 2t+1,
// 2t+8, 2t+9) and 8t+4..8t+7 to the second, for A and B alike; a dot product does not depend on the order.
#pragma once
#include "bd_common.cuh"
#include "quantize.cuh"

namespace bd {
namespace wk {

constexpr int kRows = 16;                  // weight rows of a CTA (the M of the MMA)
constexpr int kUnitBlocks = 4;             // blocks of K per unit: one scale/id atom along K
constexpr int kUnitK = kUnitBlocks * kBlock;
constexpr int kTokTile = 8;                // tokens per MMA (its N)
constexpr int kMaxTokens = 16;
constexpr int kCodeBytes = kRows * kUnitK / 2;         // 1024
constexpr int kStageBytes = kCodeBytes + kRows * 4 + kRows * 4;   // + scale words + id words = 1152
constexpr int kStages = 2;
constexpr int kRecBytes = kTokTile * kBlock * 2;       // fp16 values of a record (8 tokens x 32)
constexpr int kMaxWarps = 16;

// Records cover whole units: K is rounded up to 128 and the blocks past it hold zeros.
__host__ __device__ inline int64_t padded_blocks(int64_t K) { return (K + kUnitK - 1) / kUnitK * kUnitBlocks; }
__host__ __device__ inline size_t record_bytes(int64_t K, int nt) {
    return (size_t)padded_blocks(K) * nt * (kRecBytes + kTokTile * sizeof(float));
}
inline bool supported(int64_t M, int64_t N, int64_t K) {
    return M >= 1 && M <= kMaxTokens && N >= 1 && K >= kBlock && K % kBlock == 0 && K / kBlock < (1 << 20);
}

// ---- the activations: two-stage quantisation of up to 16 token rows into MMA-ordered records ----
// rec16: [K/32][nt][8 tokens][32 fp16]; recs: [K/32][nt][8] factors 2^(scale - 127 + 22) (anything finite for
// an all-zero block or a token past M, whose values are zeros).  Thread = (block b, token slot m of 8 * nt), m fastest.
template <int DT>
// blockIdx.y = problem of a batch: X advances by x_stride elements, the records by rec_stride bytes.
__global__ void __launch_bounds__(128) quantize_records_kernel(const void *__restrict__ X, int64_t ldx, int M, int nb, int nt,
                                                               uint8_t *__restrict__ rec16, float *__restrict__ recs, int64_t x_stride,
                                                               int64_t rec_stride) {
    __shared__ SmemTables tab;
    load_tables(tab);
    asm volatile("griddepcontrol.wait;" ::: "memory");           // X may be the previous kernel's result; the records
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // may still be read by the previous call's product
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int slots = kTokTile * nt;
    const int b = t / slots, m = t % slots;
    if (b >= (int)padded_blocks((int64_t)nb * kBlock)) return;
    X = (const char *)X + (int64_t)blockIdx.y * x_stride * Loader<DT>::kElemBytes;
    rec16 += (int64_t)blockIdx.y * rec_stride;
    recs = (float *)((uint8_t *)recs + (int64_t)blockIdx.y * rec_stride);
    uint4 out[4];
#pragma unroll
    for (int i = 0; i < 4; i++) out[i] = make_uint4(0, 0, 0, 0);
    float factor = 1.0f;
    if (m < M && b < nb) {
        uint32_t bits[32], unused[8];
        Loader<DT>::contiguous((const char *)X + ((int64_t)m * ldx + (int64_t)b * 32) * Loader<DT>::kElemBytes, bits);
        BlockResult res;
        bool nonfinite;
        quantize_two_stage_f32<false>(bits, tab, res, unused, nonfinite);
        if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
        // both operands are integers h = 2 * magnitude, the weights' carry 2^-24 on top: 2^(24 - 2) undoes both
        factor = __uint_as_float(min(res.scale + 22u, 254u) << 23);   // (block maxima of 2^103 and more would need 255)
        const uint32_t tlo = c_tables.int_lo[res.id], thi = c_tables.int_hi[res.id];
#pragma unroll
        for (int w = 0; w < 4; w++) {
            uint32_t v[4];                                        // elements 8w + 2i, 8w + 2i + 1 as two fp16 integers
#pragma unroll
            for (int i = 0; i < 4; i++) {
                uint32_t pair = 0;
#pragma unroll
                for (int j = 0; j < 2; j++) {
                    const int e = 2 * i + j;
                    const uint32_t idx = word_index(res.words[w], e);
                    const uint32_t mag = ((idx < 4 ? tlo : thi) >> (8 * (idx & 3))) & 0xffu;
                    const uint32_t f16 = (uint32_t)__half_as_ushort(__int2half_rn((int)mag)) | word_sign(res.words[w], e) << 15;
                    pair |= f16 << (16 * j);
                }
                v[i] = pair;
            }
            out[w] = make_uint4(v[0], v[1], v[2], v[3]);
        }
    }
    const size_t slot = (size_t)(b * nt + m / kTokTile) * kTokTile + m % kTokTile;
    uint4 *dst = (uint4 *)(rec16 + slot * (kBlock * 2));
#pragma unroll
    for (int i = 0; i < 4; i++) dst[i] = out[i];
    recs[slot] = factor;
}

constexpr int kMaxBatch = 64;
struct OperandBatch {                      // the operands of a batch that differ per problem (same shape and pitch)
    const uint8_t *codes[kMaxBatch], *ids[kMaxBatch], *scales[kMaxBatch];
};
// The same records from an operand that is already quantised (bd_gemm with a few rows of A).  BATCH: blockIdx.y
// picks the operand from `batch` and the records advance by rec_stride bytes.
template <bool BATCH>
__global__ void __launch_bounds__(128) records_from_qtensor_kernel(QView a, int nt, uint8_t *__restrict__ rec16, float *__restrict__ recs,
                                                                   const __grid_constant__ OperandBatch batch, int64_t rec_stride) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (BATCH) {
        a.codes = (uint8_t *)batch.codes[blockIdx.y];
        a.ids = (uint8_t *)batch.ids[blockIdx.y];
        a.scales = (uint8_t *)batch.scales[blockIdx.y];
        rec16 += (int64_t)blockIdx.y * rec_stride;
        recs = (float *)((uint8_t *)recs + (int64_t)blockIdx.y * rec_stride);
    }
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int slots = kTokTile * nt, nb = (int)(a.K / kBlock);
    const int b = t / slots, m = t % slots;
    if (b >= (int)padded_blocks(a.K)) return;
    uint4 out[4];
#pragma unroll
    for (int i = 0; i < 4; i++) out[i] = make_uint4(0, 0, 0, 0);
    float factor = 1.0f;
    if (m < a.rows && b < nb) {
        const uint4 u = *(const uint4 *)(a.codes + (int64_t)m * a.ldc + (int64_t)b * 16);
        const uint32_t words[4] = {u.x, u.y, u.z, u.w};
        const uint32_t id = (a.ids[id_byte_offset(a.rows, m, b)] >> (4 * (b & 1))) & 15u, scale = a.scales[scale_offset(a.rows, m, b)];
        factor = __uint_as_float(min(scale + 22u, 254u) << 23);
        const uint32_t tlo = c_tables.int_lo[id], thi = c_tables.int_hi[id];
#pragma unroll
        for (int w = 0; w < 4; w++) {
            uint32_t v[4];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                uint32_t pair = 0;
#pragma unroll
                for (int j = 0; j < 2; j++) {
                    const int e = 2 * i + j;
                    const uint32_t idx = word_index(words[w], e);
                    const uint32_t mag = ((idx < 4 ? tlo : thi) >> (8 * (idx & 3))) & 0xffu;
                    pair |= ((uint32_t)__half_as_ushort(__int2half_rn((int)mag)) | word_sign(words[w], e) << 15) << (16 * j);
                }
                v[i] = pair;
            }
            out[w] = make_uint4(v[0], v[1], v[2], v[3]);
        }
    }
    const size_t slot = (size_t)(b * nt + m / kTokTile) * kTokTile + m % kTokTile;
    uint4 *dst = (uint4 *)(rec16 + slot * (kBlock * 2));
#pragma unroll
    for (int i = 0; i < 4; i++) dst[i] = out[i];
    recs[slot] = factor;
}

// d = A B + c with fp16 operands and fp32 sums.
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1,
                                        const float (&c)[4]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
// Two fp32 values in a 64-bit register and the packed multiply / multiply-add on them (one instruction each).
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// One code word -> its eight elements as four fp16 pairs (0,1) (2,3) (4,5) (6,7), each element the subnormal
// sign << 15 | h with h the half-unit magnitude from the dialect's table (tlo: indices 0..3, thi: 4..7).
__device__ __forceinline__ void word_to_f16(uint32_t w, uint32_t tlo, uint32_t thi, uint32_t (&p)[4]) {
    const uint32_t sel = w & 0x77777777u;
    const uint32_t h_lo = __byte_perm(tlo, thi, sel), h_hi = __byte_perm(tlo, thi, sel >> 16);
    const uint32_t s_lo = w & 0x80808080u, s_hi = (w << 4) & 0x80808080u;
    p[0] = __byte_perm(h_lo, s_lo, 0x5140);
    p[1] = __byte_perm(h_lo, s_lo, 0x7362);
    p[2] = __byte_perm(h_hi, s_hi, 0x5140);
    p[3] = __byte_perm(h_hi, s_hi, 0x7362);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}

struct Params {
    const uint8_t *codes, *ids, *scales;   // the weights [N, K]
    int64_t ldc;                           // bytes between code rows
    int64_t row_tiles;                     // atoms per k-group
    const uint8_t *rec16;
    const float *recs;
    void *Y;
    int64_t ldy;
    int64_t N;                             // weight rows (the last CTA's tile may reach past them)
    int64_t rec_stride, y_stride;          // batch (blockIdx.y): bytes between the problems' records, elements between results
    int M, units, tail_blocks, y_bf16;     // units = ceil(K / 128); tail_blocks = blocks of the last unit if it is short, else 0
};

// What the decode-step attention adds to a batched launch (blockIdx.y = KV head).
//   MODE 1 (scores): no records; the B fragments come straight from the quantised queries' codes (a few rows, K = head_dim).
//   MODE 2 (P x V): after the product over the stored chunks the epilogue adds the recent tokens in high precision,
//                   sum_k P[q, n_q + k] * V_recent[k, c] in fp32 on the source values (kv_pv_finish_kernel's arithmetic).
struct Extra {
    const uint8_t *a_codes[kMaxBatch], *a_ids[kMaxBatch], *a_scales[kMaxBatch];   // MODE 1: the heads' query operands [M, K]
    int64_t a_ldc;
    const void *recent[kMaxBatch];         // MODE 2: the heads' high-precision value rows [32, N]
    const float *P;                        // MODE 2: probabilities, head y at P + y * p_stride, row pitch ldp
    int64_t ldp, p_stride;
    int n_q, n_recent, recent_dt;
};

// Shared memory of a CTA: per warp kStages stages of kStageBytes, then the warps' sums [warps][NT][4][32] floats.
// RAGGED: the rows do not fill the last tile of 16 or K does not fill the last unit of 128 (guards in the copy and
// store paths that whole shapes do without).
template <int NT, bool BATCH, bool RAGGED, int MODE>
__device__ __forceinline__ void gemm_warp_body(const Params &p, const OperandBatch &batch, const Extra &x) {
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ uint2 lut[16];
    const int warps = blockDim.x / 32, warp = threadIdx.x / 32, lane = threadIdx.x % 32, g = lane >> 2, t = lane & 3;
    if (threadIdx.x < 16) lut[threadIdx.x] = make_uint2(c_tables.int_lo[threadIdx.x], c_tables.int_hi[threadIdx.x]);
    const int64_t r0 = (int64_t)blockIdx.x * kRows;
    const int rr0 = (int)(r0 % kRowTile), rt = (int)(r0 / kRowTile);
    uint8_t *ring = smem + (size_t)warp * kStages * kStageBytes;
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);

    // ---- copies of one unit into a stage: two 16-byte pieces of codes per lane, a scale word or an id word ----
    // (source pointers walk from one of the warp's units to its next)
    const int crow = lane >> 2, cpiece = lane & 3;               // rows crow and crow + 8, piece = block inside the unit
    const uint8_t *w_codes = BATCH ? batch.codes[blockIdx.y] : p.codes, *w_ids = BATCH ? batch.ids[blockIdx.y] : p.ids,
                  *w_scales = BATCH ? batch.scales[blockIdx.y] : p.scales;
    const uint8_t *csrc = w_codes + (r0 + crow) * p.ldc + cpiece * 16 + (int64_t)warp * (kUnitK / 2);
    const int64_t cstep = (int64_t)warps * (kUnitK / 2), row8 = 8 * p.ldc;
    const uint32_t cdst = ring_s + (uint32_t)(crow * 64 + ((cpiece ^ (crow >> 1)) & 3) * 16);
    const int mrow = lane & 15, mrr = rr0 + mrow;                // lanes 0..15: scale word of row mrow; 16..31: id word
    const int64_t matom = lane < 16 ? kScaleAtomBytes : kIdAtomBytes;
    const uint8_t *msrc = (lane < 16 ? w_scales + (mrr % 32) * 16 + (mrr / 32) * 4 : w_ids + (mrr % 32) * 8 + (mrr / 64) * 4) +
                          ((int64_t)warp * p.row_tiles + rt) * matom;
    const int64_t mstep = (int64_t)warps * p.row_tiles * matom;
    const uint32_t mdst = ring_s + (uint32_t)(kCodeBytes + (lane < 16 ? 0 : kRows * 4) + mrow * 4);
    // rows past N and blocks past K are not read: their codes become zeros (index 0 = value 0), so whatever their
    // scale and id entries hold adds nothing
    const bool row_ok_lo = !RAGGED || r0 + crow < p.N, row_ok_hi = !RAGGED || r0 + crow + 8 < p.N;
    int next_unit = warp;
    auto issue = [&](int stage) {
        const uint32_t so = (uint32_t)stage * kStageBytes;
        const bool piece_ok = !RAGGED || !(p.tail_blocks && next_unit == p.units - 1 && cpiece >= p.tail_blocks);
        if (row_ok_lo && piece_ok) cp_async16(cdst + so, csrc);
        else asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(cdst + so), "r"(0) : "memory");
        if (row_ok_hi && piece_ok) cp_async16(cdst + so + 8 * 64, csrc + row8);
        else asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(cdst + so + 8 * 64), "r"(0) : "memory");
        cp_async4(mdst + so, msrc);
        csrc += cstep;
        msrc += mstep;
        if (RAGGED) next_unit += warps;
    };
    // this warp's units: warp, warp + warps, ...
    const int n_units = p.units > warp ? (p.units - warp + warps - 1) / warps : 0;
    // The first copies go out before the wait when a record kernel sits in front: it lets this kernel start only after
    // everything before it has completed (it waits before it lets its dependents go), so the B operand is final.
    // MODE 1 has no such kernel in front and its B operand is the key cache, which the kernel just before may have
    // appended to: there the copies wait too (the scores are one unit of K per warp, so nothing is lost).
    if (MODE != 1) {
#pragma unroll
        for (int s = 0; s < kStages; s++) {
            if (s < n_units) issue(s);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    }
    __syncthreads();                                             // the byte tables
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the records (MODE 1: the queries and the keys)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (MODE == 1) {
#pragma unroll
        for (int s = 0; s < kStages; s++) {
            if (s < n_units) issue(s);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
    }
    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.0f;
    const int id_shift = ((rr0 / 32) & 1) * 16;                  // which half of the id word holds this row group
    const int64_t rec_off = BATCH ? (int64_t)blockIdx.y * p.rec_stride : 0;
    const uint8_t *my_rec = p.rec16 + rec_off + g * (kBlock * 2) + t * 16 + (size_t)warp * (kUnitBlocks * NT * kRecBytes);
    const float *my_fac = (const float *)((const uint8_t *)p.recs + rec_off) + 2 * t + (size_t)warp * (kUnitBlocks * NT * kTokTile);
    const size_t rec_step = (size_t)warps * (kUnitBlocks * NT * kRecBytes), fac_step = (size_t)warps * (kUnitBlocks * NT * kTokTile);

    for (int i = 0; i < n_units; i++) {
        const int stage = i % kStages;
        asm volatile("cp.async.wait_group %0;" ::"n"(kStages - 1) : "memory");
        __syncwarp();
        const uint8_t *s = ring + stage * kStageBytes;
        uint32_t w_lo[kUnitBlocks], w_hi[kUnitBlocks];
#pragma unroll
        for (int b = 0; b < kUnitBlocks; b++) {
            const int off = g * 64 + ((b ^ (g >> 1)) & 3) * 16 + t * 4;
            w_lo[b] = *(const uint32_t *)(s + off);
            w_hi[b] = *(const uint32_t *)(s + off + 8 * 64);
        }
        uint32_t sc_lo = *(const uint32_t *)(s + kCodeBytes + g * 4), sc_hi = *(const uint32_t *)(s + kCodeBytes + (g + 8) * 4);
        if (RAGGED && p.tail_blocks && warp + i * warps == p.units - 1) {     // scale bytes past K may hold anything: make them 2^-127
            const uint32_t keep = (1u << (8 * p.tail_blocks)) - 1u;
            sc_lo &= keep;
            sc_hi &= keep;
        }
        const uint32_t id_lo = *(const uint32_t *)(s + kCodeBytes + kRows * 4 + g * 4) >> id_shift;
        const uint32_t id_hi = *(const uint32_t *)(s + kCodeBytes + kRows * 4 + (g + 8) * 4) >> id_shift;
        __syncwarp();                                            // everyone has read the stage: refill it
        if (i + kStages < n_units) issue(stage);
        asm volatile("cp.async.commit_group;" ::: "memory");
#pragma unroll
        for (int b = 0; b < kUnitBlocks; b++) {
            const uint2 l_lo = lut[(id_lo >> (4 * b)) & 15], l_hi = lut[(id_hi >> (4 * b)) & 15];
            uint32_t a_lo[4], a_hi[4];
            word_to_f16(w_lo[b], l_lo.x, l_lo.y, a_lo);
            word_to_f16(w_hi[b], l_hi.x, l_hi.y, a_hi);
            // 2^(scale - 127) of the two rows: byte b of the scale word moved to the exponent field
            const float f_lo = __uint_as_float((b < 3 ? sc_lo << (23 - 8 * b) : sc_lo >> 1) & 0x7f800000u);
            const float f_hi = __uint_as_float((b < 3 ? sc_hi << (23 - 8 * b) : sc_hi >> 1) & 0x7f800000u);
#pragma unroll
            for (int n = 0; n < NT; n++) {
                uint4 bb;
                float2 fa;
                if (MODE == 1) {
                    // lane group g is query row 8 n + g: its code word t of this block, expanded like the weights';
                    // the columns of this lane's sums are rows 8 n + 2 t, + 1: their block scales, with 2^46 for the
                    // two subnormal encodings and the half-units (clamped as the records' factors are)
                    const int blk = (warp + i * warps) * kUnitBlocks + b, row = n * kTokTile + g;
                    const bool blk_ok = !(p.tail_blocks && warp + i * warps == p.units - 1 && b >= p.tail_blocks);
                    uint32_t f[4] = {0, 0, 0, 0};
                    if (row < p.M && blk_ok) {
                        const uint32_t wq = *(const uint32_t *)(x.a_codes[blockIdx.y] + row * x.a_ldc + blk * 16 + t * 4);
                        const uint32_t idq = (x.a_ids[blockIdx.y][(blk / 4) * kIdAtomBytes + row * 8 + (blk % 4) / 2] >> (4 * (blk & 1))) & 15u;
                        word_to_f16(wq, lut[idq].x, lut[idq].y, f);
                    }
                    bb = make_uint4(f[0], f[1], f[2], f[3]);
                    const int c0 = n * kTokTile + 2 * t;
                    const uint8_t *sq = x.a_scales[blockIdx.y] + (blk / 4) * kScaleAtomBytes + (blk % 4);
                    fa.x = c0 < p.M && blk_ok ? __uint_as_float(min((uint32_t)sq[c0 * 16] + 46u, 254u) << 23) : 0.0f;
                    fa.y = c0 + 1 < p.M && blk_ok ? __uint_as_float(min((uint32_t)sq[(c0 + 1) * 16] + 46u, 254u) << 23) : 0.0f;
                } else {
                    bb = *(const uint4 *)(my_rec + (b * NT + n) * kRecBytes);
                    fa = *(const float2 *)(my_fac + (b * NT + n) * kTokTile);
                }
                const float zero[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                float d0[4], d[4];
                mma_f16(d0, a_lo[0], a_hi[0], a_lo[1], a_hi[1], bb.x, bb.y, zero);
                mma_f16(d, a_lo[2], a_hi[2], a_lo[3], a_hi[3], bb.z, bb.w, d0);
                acc[n][0] = fmaf(d[0] * fa.x, f_lo, acc[n][0]);
                acc[n][1] = fmaf(d[1] * fa.y, f_lo, acc[n][1]);
                acc[n][2] = fmaf(d[2] * fa.x, f_hi, acc[n][2]);
                acc[n][3] = fmaf(d[3] * fa.y, f_hi, acc[n][3]);
            }
        }
        my_rec += rec_step;
        my_fac += fac_step;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");

    // ---- the warps' sums, added in warp order; thread o < 16 * 8 * NT writes output (token o / 16, row o % 16) ----
    float *red = (float *)(smem + (size_t)warps * kStages * kStageBytes);
#pragma unroll
    for (int n = 0; n < NT; n++)
#pragma unroll
        for (int c = 0; c < 4; c++) red[((warp * NT + n) * 4 + c) * 32 + lane] = acc[n][c];
    __syncthreads();
    for (int o = threadIdx.x; o < kRows * kTokTile * NT; o += blockDim.x) {
        const int row = o % kRows, tok = o / kRows;
        if (tok >= p.M || (RAGGED && r0 + row >= p.N)) continue;
        // accumulator c of lane (row % 8) * 4 + (tok % 8) / 2 holds (row, token): c = (row / 8) * 2 + tok % 2
        const int n = tok / kTokTile, tk = tok % kTokTile, src = ((n * 4) + (row / 8) * 2 + (tk & 1)) * 32 + (row % 8) * 4 + tk / 2;
        float y = 0.0f;
        for (int w = 0; w < warps; w++) y += red[w * NT * 128 + src];
        if (MODE == 2) {                                          // the recent tokens, in fp32 on the source values
            const float *prow = x.P + (int64_t)blockIdx.y * x.p_stride + (int64_t)tok * x.ldp + x.n_q;
            const char *rec = (const char *)x.recent[blockIdx.y];
            float add = 0.0f;
            for (int k = 0; k < x.n_recent; k++) {
                const int64_t e = (int64_t)k * p.N + r0 + row;
                const uint32_t bits = x.recent_dt == BD_F32 ? Loader<BD_F32>::one(rec + e * 4)
                                    : x.recent_dt == BD_BF16 ? Loader<BD_BF16>::one(rec + e * 2) : Loader<BD_F16>::one(rec + e * 2);
                add = fmaf(prow[k], __uint_as_float(bits), add);
            }
            y += add;
        }
        const int64_t at = (BATCH ? (int64_t)blockIdx.y * p.y_stride : 0) + (int64_t)tok * p.ldy + r0 + row;
        if (p.y_bf16) ((__nv_bfloat16 *)p.Y)[at] = __float2bfloat16_rn(y);
        else ((float *)p.Y)[at] = y;
    }
}

template <int NT, bool BATCH, bool RAGGED>
__global__ void __launch_bounds__(32 * kMaxWarps, 2) gemm_warp_kernel(const __grid_constant__ Params p, const __grid_constant__ OperandBatch batch) {
    gemm_warp_body<NT, BATCH, RAGGED, 0>(p, batch, Extra{});
}
// The decode-step attention's two products (always batched, guards for ragged shapes on).
template <int NT, int MODE>
__global__ void __launch_bounds__(32 * kMaxWarps, 2) gemm_warp_attn_kernel(const __grid_constant__ Params p, const __grid_constant__ OperandBatch batch,
                                                                           const __grid_constant__ Extra x) {
    gemm_warp_body<NT, true, true, MODE>(p, batch, x);
}

}  // namespace wk
}  // namespace bd
