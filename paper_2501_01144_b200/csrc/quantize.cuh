// BlockDialect quantizer kernels: one thread owns one block of 32 elements.
//
// Per block (Sec. 3.2 preprocessing, two-stage selection; Sec. 3.3 rounding):
//   amax  -> shared exponent e = floor(log2 amax) - 2 (kept >= -127)
//   q5[k] = floor(4 * |x_k| * 2^-e)            (3 integer + 2 fraction bits, truncated)
//   pair  = the dialect pair whose maximum equals (max q5 + 1) >> 1 (saturated at 15)
//   id    = even member unless more elements fall in the odd member's beneficial range
//   idx_k = number of rounding thresholds of dialect id that are <= q5[k]
// All decisions are integer; the only floating-point step is an exact
// power-of-two scaling followed by truncation (fma with round-toward-zero onto 2^23).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "bd_common.cuh"
#include "ptx_sm100.cuh"

#ifndef BD_QUANT_MIN_BLOCKS
#define BD_QUANT_MIN_BLOCKS 3
#endif

namespace bd {

__constant__ DeviceTables c_tables = kTables;

// Tables in shared memory: 32-bit words, at most 32 per table group, so that any
// mix of per-thread indices is free of bank conflicts (one word per bank).
struct SmemTables {
    uint32_t round_mask[16];
    uint32_t even_mask[8];
    uint32_t odd_mask[8];
    uint32_t e4m3_lo[16], e4m3_hi[16];
    uint32_t merged_above[8];
    uint32_t direct_lo[16], direct_hi[16], direct_top[16];
};
__device__ __forceinline__ void load_tables(SmemTables &s) {
    for (int i = threadIdx.x; i < 16; i += blockDim.x) {
        s.round_mask[i] = c_tables.round_mask[i];
        s.e4m3_lo[i] = c_tables.e4m3_lo[i];
        s.e4m3_hi[i] = c_tables.e4m3_hi[i];
        s.direct_lo[i] = c_tables.direct_lo[i];
        s.direct_hi[i] = c_tables.direct_hi[i];
        s.direct_top[i] = c_tables.direct_top[i];
        if (i < 8) {
            s.even_mask[i] = c_tables.even_mask[i];
            s.odd_mask[i] = c_tables.odd_mask[i];
            s.merged_above[i] = c_tables.merged_above[i];
        }
    }
    __syncthreads();
}

// ---- loading 32 elements of a block as fp32 bit patterns -------------------
template <int DT>
struct Loader;
template <>
struct Loader<BD_F32> {
    static constexpr int kElemBytes = 4;
    __device__ static void contiguous(const void *p, uint32_t (&bits)[32]) {
        const uint4 *q = (const uint4 *)p;
#pragma unroll
        for (int i = 0; i < 8; i++) {
            uint4 u = __ldg(q + i);
            bits[4 * i] = u.x; bits[4 * i + 1] = u.y; bits[4 * i + 2] = u.z; bits[4 * i + 3] = u.w;
        }
    }
    __device__ static uint32_t one(const void *p) { return __ldg((const uint32_t *)p); }
};
template <>
struct Loader<BD_BF16> {
    static constexpr int kElemBytes = 2;
    __device__ static void contiguous(const void *p, uint32_t (&bits)[32]) {
        const uint4 *q = (const uint4 *)p;
#pragma unroll
        for (int i = 0; i < 4; i++) {
            uint4 u = __ldg(q + i);
            uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; j++) {
                bits[8 * i + 2 * j] = w[j] << 16;
                bits[8 * i + 2 * j + 1] = w[j] & 0xffff0000u;
            }
        }
    }
    __device__ static uint32_t one(const void *p) { return (uint32_t)__ldg((const uint16_t *)p) << 16; }
};
template <>
struct Loader<BD_F16> {
    static constexpr int kElemBytes = 2;
    __device__ static uint32_t cvt(uint16_t h) { return __float_as_uint(__half2float(__ushort_as_half(h))); }
    __device__ static void contiguous(const void *p, uint32_t (&bits)[32]) {
        const uint4 *q = (const uint4 *)p;
#pragma unroll
        for (int i = 0; i < 4; i++) {
            uint4 u = __ldg(q + i);
            uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; j++) {
                bits[8 * i + 2 * j] = cvt((uint16_t)(w[j] & 0xffffu));
                bits[8 * i + 2 * j + 1] = cvt((uint16_t)(w[j] >> 16));
            }
        }
    }
    __device__ static uint32_t one(const void *p) { return cvt(__ldg((const uint16_t *)p)); }
};

// floor(|x| * 2^(2-e)) for |x| given as fp32 bits (sign cleared).  eadj = max(biased
// exponent of the block maximum, 2), so that e = eadj - 129.
struct Scaler {
    float s1, s2;
    bool two_step;
    __device__ explicit Scaler(uint32_t eadj) {
        two_step = eadj < 4;                                     // 2^(131-eadj) would overflow fp32
        s1 = two_step ? 18446744073709551616.0f /* 2^64 */ : __uint_as_float((258u - eadj) << 23);
        s2 = __uint_as_float((two_step ? 194u - eadj : 127u) << 23);   // 2^(67-eadj) or 1
    }
    __device__ __forceinline__ uint32_t q5(uint32_t abits) const {
        float a = __uint_as_float(abits);
        float t = two_step ? __fmaf_rz(a * s1, s2, 8388608.0f) : __fmaf_rz(a, s1, 8388608.0f);
        return __float_as_uint(t) & 63u;
    }
};

struct BlockResult {
    uint32_t words[4];
    uint32_t id;
    uint32_t scale;   // e + 127
};

// Element rounding and packing for a chosen dialect.
__device__ __forceinline__ void encode_block(const uint32_t (&bits)[32], const Scaler &sc, uint32_t mask,
                                             uint32_t (&words)[4]) {
#pragma unroll
    for (int w = 0; w < 4; w++) {
        uint32_t word = 0;
#pragma unroll
        for (int j = 0; j < 8; j++) {
            uint32_t b = bits[8 * w + j];
            uint32_t q = sc.q5(b & 0x7fffffffu);
            uint32_t idx = __popc(mask & ((2u << q) - 1u));
            word |= word_insert(idx, b >> 31, j);
        }
        words[w] = word;
    }
}

__device__ __forceinline__ uint32_t prmt_b32(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}
// max(|a|, |b|) on both bf16 halves (the result's sign bits are the xor of the inputs'); a NaN input
// gives NaN, so non-finite inputs still show in the maximum.
__device__ __forceinline__ uint32_t absmax_bf16x2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t byte_sum(uint32_t x) { return (x * 0x01010101u) >> 24; }

// Second half of the two-stage rule, on packed nibbles.  v[w] holds, for the eight
// elements of group w (nibble = slot), the number of merged thresholds of the pair
// ABOVE the element's 5-bit code (0..10).  u = 10 - v is the number at or below it
// (see merged_mask).  Counts the two beneficial ranges with one byte-permute table
// lookup per four elements, picks the dialect, and turns u into the 3-bit index with
// nibble-parallel arithmetic.  signs[w] already holds the sign bits in place.
__device__ __forceinline__ void finish_two_stage(const uint32_t (&v)[4], const uint32_t (&signs)[4], uint32_t pair,
                                                 uint32_t &id, uint32_t (&words)[4]) {
    // table byte of v: 0x01 for v in {1,2} (u in {9,8}: even range), 0x10 for v in {3,4} (odd range);
    // v >= 8 selects "replicate the top bit" of bytes 0..2, which is 0.
    uint32_t acc = 0;
#pragma unroll
    for (int w = 0; w < 4; w++)
        acc += prmt_b32(0x10010100u, 0x00000010u, v[w]) + prmt_b32(0x10010100u, 0x00000010u, v[w] >> 16);
    const uint32_t cnt_even = byte_sum(acc & 0x0f0f0f0fu), cnt_odd = byte_sum((acc >> 4) & 0x0f0f0f0fu);
    const uint32_t odd = cnt_odd > cnt_even ? 1u : 0u;             // equal counts: the even member
    id = 2u * pair + odd;
    const uint32_t first_step = odd ? 0x11111111u : 0x22222222u;   // [u >= 7] or [u >= 6] via a carry into bit 3
    const uint32_t odd_mask = 0u - odd;
#pragma unroll
    for (int w = 0; w < 4; w++) {
        const uint32_t u = 0xaaaaaaaau - v[w];                      // nibble-wise 10 - v, no borrows
        const uint32_t b3 = (u >> 3) & 0x11111111u, b1 = (u >> 1) & 0x11111111u, b0 = u & 0x11111111u;
        const uint32_t f = ((u + first_step) >> 3) & 0x11111111u;
        const uint32_t top = b3 & (b1 | (b0 & ~odd_mask));          // [u >= 9] (even) or [u >= 10] (odd)
        words[w] = (u - f - b3 - top) | signs[w];
    }
}

// The same selection, emitting operand bytes (E4M3) instead of indices: with the dialect known, the byte of an
// element is a function of its v alone, an eleven-entry table.  Two byte permutes read it: entries 0..7 with v
// as the selector (v >= 8 selects "replicate the top bit" of a byte whose top bit is clear: zero), entries 8..10
// with v ^ 8 (now v < 8 gives zero).  s03 / s47 hold the high bytes of elements 0..3 / 4..7 of each group.
__device__ __forceinline__ void finish_two_stage_e4m3(const uint32_t (&v)[4], const uint32_t (&s03)[4],
                                                      const uint32_t (&s47)[4], uint32_t pair, const SmemTables &tab,
                                                      uint32_t &id, uint32_t (&out)[8]) {
    uint32_t acc = 0;
#pragma unroll
    for (int w = 0; w < 4; w++)
        acc += prmt_b32(0x10010100u, 0x00000010u, v[w]) + prmt_b32(0x10010100u, 0x00000010u, v[w] >> 16);
    const uint32_t cnt_even = byte_sum(acc & 0x0f0f0f0fu), cnt_odd = byte_sum((acc >> 4) & 0x0f0f0f0fu);
    id = 2u * pair + (cnt_odd > cnt_even ? 1u : 0u);              // equal counts: the even member
    const uint32_t lo = tab.direct_lo[id], hi = tab.direct_hi[id], top = tab.direct_top[id];
#pragma unroll
    for (int w = 0; w < 4; w++) {
        const uint32_t x = v[w] ^ 0x88888888u;
        out[2 * w] = (prmt_b32(lo, hi, v[w]) | prmt_b32(top, 0u, x)) | (s03[w] & 0x80808080u);
        out[2 * w + 1] = (prmt_b32(lo, hi, v[w] >> 16) | prmt_b32(top, 0u, x >> 16)) | (s47[w] & 0x80808080u);
    }
}

// Exact-MSE rule (Sec. 3.2 first paragraph; Sec. 4.3): all 16 dialects, squared
// error against the untruncated scaled magnitude, fp64, element order, no
// contraction; the lowest id wins equal sums.
__device__ __forceinline__ BlockResult quantize_mse(const uint32_t (&bits)[32], const SmemTables &tab,
                                                    bool &nonfinite) {
    uint32_t amax = 0;
#pragma unroll
    for (int k = 0; k < 32; k++) amax = max(amax, bits[k] & 0x7fffffffu);
    nonfinite = amax >= 0x7f800000u;
    uint32_t eadj = max(amax >> 23, 2u);
    Scaler sc(eadj);
    // 2^-e as a double: e = eadj - 129  ->  biased double exponent 1023 - e
    double inv = __longlong_as_double((long long)(1023 + 129 - (int)eadj) << 52);
    uint32_t best = 0;
    double best_err = __longlong_as_double(0x7ff0000000000000LL);
    for (uint32_t d = 0; d < 16; d++) {
        uint32_t mask = tab.round_mask[d];
        uint64_t lut = (uint64_t)c_tables.int_hi[d] << 32 | c_tables.int_lo[d];
        double err = 0.0;
#pragma unroll
        for (int k = 0; k < 32; k++) {
            uint32_t a = bits[k] & 0x7fffffffu;
            uint32_t idx = __popc(mask & ((2u << sc.q5(a)) - 1u));
            double h = (double)((lut >> (8 * idx)) & 0xff);
            double t = __dsub_rn(__dmul_rn((double)__uint_as_float(a), inv), __dmul_rn(0.5, h));
            err = __dadd_rn(err, __dmul_rn(t, t));
        }
        if (err < best_err) {
            best_err = err;
            best = d;
        }
    }
    BlockResult r;
    r.id = best;
    r.scale = eadj - 2u;
    encode_block(bits, sc, tab.round_mask[best], r.words);
    return r;
}

// max(|a|, |b|) of two fp32 values (the result's sign is the xor of the inputs'); a NaN input gives NaN.
__device__ __forceinline__ uint32_t absmax_f32(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("max.NaN.xorsign.abs.f32 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// Two-stage rule on a block of 32 fp32 bit patterns with the arithmetic of the bf16 fast path below: the
// maximum as a tree of |.|-maxima, one fma.rz per element on |x| for its 5-bit code (a clamped block is
// prescaled by 2^64 first), popcount of the shifted merged threshold mask, signs gathered with byte permutes
// (three per four elements).  BYTES: operand bytes in e4m3[0..7] instead of indices in res.words.
template <bool BYTES>
__device__ __forceinline__ void quantize_two_stage_f32(const uint32_t (&bits_in)[32], const SmemTables &tab, BlockResult &res,
                                                       uint32_t (&e4m3)[8], bool &nonfinite) {
    uint32_t bits[32], t16[16];
#pragma unroll
    for (int k = 0; k < 32; k++) bits[k] = bits_in[k];
#pragma unroll
    for (int i = 0; i < 16; i++) t16[i] = absmax_f32(bits[2 * i], bits[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < 8; i++) t16[i] = absmax_f32(t16[2 * i], t16[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < 4; i++) t16[i] = absmax_f32(t16[2 * i], t16[2 * i + 1]);
    const uint32_t amax = absmax_f32(absmax_f32(t16[0], t16[1]), absmax_f32(t16[2], t16[3])) & 0x7fffffffu;
    nonfinite = amax >= 0x7f800000u;
    const uint32_t eadj = max(amax >> 23, 2u);
    float amax_f = __uint_as_float(amax);
    uint32_t eadj_eff = eadj;
    if (eadj < 4u) {                                              // 2^(131 - eadj) would overflow: move 2^64 into the data
#pragma unroll
        for (int k = 0; k < 32; k++) bits[k] = __float_as_uint(__uint_as_float(bits[k]) * 18446744073709551616.0f);
        amax_f *= 18446744073709551616.0f;
        eadj_eff = eadj + 64u;
    }
    const float scale = __uint_as_float((258u - eadj_eff) << 23);
    const uint32_t m5 = __float_as_uint(__fmaf_rz(amax_f, scale, 8388608.0f)) & 63u;
    const uint32_t pair = min(7u, 15u - min(15u, (m5 + 1u) >> 1));
    const uint32_t above = tab.merged_above[pair];
    uint32_t v[4] = {0, 0, 0, 0}, s03[4], s47[4];
#pragma unroll
    for (int k = 0; k < 32; k++) {
        const uint32_t t = __float_as_uint(__fmaf_rz(fabsf(__uint_as_float(bits[k])), scale, 8388608.0f));
        v[k / 8] = (uint32_t)__popc(__funnelshift_r(above, 0u, t)) * (1u << (4 * slot_of(k % 8))) + v[k / 8];
    }
#pragma unroll
    for (int w = 0; w < 4; w++) {                                 // the top bytes of the group's eight elements
        s03[w] = prmt_b32(prmt_b32(bits[8 * w], bits[8 * w + 1], 0x0073u), prmt_b32(bits[8 * w + 2], bits[8 * w + 3], 0x0073u), 0x5410u);
        s47[w] = prmt_b32(prmt_b32(bits[8 * w + 4], bits[8 * w + 5], 0x0073u), prmt_b32(bits[8 * w + 6], bits[8 * w + 7], 0x0073u), 0x5410u);
    }
    res.scale = eadj - 2u;
    if (BYTES) {
        finish_two_stage_e4m3(v, s03, s47, pair, tab, res.id, e4m3);
    } else {
        uint32_t signs[4];
#pragma unroll
        for (int w = 0; w < 4; w++) signs[w] = (s03[w] & 0x80808080u) | ((s47[w] >> 4) & 0x08080808u);
        finish_two_stage(v, signs, pair, res.id, res.words);
    }
}

// ---------------------------------------------------------------------------
// bf16 fast path of the contiguous-axis quantizer (same thread-to-block map and outputs
// as quantize_contig_kernel).  The 32 elements stay packed two per register:
//   absmax      max.NaN.xorsign.abs.bf16x2 on the packed elements (off the integer pipe);
//   q5          one fma.rz per element; the upper element of a pair is used in place (the
//               lower half then only adds less than one bf16 ulp, which cannot reach the
//               next integer of the scaled value), the lower one after a 16-bit shift;
//   selection   popcount of the pair's merged threshold mask shifted by q5, accumulated as
//               nibbles, then finish_two_stage;
//   signs       two byte permutes gather the high bytes of a group's eight elements; one shift by 4
//               puts elements 4..7 on their sign bits.
// ---------------------------------------------------------------------------
// Two-stage rule on one block held as sixteen packed bf16 pairs.  BYTES: emit the operand bytes (e4m3[0..7],
// eight elements per pair of words) instead of the packed indices (res.words).
// A block whose exponent is clamped (maximum below 2^-123, eadj < 4) would need a scale of 2^128 or more: its
// elements are first multiplied by 2^64 (exact for a power of two, subnormal inputs included) and the scale
// shrinks by the same factor, so the common arithmetic serves it too, with no call and no local memory.
template <bool BYTES>
__device__ __forceinline__ void quantize_bf16_block(const uint32_t (&Rin)[16], const SmemTables &tab, BlockResult &res,
                                                    uint32_t (&e4m3)[8]) {
    uint32_t R[16], s03[4], s47[4];
#pragma unroll
    for (int i = 0; i < 16; i++) R[i] = Rin[i];
    // |.| maximum per half as a tree (four levels instead of a chain of fifteen); NaN wins; the sign bits are noise
    uint32_t t8[8], m;
#pragma unroll
    for (int i = 0; i < 8; i++) t8[i] = absmax_bf16x2(R[2 * i], R[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < 4; i++) t8[i] = absmax_bf16x2(t8[2 * i], t8[2 * i + 1]);
    m = absmax_bf16x2(absmax_bf16x2(t8[0], t8[1]), absmax_bf16x2(t8[2], t8[3]));
    m &= 0x7fff7fffu;
    const uint32_t amax = max(m & 0xffffu, m >> 16);              // bf16 magnitude bits of the block maximum
    if (amax >= 0x7f80u) atomicOr(&g_status_word, kStatusNonfinite);
    const uint32_t eadj = max(amax >> 7, 2u);
    float amax_f = __uint_as_float(amax << 16);
    uint32_t eadj_eff = eadj;
    if (eadj < 4u) {
        const uint32_t two64 = 0x5f805f80u;                      // 2^64 in both halves
#pragma unroll
        for (int i = 0; i < 16; i++) asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(R[i]) : "r"(R[i]), "r"(two64));
        amax_f *= 18446744073709551616.0f;
        eadj_eff = eadj + 64u;
    }
#pragma unroll
    for (int w = 0; w < 4; w++) {
        // the high byte of each bf16 carries its sign in bit 7
        s03[w] = prmt_b32(R[4 * w], R[4 * w + 1], 0x7531u);
        s47[w] = prmt_b32(R[4 * w + 2], R[4 * w + 3], 0x7531u);
    }
    const float scale = __uint_as_float((258u - eadj_eff) << 23);        // 2^(2 - e) (over 2^64 for a clamped block), e = eadj - 129
    const uint32_t m5 = __float_as_uint(__fmaf_rz(amax_f, scale, 8388608.0f)) & 63u;
    const uint32_t pair = min(7u, 15u - min(15u, (m5 + 1u) >> 1));
    const uint32_t above = tab.merged_above[pair];
    uint32_t v[4] = {0, 0, 0, 0};
#pragma unroll
    for (int i = 0; i < 16; i++) {
        // magnitudes through the multiplier's |.| operand modifier; the upper element keeps the lower one's
        // bits below its own last place (less than one bf16 ulp, sign bit of the lower element included)
        const uint32_t t_lo = __float_as_uint(__fmaf_rz(fabsf(__uint_as_float(R[i] << 16)), scale, 8388608.0f));
        const uint32_t t_hi = __float_as_uint(__fmaf_rz(fabsf(__uint_as_float(R[i])), scale, 8388608.0f));
        // funnel shift in wrap mode uses only the low five bits of the count, i.e. q5
        const uint32_t v_lo = __popc(__funnelshift_r(above, 0u, t_lo));
        const uint32_t v_hi = __popc(__funnelshift_r(above, 0u, t_hi));
        v[i / 4] = v_lo * (1u << (4 * slot_of(2 * (i % 4)))) + v[i / 4];
        v[i / 4] = v_hi * (1u << (4 * slot_of(2 * (i % 4) + 1))) + v[i / 4];
    }
    res.scale = eadj - 2u;
    if (BYTES) {
        finish_two_stage_e4m3(v, s03, s47, pair, tab, res.id, e4m3);
    } else {
        uint32_t signs[4];
#pragma unroll
        for (int w = 0; w < 4; w++)                               // elements 4..7 carry their sign in bit 3 of the same bytes
            signs[w] = (s03[w] & 0x80808080u) | ((s47[w] >> 4) & 0x08080808u);
        finish_two_stage(v, signs, pair, res.id, res.words);
    }
}

// Work is cut into chunks of 256 blocks = 64 rows x one k-group (4 blocks) that fill whole sectors
// of the scale and id atoms: chunk c covers k-group c % k_groups of the rows
//   tile * 128 + 16 * half + i + 32 * j,  i in 0..15, j in 0..3,  (tile, half) = c / k_groups,
// i.e. bytes [256 * half, +256) of the scale atom and [128 * half, +128) of the id atom.  Lane l of
// warp w owns i = 2 w + l / 16, j = (l / 4) % 4, block b = l % 4, so the sixteen lanes of one i
// assemble one 16-byte scale unit and one 8-byte id unit, and every warp store of scales or ids is
// one contiguous 32- or 16-byte piece.  The four lanes of a row read 256 contiguous bytes.
// A CTA takes chunks blockIdx.x, blockIdx.x + gridDim.x, ... (consecutive chunks walk along K) and
// loads the next chunk's elements before it works on the current ones.
// The loop of one warp over its share of the chunks' eight warp-parts (warp-part wp = 8 * chunk + w, w the
// warp's place in the chunk): parts first, first + stride, ...  Two register sets take turns, so the
// prefetched part is never copied.  Every lane of the warp must call this (shuffles).
// REGULAR: rows is a multiple of 128 (a chunk takes its 64 rows from all four quarters of a 128-row tile) and
// K a multiple of 128, so no chunk has padding rows or blocks.
template <bool WRITE_CODES, bool WRITE_E4M3, bool REGULAR>
__device__ __forceinline__ void quantize_bf16_parts(const uint16_t *__restrict__ X, int64_t ld, const QView &out,
                                                    uint8_t *__restrict__ e4m3, const SmemTables &tab, uint32_t first,
                                                    uint32_t stride, uint32_t parts, uint32_t nb, uint32_t kgroups,
                                                    FastDiv div_kgroups) {
    const uint32_t rows = (uint32_t)out.rows, tiles = (rows + kRowTile - 1) / kRowTile, half_k = (uint32_t)out.ldc, row_k = (uint32_t)out.K;
    const uint32_t lane = threadIdx.x % 32u, b4 = lane & 3u, j = (lane >> 2) & 3u;
    const uint32_t row_in_part = (lane >> 4) + 32u * j;           // + 2 * w + 16 * half
    struct Part {
        uint4 l0, l1, l2, l3;          // the block's 32 elements
        uint32_t r, b, kg, th;         // row, block, k-group, 2 * tile + half
        bool valid;
    };
    // where part wp is, and its loads
    auto fetch = [&](Part &k, uint32_t wp) {
        const uint32_t c = wp >> 3;
        k.th = fast_div(c, div_kgroups);
        k.kg = c - k.th * kgroups;
        k.r = (k.th >> 1) * kRowTile + (k.th & 1u) * 16u + 2u * (wp & 7u) + row_in_part;
        k.b = k.kg * kBlocksPerAtom + b4;
        k.valid = REGULAR || (k.r < rows && k.b < nb);
        if (k.valid) {
            const uint4 *src = (const uint4 *)(X + (int64_t)k.r * ld + k.b * 32u);
            k.l0 = __ldcs(src); k.l1 = __ldcs(src + 1); k.l2 = __ldcs(src + 2); k.l3 = __ldcs(src + 3);   // read once: streaming
        }
    };
    auto process = [&](const Part &k) {
        BlockResult res;
        res.id = 0; res.scale = 0;
        res.words[0] = res.words[1] = res.words[2] = res.words[3] = 0;
        if (k.valid) {
            const uint32_t R[16] = {k.l0.x, k.l0.y, k.l0.z, k.l0.w, k.l1.x, k.l1.y, k.l1.z, k.l1.w,
                                    k.l2.x, k.l2.y, k.l2.z, k.l2.w, k.l3.x, k.l3.y, k.l3.z, k.l3.w};
            uint32_t o[8];
            quantize_bf16_block<WRITE_E4M3 && !WRITE_CODES>(R, tab, res, o);
            if (WRITE_CODES)
                *(uint4 *)(out.codes + (uint64_t)k.r * half_k + k.b * 16u) =
                    make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
            if (WRITE_E4M3) {
                if (WRITE_CODES) {                                // both forms: the bytes from the indices
                    uint32_t lo = tab.e4m3_lo[res.id], hi = tab.e4m3_hi[res.id];
#pragma unroll
                    for (int w = 0; w < 4; w++) decode_word(res.words[w], lo, hi, o[2 * w], o[2 * w + 1]);
                }
                uint4 *dst = (uint4 *)(e4m3 + (uint64_t)k.r * row_k + k.b * 32u);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        // the four lanes of a row merge their scale bytes and id nibbles
        uint32_t sc = res.scale << (8 * b4);
        uint32_t idn = res.id << (4 * b4);
        sc |= __shfl_xor_sync(0xffffffffu, sc, 1);
        idn |= __shfl_xor_sync(0xffffffffu, idn, 1);
        sc |= __shfl_xor_sync(0xffffffffu, sc, 2);
        idn |= __shfl_xor_sync(0xffffffffu, idn, 2);
        if (b4 == 0) {
            const uint32_t atom = k.kg * tiles + (k.th >> 1), r32 = k.r % 32u;
            *(uint32_t *)(out.scales + (size_t)atom * kScaleAtomBytes + r32 * 16u + j * 4u) = sc;
            if (WRITE_CODES) *(uint16_t *)(out.ids + (size_t)atom * kIdAtomBytes + r32 * 8u + j * 2u) = (uint16_t)idn;
        }
    };
    Part ka, kb;
    ka.valid = kb.valid = false;
    uint32_t wp = first;
    if (wp >= parts) return;
    fetch(ka, wp);
    while (true) {
        wp += stride;
        if (wp < parts) fetch(kb, wp);
        process(ka);
        if (wp >= parts) break;
        wp += stride;
        if (wp < parts) fetch(ka, wp);
        process(kb);
        if (wp >= parts) break;
    }
}

// Persistent CTAs of eight warps: CTA x takes chunks x, x + gridDim.x, ...
template <bool WRITE_CODES, bool WRITE_E4M3, bool REGULAR>
__global__ void __launch_bounds__(256, BD_QUANT_MIN_BLOCKS) quantize_bf16_kernel(const uint16_t *__restrict__ X, int64_t ld, QView out,
                                                            uint8_t *__restrict__ e4m3, uint32_t chunks, uint32_t nb,
                                                            uint32_t kgroups, FastDiv div_kgroups) {
    __shared__ SmemTables tab;
    load_tables(tab);
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the source may be the previous kernel's output
    // everything earlier in the stream is complete now: the next kernel may take the processors this grid
    // leaves and set itself up; it waits for this grid's results in the same way
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    quantize_bf16_parts<WRITE_CODES, WRITE_E4M3, REGULAR>(X, ld, out, e4m3, tab, 8u * blockIdx.x + threadIdx.x / 32u,
                                                          8u * gridDim.x, 8u * chunks, nb, kgroups, div_kgroups);
}

// ---------------------------------------------------------------------------
// Contiguous-axis quantizer for every source type and both selection rules (the bf16 two-stage
// case has the faster kernel above).  One CTA per chunk of 64 rows x one k-group, with the same
// thread-to-block map as above: the four lanes of a row read neighbouring blocks, sixteen lanes
// assemble one 16-byte scale unit, and the stores of scales and ids are whole sectors.  Threads
// past the real rows or blocks write the zero padding of the atoms.
// Optional second output: the decoded operand bytes (E4M3 of 0.5 * value, sign in bit 7) as a
// plain [rows][K] byte matrix, the form the tensor-core GEMM loads.
// ---------------------------------------------------------------------------
constexpr int kContigStageBytes = 2 * 8 * 4096;               // two buffers of 4 KiB per warp
// REGULAR: rows is a multiple of 128 (a chunk takes its 64 rows from all four quarters of a 128-row tile) and
// K a multiple of 128, so no chunk has padding rows or blocks.
template <int DT, int SELECT, bool WRITE_CODES, bool WRITE_E4M3, bool REGULAR>
__global__ void __launch_bounds__(256) quantize_contig_kernel(const void *__restrict__ X, int64_t ld, QView out,
                                                              uint8_t *__restrict__ e4m3, int nb, int kgroups, uint32_t chunks,
                                                              FastDiv div_kgroups) {
    __shared__ SmemTables tab;
    load_tables(tab);
    // launched with programmatic stream serialisation, like the bf16 kernel below: wait for the previous
    // kernel's results, then let the next kernel set itself up on the processors this grid leaves
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t lane = threadIdx.x % 32u, b4 = lane & 3u, j = (lane >> 2) & 3u, warp = threadIdx.x / 32u;
    // fp32 blocks are 128 bytes, one cache line each: read thread by thread, every 16-byte load of a warp
    // would touch 32 lines.  Instead the warp copies its eight rows line by line (the four blocks of a row
    // are 512 contiguous bytes, 16 per lane) into shared memory, asynchronously, and each thread then
    // picks up its own block; an xor of the chunk index keeps both sides free of bank conflicts.  Two such
    // buffers per warp: the copy of the CTA's next chunk runs while the current one is quantised.
    // (dynamic shared memory: kContigStageBytes for fp32 sources, none otherwise)
    extern __shared__ __align__(128) uint8_t stage[];
    // the copy's addresses: per chunk one 64-bit base; the eight rows of a lane are 0 or 1 and 0, 32, 64 or 96 rows
    // further on, and their places in the buffer differ by constants (the xor term depends on the parity of i only)
    const int64_t ld_bytes = ld * 4;
    const uint32_t stage_base = (uint32_t)__cvta_generic_to_shared(stage) + warp * 4096u + (lane >> 3) * 128u;
    const uint32_t swz_even = ((lane & 7u) ^ ((lane >> 3) & 7u)) * 16u, swz_odd = ((lane & 7u) ^ ((4u + (lane >> 3)) & 7u)) * 16u;
    auto copy_in = [&](uint32_t chunk, uint32_t buf) {
        const uint32_t th = fast_div(chunk, div_kgroups), kg = chunk - th * (uint32_t)kgroups;
        const int64_t row0 = (int64_t)(th >> 1) * kRowTile + (th & 1u) * 16 + 2 * warp;
        const int cb = (int)(kg * kBlocksPerAtom) + (int)(lane >> 3);            // the block this lane copies from
        const char *src0 = (const char *)X + (row0 * ld + (int64_t)cb * 32) * 4 + (lane & 7u) * 16;
        const uint32_t dst0 = stage_base + buf * 32768u;
#pragma unroll
        for (int i = 0; i < 8; i++) {
            const bool ok = REGULAR || (row0 + (i >> 2) + 32 * (i & 3) < out.rows && cb < nb);
            const char *src = ok ? src0 + ((i >> 2) + 32 * (i & 3)) * ld_bytes : (const char *)X;
            const uint32_t dst = dst0 + 512u * i + ((i & 1) ? swz_odd : swz_even);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(ok ? 16 : 0) : "memory");
        }
    };
    // CTA x takes chunks x, x + gridDim.x, ...
    uint32_t chunk = blockIdx.x, buf = 0;
    if (DT == BD_F32) {
        if (chunk < chunks) copy_in(chunk, 0);
        asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (; chunk < chunks; chunk += gridDim.x, buf ^= 1u) {
        const uint32_t th = fast_div(chunk, div_kgroups);        // 2 * tile + half
        const uint32_t kg = chunk - th * (uint32_t)kgroups;
        const int64_t r = (int64_t)(th >> 1) * kRowTile + (th & 1u) * 16 + 2 * warp + (lane >> 4) + 32 * j;
        const int b = (int)(kg * kBlocksPerAtom + b4);
        const bool valid = REGULAR || (r < out.rows && b < nb);
        BlockResult res;
        res.id = 0; res.scale = 0;
        res.words[0] = res.words[1] = res.words[2] = res.words[3] = 0;
        if (DT == BD_F32) {
            if (chunk + gridDim.x < chunks) copy_in(chunk + gridDim.x, buf ^ 1u);
            asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 1;" ::: "memory");   // all but the newest group: this chunk is in
            __syncwarp();
        }
        if (valid) {
            uint32_t bits[32];
            if (DT == BD_F32) {
                const uint8_t *mine = stage + buf * 32768u + warp * 4096u + lane * 128u;
#pragma unroll
                for (int k = 0; k < 8; k++) {
                    const uint4 u = *(const uint4 *)(mine + ((k ^ (lane & 7u)) * 16u));
                    bits[4 * k] = u.x; bits[4 * k + 1] = u.y; bits[4 * k + 2] = u.z; bits[4 * k + 3] = u.w;
                }
            } else {
                Loader<DT>::contiguous((const char *)X + (r * ld + (int64_t)b * 32) * Loader<DT>::kElemBytes, bits);
            }
            bool nonfinite;
            uint32_t o[8];
            constexpr bool kBytesOnly = WRITE_E4M3 && !WRITE_CODES && SELECT != BD_SELECT_MSE;
            if (SELECT == BD_SELECT_MSE) res = quantize_mse(bits, tab, nonfinite);
            else quantize_two_stage_f32<kBytesOnly>(bits, tab, res, o, nonfinite);
            if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
            if (WRITE_CODES)
                *(uint4 *)(out.codes + r * out.ldc + (int64_t)b * 16) =
                    make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
            if (WRITE_E4M3) {
                if (!kBytesOnly) {
                    uint32_t lo = tab.e4m3_lo[res.id], hi = tab.e4m3_hi[res.id];
#pragma unroll
                    for (int w = 0; w < 4; w++) decode_word(res.words[w], lo, hi, o[2 * w], o[2 * w + 1]);
                }
                uint4 *dst = (uint4 *)(e4m3 + r * out.K + (int64_t)b * 32);
                dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
            }
        }
        // the four lanes of a row merge their scale bytes and id nibbles
        uint32_t sc = res.scale << (8 * b4);
        uint32_t idn = res.id << (4 * b4);
        sc |= __shfl_xor_sync(0xffffffffu, sc, 1);
        idn |= __shfl_xor_sync(0xffffffffu, idn, 1);
        sc |= __shfl_xor_sync(0xffffffffu, sc, 2);
        idn |= __shfl_xor_sync(0xffffffffu, idn, 2);
        if (b4 == 0) {
            *(uint32_t *)(out.scales + scale_offset(out.rows, r, b)) = sc;
            if (WRITE_CODES) *(uint16_t *)(out.ids + id_byte_offset(out.rows, r, b)) = (uint16_t)idn;
        }
        __syncwarp();                                            // the buffer read above is the next iteration's copy target
    }
}

// ---------------------------------------------------------------------------
// Strided-axis quantizer (the value matrix V, blocks along the token axis).
// Source X is [K, rows] with `rows` contiguous; thread t owns output row
// r = t % rows_pad and the pair of blocks (2*bp, 2*bp+1), bp = t / rows_pad, so
// that consecutive lanes read consecutive addresses and each id byte has one
// writer.
// ---------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(256) quantize_strided_kernel(const void *__restrict__ X, int64_t ld, QView out,
                                                               int64_t rows_pad, int nb, int nb_pad) {
    __shared__ SmemTables tab;
    load_tables(tab);
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows_pad * (nb_pad / 2)) return;
    int64_t bp = t / rows_pad;
    int64_t r = t - bp * rows_pad;
    uint32_t idbyte = 0;
    for (int h = 0; h < 2; h++) {
        int b = (int)(2 * bp + h);
        BlockResult res;
        res.id = 0; res.scale = 0;
        if (r < out.rows && b < nb) {
            uint32_t bits[32];
#pragma unroll
            for (int k = 0; k < 32; k++)
                bits[k] = Loader<DT>::one((const char *)X + (((int64_t)b * 32 + k) * ld + r) * Loader<DT>::kElemBytes);
            bool nonfinite;
            uint32_t unused[8];
            quantize_two_stage_f32<false>(bits, tab, res, unused, nonfinite);
            if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
            *(uint4 *)(out.codes + r * out.ldc + (int64_t)b * 16) =
                make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
        }
        out.scales[scale_offset(out.rows, r, b)] = (uint8_t)res.scale;
        idbyte |= res.id << (4 * h);
    }
    out.ids[id_byte_offset(out.rows, r, 2 * bp)] = (uint8_t)idbyte;
}

// ---------------------------------------------------------------------------
// Layout conversion and dequantisation: one thread per block.
// ---------------------------------------------------------------------------
__global__ void export_canonical_kernel(QView q, uint8_t *__restrict__ codes, uint8_t *__restrict__ ids,
                                        uint8_t *__restrict__ scales, int nb) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= q.rows * nb) return;
    int64_t r = t / nb;
    int b = (int)(t - r * nb);
    uint4 u = *(const uint4 *)(q.codes + r * q.ldc + (int64_t)b * 16);
    uint32_t w[4] = {u.x, u.y, u.z, u.w}, o[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        uint32_t c = 0;
#pragma unroll
        for (int j = 0; j < 8; j++) c |= (word_sign(w[i], j) << 3 | word_index(w[i], j)) << (4 * j);
        o[i] = c;
    }
    *(uint4 *)(codes + r * (q.K / 2) + (int64_t)b * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    ids[r * nb + b] = (q.ids[id_byte_offset(q.rows, r, b)] >> (4 * (b & 1))) & 15;
    scales[r * nb + b] = q.scales[scale_offset(q.rows, r, b)];
}

// Thread t owns (r, b) over the padded grid, as in the contiguous quantizer.
__global__ void import_canonical_kernel(const uint8_t *__restrict__ codes, const uint8_t *__restrict__ ids,
                                        const uint8_t *__restrict__ scales, QView q, int64_t rows_pad, int nb,
                                        int nb_pad) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= rows_pad * nb_pad) return;
    int64_t r = t / nb_pad;
    int b = (int)(t - r * nb_pad);
    bool valid = r < q.rows && b < nb;
    uint32_t id = 0, sc = 0;
    if (valid) {
        uint4 u = *(const uint4 *)(codes + r * (q.K / 2) + (int64_t)b * 16);
        uint32_t c[4] = {u.x, u.y, u.z, u.w}, o[4];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            uint32_t w = 0;
#pragma unroll
            for (int j = 0; j < 8; j++) {
                uint32_t nib = (c[i] >> (4 * j)) & 15u;
                w |= word_insert(nib & 7u, nib >> 3, j);
            }
            o[i] = w;
        }
        *(uint4 *)(q.codes + r * q.ldc + (int64_t)b * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        id = ids[r * nb + b] & 15u;
        sc = scales[r * nb + b];
    }
    uint32_t scw = sc << (8 * (b & 3)), idn = id << (4 * (b & 3));
    scw |= __shfl_xor_sync(0xffffffffu, scw, 1);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 1);
    scw |= __shfl_xor_sync(0xffffffffu, scw, 2);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 2);
    if ((b & 3) == 0) {
        *(uint32_t *)(q.scales + scale_offset(q.rows, r, b)) = scw;
        *(uint16_t *)(q.ids + id_byte_offset(q.rows, r, b)) = (uint16_t)idn;
    }
}

__global__ void dequantize_kernel(QView q, float *__restrict__ out, int64_t ld, int nb) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= q.rows * nb) return;
    int64_t r = t / nb;
    int b = (int)(t - r * nb);
    uint4 u = *(const uint4 *)(q.codes + r * q.ldc + (int64_t)b * 16);
    uint32_t w[4] = {u.x, u.y, u.z, u.w};
    uint32_t id = (q.ids[id_byte_offset(q.rows, r, b)] >> (4 * (b & 1))) & 15;
    int e = (int)q.scales[scale_offset(q.rows, r, b)] - 127;
    uint64_t lut = (uint64_t)c_tables.int_hi[id] << 32 | c_tables.int_lo[id];
    float *dst = out + r * ld + (int64_t)b * 32;
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 8; j++) {
            float h = (float)((lut >> (8 * word_index(w[i], j))) & 0xff);
            float v = scalbnf(h, e - 1);                          // 0.5 * h * 2^e, exact
            dst[8 * i + j] = word_sign(w[i], j) ? -v : v;
        }
}

// Decode a packed operand into the plain [rows][K] operand-byte matrix (E4M3).
__global__ void decode_e4m3_kernel(QView q, uint8_t *__restrict__ out, int nb) {
    // launched in plain stream order, so everything earlier has completed: the GEMM that follows may set itself
    // up and fetch its weights while this grid runs (it waits for this grid before it reads `out`)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= q.rows * nb) return;
    int64_t r = t / nb;
    int b = (int)(t - r * nb);
    uint4 u = *(const uint4 *)(q.codes + r * q.ldc + (int64_t)b * 16);
    uint32_t w[4] = {u.x, u.y, u.z, u.w}, o[8];
    uint32_t id = (q.ids[id_byte_offset(q.rows, r, b)] >> (4 * (b & 1))) & 15;
    uint32_t lo = c_tables.e4m3_lo[id], hi = c_tables.e4m3_hi[id];
#pragma unroll
    for (int i = 0; i < 4; i++) decode_word(w[i], lo, hi, o[2 * i], o[2 * i + 1]);
    uint4 *dst = (uint4 *)(out + r * q.K + (int64_t)b * 32);
    dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
    dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
}

// Decode up to kStackMax packed operands of the same shape into one stacked operand-byte matrix
// [count * rows][K] and gather their scale atoms in the stacked operand's atom order
// (k-group-major over count * row_tiles row tiles), so that one GEMM launch serves them all.
// rows must be a multiple of 128 (whole row tiles per operand).  blockIdx.y = operand.
constexpr int kStackMax = 8;
struct StackedViews {
    const uint8_t *codes[kStackMax], *ids[kStackMax], *scales[kStackMax];
};
__global__ void decode_e4m3_stacked_kernel(StackedViews v, int count, int64_t rows, int64_t K, uint8_t *__restrict__ out,
                                           uint8_t *__restrict__ out_scales, int nb) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // see decode_e4m3_kernel
    const int h = blockIdx.y;
    const int64_t tiles = rows / kRowTile, kgs = (nb + kBlocksPerAtom - 1) / kBlocksPerAtom;
    QView q{(uint8_t *)v.codes[h], (uint8_t *)v.ids[h], (uint8_t *)v.scales[h], rows, K, K / 2};
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < rows * nb) {
        const int64_t r = t / nb;
        const int b = (int)(t - r * nb);
        uint4 u = *(const uint4 *)(q.codes + r * (K / 2) + (int64_t)b * 16);
        uint32_t w[4] = {u.x, u.y, u.z, u.w}, o[8];
        uint32_t id = (q.ids[id_byte_offset(rows, r, b)] >> (4 * (b & 1))) & 15;
        uint32_t lo = c_tables.e4m3_lo[id], hi = c_tables.e4m3_hi[id];
#pragma unroll
        for (int i = 0; i < 4; i++) decode_word(w[i], lo, hi, o[2 * i], o[2 * i + 1]);
        uint4 *dst = (uint4 *)(out + ((int64_t)h * rows + r) * K + (int64_t)b * 32);
        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
    // scale atoms, 16 bytes per thread: atom (kg, rt) of operand h goes to (kg, h * tiles + rt)
    const int64_t vecs = kgs * tiles * (kScaleAtomBytes / 16);
    for (int64_t i = t; i < vecs; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t atom = i / (kScaleAtomBytes / 16), within = i % (kScaleAtomBytes / 16);
        const int64_t kg = atom / tiles, rt = atom % tiles;
        const uint4 val = *(const uint4 *)(q.scales + atom * kScaleAtomBytes + within * 16);
        *(uint4 *)(out_scales + (kg * (count * tiles) + h * tiles + rt) * kScaleAtomBytes + within * 16) = val;
    }
}

}  // namespace bd
