// Shared definitions of the CUDA library: the DialectFP4 formatbook and the
// tables derived from it, the physical storage layout, and the status word.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bd.h"

namespace bd {

constexpr int kBlock = 32;          // elements per block along K (Sec. 3.1; Sec. 4.1 "Block size is 32")
constexpr int kRowTile = 128;       // rows per scale/id atom
constexpr int kBlocksPerAtom = 4;   // k-blocks per scale/id atom (128 elements of K)
constexpr int kScaleAtomBytes = 512;
constexpr int kIdAtomBytes = 256;

// ---------------------------------------------------------------------------
// DialectFP4 formatbook (Sec. 3.1, Fig. 4): 16 dialects x 8 magnitudes in units
// of 0.5, ascending.  Eight pairs, one per possible rounded block maximum
// 7.5 ... 4.0; the two members share the maximum (index 7) and differ in the
// value at index 6, the even member holding the larger.  Dialect 4 is the one
// the paper prints (0.5 * {0,1,2,3,4,6,10,13}); dialect 7 is FP4 E2M1.
// Everything below (thresholds, ranges, decode tables) is computed from this
// one table at compile time.
// ---------------------------------------------------------------------------
struct Formatbook {
    uint8_t v[16][8];
};
constexpr Formatbook kBook = {{
    {0, 1, 2, 3, 4, 6, 12, 15}, {0, 1, 2, 3, 4, 6, 10, 15},
    {0, 1, 2, 3, 4, 6, 11, 14}, {0, 1, 2, 3, 4, 6, 9, 14},
    {0, 1, 2, 3, 4, 6, 10, 13}, {0, 1, 2, 3, 4, 6, 8, 13},
    {0, 1, 2, 3, 4, 6, 9, 12},  {0, 1, 2, 3, 4, 6, 8, 12},
    {0, 1, 2, 3, 4, 6, 9, 11},  {0, 1, 2, 3, 4, 6, 8, 11},
    {0, 1, 2, 3, 4, 6, 8, 10},  {0, 1, 2, 3, 4, 6, 7, 10},
    {0, 1, 2, 3, 4, 6, 8, 9},   {0, 1, 2, 3, 4, 6, 7, 9},
    {0, 1, 2, 3, 4, 5, 7, 8},   {0, 1, 2, 3, 4, 5, 6, 8},
}};

// Rounding thresholds on the 5-bit code q5 (units of 0.25): a code rounds to
// index j or above exactly when q5 >= v[j-1] + v[j] (midpoint of two multiples
// of 0.5, ties to the larger magnitude; Sec. 3.3).  Stored as a bit mask with
// bit t set for each threshold t, so that index = popcount(mask & ((2 << q5) - 1)).
constexpr uint32_t round_mask(const Formatbook &b, int d) {
    uint32_t m = 0;
    for (int j = 1; j < 8; j++) m |= 1u << (b.v[d][j - 1] + b.v[d][j]);
    return m;
}

// Beneficial ranges (Sec. 3.2, Fig. 5c) as bit masks over q5.
//   even member: [ (dE + dO)/2 , (dE + max)/2 )   -> q5 in [dE + dO, dE + max)
//   odd member:  [ (dO + next lower)/2 , (dE + dO)/2 ) -> q5 in [dO + v5, dE + dO)
constexpr uint32_t range_bits(int lo, int hi) {
    uint32_t m = 0;
    for (int q = lo; q < hi && q < 32; q++) m |= 1u << q;
    return m;
}
constexpr uint32_t even_range_mask(const Formatbook &b, int p) {
    return range_bits(b.v[2 * p][6] + b.v[2 * p + 1][6], b.v[2 * p][6] + b.v[2 * p][7]);
}
constexpr uint32_t odd_range_mask(const Formatbook &b, int p) {
    return range_bits(b.v[2 * p + 1][6] + b.v[2 * p + 1][5], b.v[2 * p][6] + b.v[2 * p + 1][6]);
}

// E4M3 encoding of the magnitude 0.5 * h, h in 0..15 (exact: four significant bits).
constexpr uint8_t e4m3_of_half_units(int h) {
    if (h == 0) return 0;
    int msb = 0;
    for (int b = 3; b >= 0; b--)
        if (h >> b & 1) { msb = b; break; }
    int exp_field = msb - 1 + 7;                           // value = 2^(msb-1) * 1.mmm
    int mant = ((h << 3) >> msb) & 7;                      // three bits below the leading one
    return (uint8_t)(exp_field << 3 | mant);
}
// Eight-byte decode tables of a dialect: byte i = operand byte of index i.
constexpr uint64_t e4m3_lut(const Formatbook &b, int d) {
    uint64_t t = 0;
    for (int i = 0; i < 8; i++) t |= (uint64_t)e4m3_of_half_units(b.v[d][i]) << (8 * i);
    return t;
}
// The one-pass quantizer knows an element by u = the number of merged thresholds of its dialect pair at or
// below its 5-bit code (0..10, see merged_mask).  Its index in the chosen dialect: the pair's members skip
// different thresholds of the merged list.
constexpr int index_of_count(int u, bool odd) { return u - (u >= (odd ? 7 : 6)) - (u >= 8) - (u >= (odd ? 10 : 9)); }
// Operand bytes of a dialect by v = 10 - u (what the quantizer accumulates): bytes 0..7 are v = 0..7, bytes
// 8..10 are v = 8..10 (the three smallest magnitudes); all have a clear top bit.
constexpr uint8_t direct_byte(const Formatbook &b, int d, int v) {
    return e4m3_of_half_units(b.v[d][index_of_count(10 - v, (d & 1) != 0)]);
}
constexpr uint64_t int_lut(const Formatbook &b, int d) {
    uint64_t t = 0;
    for (int i = 0; i < 8; i++) t |= (uint64_t)b.v[d][i] << (8 * i);
    return t;
}



// ---------------------------------------------------------------------------
// Physical layout of a quantised [rows, K] operand.
//
// codes: [rows][K/2] bytes, row-major.  Each aligned group of 8 elements is one
//   little-endian 32-bit word w: the 3-bit index of element j sits in bits
//   4j+2 .. 4j; the sign of element j sits in bit 8j+7 for j < 4 and in bit
//   8(j-4)+3 for j >= 4.  With this order a word decodes to eight operand bytes
//   with two byte-permute lookups (the masked word is the selector) and two
//   and-or operations that move the signs into bit 7 of each byte.
//
// scales: atoms of 512 bytes covering 128 rows x 4 k-blocks, atom index
//   kg * row_tiles + rt; inside an atom the byte of (row r, block b) is at
//   (r % 32) * 16 + (r % 128 / 32) * 4 + b % 4: the order tcgen05.cp expects for
//   block-scaled MMA scale factors (32 lanes x 16 bytes, four row groups side by
//   side).  Padding entries hold 0.
//
// ids: atoms of 256 bytes in the same atom order and the same row order as the scales: (row r,
//   block b) is nibble b % 2 of byte (r % 32) * 8 + (r % 128 / 32) * 2 + (b % 4) / 2.
// ---------------------------------------------------------------------------
__host__ __device__ inline int64_t row_tiles(int64_t rows) { return (rows + kRowTile - 1) / kRowTile; }
__host__ __device__ inline int64_t k_groups(int64_t K) { return (K / kBlock + kBlocksPerAtom - 1) / kBlocksPerAtom; }

__host__ __device__ inline int64_t scale_offset(int64_t rows, int64_t r, int64_t b) {
    int64_t atom = (b / kBlocksPerAtom) * row_tiles(rows) + r / kRowTile;
    int rr = (int)(r % kRowTile);
    return atom * kScaleAtomBytes + (rr % 32) * 16 + (rr / 32) * 4 + (int)(b % kBlocksPerAtom);
}
__host__ __device__ inline int64_t id_byte_offset(int64_t rows, int64_t r, int64_t b) {
    int64_t atom = (b / kBlocksPerAtom) * row_tiles(rows) + r / kRowTile;
    int rr = (int)(r % kRowTile);
    return atom * kIdAtomBytes + (rr % 32) * 8 + (rr / 32) * 2 + (int)(b % kBlocksPerAtom) / 2;
}

// n / d for n < 2^31 as one widening multiply and a shift.  With s = ceil(log2 d), k = 31 + s and
// mul = floor(2^k / d) + 1 (which fits 32 bits), mul * d = 2^k + e with 0 < e <= d, so
// n * mul / 2^k = n / d + n * e / (d * 2^k), and the second term is below 1 / d because n * d < 2^k.
struct FastDiv {
    uint32_t mul, shift;
};
inline FastDiv make_fast_div(uint32_t d) {
    uint32_t s = 0;
    while ((1ull << s) < d) s++;
    FastDiv f;
    f.shift = 31 + s;
    f.mul = (uint32_t)((1ull << f.shift) / d + 1);
    return f;
}
__host__ __device__ inline uint32_t fast_div(uint32_t n, FastDiv f) { return (uint32_t)(((uint64_t)n * f.mul) >> f.shift); }

// Decode one code word into eight operand bytes (lo = elements 0..3, hi = 4..7)
// through the dialect's eight-byte table.
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t lut_lo, uint32_t lut_hi, uint32_t &lo,
                                            uint32_t &hi) {
    uint32_t sel = w & 0x77777777u;
    lo = (w & 0x80808080u) | __byte_perm(lut_lo, lut_hi, sel);
    hi = ((w << 4) & 0x80808080u) | __byte_perm(lut_lo, lut_hi, sel >> 16);
}

// Where logical element e (0..7) of an 8-element group sits in its code word: slot e.  Every
// producer and consumer of code words goes through these helpers or through decode_word, so the
// order inside a group is a library-internal choice (a block of 32 shares one scale).
//   slot s: index in bits 4s..4s+2; sign in bit 8s+7 (s < 4) or 8(s-4)+3 (s >= 4);
//   decode_word emits slot s as operand byte s (lo = slots 0..3, hi = slots 4..7).
// The sign positions are the ones the bf16 quantizer reaches with two byte permutes (the high
// bytes of eight packed elements) and one shift by 4.
__host__ __device__ constexpr int slot_of(int e) { return e; }
__host__ __device__ constexpr int sign_bit_of_slot(int s) { return s < 4 ? 8 * s + 7 : 8 * (s - 4) + 3; }
__host__ __device__ inline uint32_t word_index(uint32_t w, int e) { return (w >> (4 * slot_of(e))) & 7u; }
__host__ __device__ inline uint32_t word_sign(uint32_t w, int e) { return (w >> sign_bit_of_slot(slot_of(e))) & 1u; }
__host__ __device__ inline uint32_t word_insert(uint32_t idx, uint32_t sign, int e) {
    return idx << (4 * slot_of(e)) | sign << sign_bit_of_slot(slot_of(e));
}

// ---------------------------------------------------------------------------
// Merged thresholds of a dialect pair, for the one-pass quantizer.  With v5 the common
// value below the differing slot, dE > dO the two differing values and mx the shared
// maximum, the ten thresholds on q5
//   t0..t4 (common), v5+dO, v5+dE, dE+dO, dO+mx, dE+mx
// are strictly increasing.  u = #{thresholds <= q5} then decides everything:
//   u in {6,7}: inside the odd member's beneficial range [v5+dO, dE+dO);
//   u in {8,9}: inside the even member's range [dE+dO, dE+mx);
//   index under the even member = u - [u>=6] - [u>=8] - [u>=9];
//   index under the odd member  = u - [u>=7] - [u>=8] - [u>=10].
// pair_tables_ok() checks all of this against the plain definitions for every code.
// ---------------------------------------------------------------------------
constexpr uint32_t merged_mask(const Formatbook &b, int p) {
    const uint8_t *ev = b.v[2 * p], *od = b.v[2 * p + 1];
    uint32_t m = 0;
    for (int j = 1; j <= 5; j++) m |= 1u << (ev[j - 1] + ev[j]);
    m |= 1u << (od[5] + od[6]);
    m |= 1u << (ev[5] + ev[6]);
    m |= 1u << (ev[6] + od[6]);
    m |= 1u << (od[6] + od[7]);
    m |= 1u << (ev[6] + ev[7]);
    return m;
}
constexpr int popcount32(uint32_t x) {
    int c = 0;
    for (; x; x &= x - 1) c++;
    return c;
}
constexpr bool pair_tables_ok(const Formatbook &b) {
    for (int p = 0; p < 8; p++) {
        const uint32_t mm = merged_mask(b, p);
        if (popcount32(mm) != 10) return false;
        for (int j = 0; j < 6; j++)
            if (b.v[2 * p][j] != b.v[2 * p + 1][j]) return false;
        for (int q = 0; q < 32; q++) {
            const int u = popcount32(mm & ((2u << q) - 1u));
            const int idx_e = u - (u >= 6) - (u >= 8) - (u >= 9);
            const int idx_o = u - (u >= 7) - (u >= 8) - (u >= 10);
            if (idx_e != popcount32(round_mask(b, 2 * p) & ((2u << q) - 1u))) return false;
            if (idx_o != popcount32(round_mask(b, 2 * p + 1) & ((2u << q) - 1u))) return false;
            if (((even_range_mask(b, p) >> q) & 1u) != (uint32_t)(u == 8 || u == 9)) return false;
            if (((odd_range_mask(b, p) >> q) & 1u) != (uint32_t)(u == 6 || u == 7)) return false;
        }
    }
    return true;
}
static_assert(pair_tables_ok(kBook), "merged-threshold shortcut does not match the formatbook");

// What the kernels assume of a formatbook (bd_set_formatbook checks it before it replaces the tables):
// every row strictly ascending from 0 with values <= 15; pair p = rows 2p, 2p + 1 shares every value but
// the one at index 6, where the even row holds the larger; the pair's maximum is 15 - p (stage 1 maps the
// rounded block maximum straight to the pair); and the merged-threshold shortcut reproduces the plain
// definitions of rounding and beneficial ranges for every 5-bit code.
constexpr bool formatbook_ok(const Formatbook &b) {
    for (int d = 0; d < 16; d++) {
        if (b.v[d][0] != 0 || b.v[d][7] > 15) return false;
        for (int j = 1; j < 8; j++)
            if (b.v[d][j] <= b.v[d][j - 1]) return false;
    }
    for (int p = 0; p < 8; p++) {
        if (b.v[2 * p][7] != 15 - p || b.v[2 * p + 1][7] != 15 - p) return false;
        if (b.v[2 * p][6] <= b.v[2 * p + 1][6]) return false;
    }
    return pair_tables_ok(b);
}

struct DeviceTables {
    uint32_t round_mask[16];
    uint32_t even_mask[8];
    uint32_t odd_mask[8];
    uint32_t e4m3_lo[16], e4m3_hi[16];
    uint32_t int_lo[16], int_hi[16];
    uint32_t merged_above[8];     // merged_mask(p) >> 1: popcount(x >> q5) = thresholds above q5
    uint32_t direct_lo[16], direct_hi[16], direct_top[16];   // direct_byte for v = 0..3, 4..7, 8..10
};
constexpr DeviceTables make_tables(const Formatbook &b) {
    DeviceTables t{};
    for (int d = 0; d < 16; d++) {
        t.round_mask[d] = round_mask(b, d);
        t.e4m3_lo[d] = (uint32_t)e4m3_lut(b, d);
        t.e4m3_hi[d] = (uint32_t)(e4m3_lut(b, d) >> 32);
        t.int_lo[d] = (uint32_t)int_lut(b, d);
        t.int_hi[d] = (uint32_t)(int_lut(b, d) >> 32);
        for (int v = 0; v < 4; v++) {
            t.direct_lo[d] |= (uint32_t)direct_byte(b, d, v) << (8 * v);
            t.direct_hi[d] |= (uint32_t)direct_byte(b, d, 4 + v) << (8 * v);
            if (v < 3) t.direct_top[d] |= (uint32_t)direct_byte(b, d, 8 + v) << (8 * v);
        }
    }
    for (int p = 0; p < 8; p++) {
        t.even_mask[p] = even_range_mask(b, p);
        t.odd_mask[p] = odd_range_mask(b, p);
        t.merged_above[p] = merged_mask(b, p) >> 1;
    }
    return t;
}
constexpr DeviceTables kTables = make_tables(kBook);

// Bits of the device status word (defined in quantize.cuh; the library is one
// translation unit).  bd_poll_status reads and clears it.
enum : uint32_t { kStatusNonfinite = 1u, kStatusTimeout = 2u };

// Launch helpers shared by the translation units.
struct QView {                 // a qtensor as kernels see it
    uint8_t *codes;
    uint8_t *ids;
    uint8_t *scales;
    int64_t rows, K;
    int64_t ldc;               // bytes between the code rows: K / 2, or more for a view of the first K elements of
                               // longer rows (the value cache, whose token axis grows)
};
inline QView view_of(const bd_qtensor *q) {
    return QView{(uint8_t *)q->codes, (uint8_t *)q->ids, (uint8_t *)q->scales, q->rows, q->K, q->K / 2};
}

}  // namespace bd
