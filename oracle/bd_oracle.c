/*
 * BlockDialect CPU oracle (TEST INFRASTRUCTURE, not a product path).
 *
 * A plain, slow, step-by-step restatement of what the BlockDialect quantized
 * linear layer computes, written from the paper (arXiv 2501.01144):
 *   - the DialectFP4 formatbook              (Sec. 3.1, Fig. 4)
 *   - block preprocessing                    (Sec. 3.2 "Preprocessing Stage", Fig. 5a)
 *   - two-stage dialect selection            (Sec. 3.2, Fig. 5b/5c)
 *   - exact-MSE dialect selection            (Sec. 3.2 first paragraph, Sec. 4.3)
 *   - element rounding / 4-bit encoding      (Sec. 3.3)
 *   - dequantisation and the block MAC       (Sec. 3.3, Fig. 6)
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline / reference arm
 * may call this file.  It shares no code, table generator or header with the
 * CUDA library and is never used as a fallback.
 *
 * Parity status of the formatbook: the paper gives the table only as a figure.
 * Rows 4 and 5 are pinned by values printed in Sec. 3.2 / 3.3; the remaining
 * rows follow the structural rules of Sec. 3.1 and are "parity unpinned".
 *
 * All floating point is fp64; every quantity that decides an integer result is
 * an exact integer or an exactly representable double.
 *
 * Canonical output layout (rows x K operand, blocks of B = 32 elements along K;
 * the *_bs entry points take B = 16, 32 or 64, the block sizes of the paper's
 * block-size study, Sec. 4.2 and its Table 3):
 *   codes  [rows][K/2]  byte j: element 2j in bits 3:0, element 2j+1 in bits 7:4,
 *                        nibble = sign<<3 | idx
 *   ids    [rows][K/B]  one byte per block, 0..15
 *   scales [rows][K/B]  one byte per block, e + 127
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#define BDO_BLOCK 32
#define BDO_MAX_BLOCK 64
#define BDO_OK 0
#define BDO_ERR_ARG 1
#define BDO_ERR_NONFINITE 2

enum { BDO_F32 = 0, BDO_BF16 = 1, BDO_F16 = 2 };
enum { BDO_SELECT_TWO_STAGE = 0, BDO_SELECT_MSE = 1 };

/* ---------------------------------------------------------------------------
 * Formatbook (Sec. 3.1, Fig. 4).  Magnitudes in units of 0.5, ascending, so
 * index 7 is the dialect's maximum and index 6 the value in which the two
 * dialects of a pair differ.  Rules taken from the text: unit 0.5, range up to
 * 7.5; eight pairs cover the eight possible rounded block maxima 7.5 ... 4.0;
 * the two dialects of a pair share the maximum and differ in one large value,
 * the even-numbered one holding the larger; the six smallest values stay those
 * of FP4 E2M1 (0, 0.5, 1, 1.5, 2, 3) wherever the maximum leaves room.
 * Dialect 4 = 0.5*{0,1,2,3,4,6,10,13} is printed in Sec. 3.3; dialect 5 swaps
 * 5.0 for 4.0 (Sec. 3.2).
 * ------------------------------------------------------------------------- */
#define BDO_DEFAULT_FORMATBOOK { \
    {0, 1, 2, 3, 4, 6, 12, 15}, {0, 1, 2, 3, 4, 6, 10, 15}, /* max 7.5 */ \
    {0, 1, 2, 3, 4, 6, 11, 14}, {0, 1, 2, 3, 4, 6, 9, 14},  /* max 7.0 */ \
    {0, 1, 2, 3, 4, 6, 10, 13}, {0, 1, 2, 3, 4, 6, 8, 13},  /* max 6.5 */ \
    {0, 1, 2, 3, 4, 6, 9, 12},  {0, 1, 2, 3, 4, 6, 8, 12},  /* max 6.0 (odd = FP4 E2M1) */ \
    {0, 1, 2, 3, 4, 6, 9, 11},  {0, 1, 2, 3, 4, 6, 8, 11},  /* max 5.5 */ \
    {0, 1, 2, 3, 4, 6, 8, 10},  {0, 1, 2, 3, 4, 6, 7, 10},  /* max 5.0 */ \
    {0, 1, 2, 3, 4, 6, 8, 9},   {0, 1, 2, 3, 4, 6, 7, 9},   /* max 4.5 */ \
    {0, 1, 2, 3, 4, 5, 7, 8},   {0, 1, 2, 3, 4, 5, 6, 8},   /* max 4.0 */ \
}
static const uint8_t DEFAULT_FORMATBOOK[16][8] = BDO_DEFAULT_FORMATBOOK;


/* The table in use.  It starts as the reconstruction above; bdo_set_formatbook replaces it so that a
 * test can run the same alternative table through the oracle and through the library. */
static uint8_t FORMATBOOK[16][8] = BDO_DEFAULT_FORMATBOOK;

int bdo_formatbook(uint8_t out[16][8]) {
    memcpy(out, FORMATBOOK, sizeof(FORMATBOOK));
    return BDO_OK;
}

/* in == NULL restores the default.  A table is taken only if it has the shape Sec. 3.1 and 3.2 describe:
 * ascending magnitudes from 0 up to at most 7.5, eight pairs in descending order of their shared maximum
 * 7.5 ... 4.0, the two members of a pair equal except for the value below the maximum, the even one larger. */
int bdo_set_formatbook(const uint8_t in[16][8]) {
    if (!in) {
        memcpy(FORMATBOOK, DEFAULT_FORMATBOOK, sizeof(FORMATBOOK));
        return BDO_OK;
    }
    for (int d = 0; d < 16; d++) {
        if (in[d][0] != 0 || in[d][7] > 15) return BDO_ERR_ARG;
        for (int j = 1; j < 8; j++)
            if (in[d][j] <= in[d][j - 1]) return BDO_ERR_ARG;
    }
    for (int p = 0; p < 8; p++) {
        const uint8_t *even = in[2 * p], *odd = in[2 * p + 1];
        if (even[7] != 15 - p || odd[7] != 15 - p) return BDO_ERR_ARG;
        for (int j = 0; j < 6; j++)
            if (even[j] != odd[j]) return BDO_ERR_ARG;
        if (even[6] <= odd[6]) return BDO_ERR_ARG;
    }
    memcpy(FORMATBOOK, in, sizeof(FORMATBOOK));
    return BDO_OK;
}

/* ---------------------------------------------------------------------------
 * Reading an input element as an exact real number.
 * ------------------------------------------------------------------------- */
static double load_f32(const void *p, int64_t i) {
    float f;
    memcpy(&f, (const char *)p + 4 * i, 4);
    return (double)f;
}
static double load_bf16(const void *p, int64_t i) {
    uint16_t h;
    memcpy(&h, (const char *)p + 2 * i, 2);
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}
static double load_f16(const void *p, int64_t i) {
    uint16_t h;
    memcpy(&h, (const char *)p + 2 * i, 2);
    int sign = h >> 15, ex = (h >> 10) & 31, fr = h & 1023;
    double v;
    if (ex == 0) v = ldexp((double)fr, -24);
    else if (ex == 31) v = fr ? NAN : INFINITY;
    else v = ldexp((double)(1024 + fr), ex - 25);
    return sign ? -v : v;
}
static double load_elem(const void *p, int dtype, int64_t i) {
    if (dtype == BDO_F32) return load_f32(p, i);
    if (dtype == BDO_BF16) return load_bf16(p, i);
    return load_f16(p, i);
}

/* ---------------------------------------------------------------------------
 * Preprocessing (Sec. 3.2, Fig. 5a; Sec. 3.1 for the exponent).
 *   e     = floor(log2(block max magnitude)) - 2, kept >= -127 so that e + 127
 *           fits an unsigned byte (an all-zero block takes e = -127)
 *   q5[k] = the scaled magnitude |x_k| * 2^-e with three integer and two
 *           fractional bits, lower bits truncated: floor(4 * |x_k| * 2^-e)
 * ------------------------------------------------------------------------- */
static int shared_exponent(const double *mag, int bs) {
    double amax = 0.0;
    for (int k = 0; k < bs; k++)
        if (mag[k] > amax) amax = mag[k];
    if (amax == 0.0) return -127;
    int ex;
    frexp(amax, &ex); /* amax = f * 2^ex, f in [0.5, 1)  =>  floor(log2 amax) = ex - 1 */
    int e = (ex - 1) - 2;
    return e < -127 ? -127 : e;
}

static int mag_trunc(double mag, int e) {
    double q = floor(ldexp(mag, 2 - e)); /* exact: power-of-two scaling */
    return q > 31.0 ? 31 : (int)q;       /* guard; the scaled maximum is < 8 by construction */
}

/* ---------------------------------------------------------------------------
 * Stage 1 (Sec. 3.2, Fig. 5b): round the 5-bit block maximum at its second
 * fractional bit to the 0.5 grid (half goes up), saturate at 7.5, and take the
 * pair of dialects whose maximum equals it.  A maximum below 4.0 (only after
 * the exponent clamp) takes the last pair.
 * ------------------------------------------------------------------------- */
static int stage1_pair(const int *q5, int bs) {
    int m5 = 0;
    for (int k = 0; k < bs; k++)
        if (q5[k] > m5) m5 = q5[k];
    int max_hu = (m5 + 1) / 2; /* half-units */
    if (max_hu > 15) max_hu = 15;
    for (int p = 0; p < 8; p++)
        if (FORMATBOOK[2 * p][7] == max_hu) return p;
    return 7;
}

/* ---------------------------------------------------------------------------
 * Beneficial range of a dialect (Sec. 3.2, Fig. 5c), in units of 0.25 so that
 * every midpoint is an integer: [lo, hi) on the 5-bit code.
 *   even dialect: from the midpoint of the two differing values up to the
 *                 midpoint of its differing value and the shared maximum;
 *   odd dialect:  from the midpoint of its differing value and the next lower
 *                 value up to the midpoint of the two differing values.
 * ------------------------------------------------------------------------- */
int bdo_beneficial_range(int dialect, int *lo, int *hi) {
    if (dialect < 0 || dialect > 15) return BDO_ERR_ARG;
    int p = dialect / 2;
    int d_even = FORMATBOOK[2 * p][6], d_odd = FORMATBOOK[2 * p + 1][6];
    if (dialect % 2 == 0) {
        *lo = d_even + d_odd;               /* 2 * (d_even/2 + d_odd/2)/2 in quarter units */
        *hi = d_even + FORMATBOOK[2 * p][7];
    } else {
        *lo = d_odd + FORMATBOOK[2 * p + 1][5];
        *hi = d_even + d_odd;
    }
    return BDO_OK;
}

/* Stage 2: the dialect of the pair with more block elements inside its
 * beneficial range; on equal counts the even one (larger magnitudes first). */
static int stage2_pick(const int *q5, int pair, int bs) {
    int lo_e, hi_e, lo_o, hi_o, cnt_e = 0, cnt_o = 0;
    bdo_beneficial_range(2 * pair, &lo_e, &hi_e);
    bdo_beneficial_range(2 * pair + 1, &lo_o, &hi_o);
    for (int k = 0; k < bs; k++) {
        if (q5[k] >= lo_e && q5[k] < hi_e) cnt_e++;
        if (q5[k] >= lo_o && q5[k] < hi_o) cnt_o++;
    }
    return cnt_e >= cnt_o ? 2 * pair : 2 * pair + 1;
}

/* ---------------------------------------------------------------------------
 * Element rounding (Sec. 3.3): the index of the representable value of the
 * dialect nearest to the 5-bit code; of two equally near values the larger.
 * Distances are compared in quarter units: |q5 - 2 * v|.
 * ------------------------------------------------------------------------- */
int bdo_round_code(int dialect, int q5) {
    int best = 0, best_dist = 1 << 20;
    for (int j = 0; j < 8; j++) {
        int dist = q5 - 2 * (int)FORMATBOOK[dialect][j];
        if (dist < 0) dist = -dist;
        if (dist <= best_dist) { /* "<=": the later (larger) value wins a tie */
            best = j;
            best_dist = dist;
        }
    }
    return best;
}

/* Exact-MSE selection (Sec. 3.2, Sec. 4.3): quantise the block onto each of
 * the 16 dialects with the block's shared exponent and keep the dialect with
 * the smallest sum of squared errors against the untruncated scaled
 * magnitudes; the lowest number wins equal sums. */
static int select_mse(const double *mag, const int *q5, int e, int bs) {
    int best = 0;
    double best_err = INFINITY;
    for (int d = 0; d < 16; d++) {
        double err = 0.0;
        for (int k = 0; k < bs; k++) {
            double t = ldexp(mag[k], -e) - 0.5 * (double)FORMATBOOK[d][bdo_round_code(d, q5[k])];
            err = err + t * t;
        }
        if (err < best_err) {
            best_err = err;
            best = d;
        }
    }
    return best;
}

/* One block: bs reals -> bs nibbles, dialect id, shared exponent.  The block size only sets how many elements
 * share the exponent and the dialect (Sec. 4.2, Table 3); every step is the same. */
static int quantize_block(const double *x, int select, int bs, uint8_t *nib, int *id_out, int *e_out) {
    double mag[BDO_MAX_BLOCK];
    int q5[BDO_MAX_BLOCK];
    for (int k = 0; k < bs; k++) {
        if (!isfinite(x[k])) return BDO_ERR_NONFINITE;
        mag[k] = fabs(x[k]);
    }
    int e = shared_exponent(mag, bs);
    for (int k = 0; k < bs; k++) q5[k] = mag_trunc(mag[k], e);
    int id;
    if (select == BDO_SELECT_MSE) id = select_mse(mag, q5, e, bs);
    else id = stage2_pick(q5, stage1_pair(q5, bs), bs);
    for (int k = 0; k < bs; k++) {
        int sign = signbit(x[k]) ? 1 : 0;
        nib[k] = (uint8_t)(sign << 3 | bdo_round_code(id, q5[k]));
    }
    *id_out = id;
    *e_out = e;
    return BDO_OK;
}

/* Quantise a [rows, K] operand whose blocks run along the contiguous K axis.
 * ld = row stride in elements.  Returns BDO_ERR_NONFINITE if any element is
 * Inf or NaN (outputs then unspecified). */
static int block_size_ok(int bs) { return bs == 16 || bs == 32 || bs == 64; }

int bdo_quantize_bs(const void *x, int dtype, int64_t rows, int64_t K, int64_t ld, int select, int bs,
                    uint8_t *codes, uint8_t *ids, uint8_t *scales) {
    if (!block_size_ok(bs) || K % bs || rows < 0 || K < 0 || ld < K) return BDO_ERR_ARG;
    int status = BDO_OK;
    int64_t nb = K / bs;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) reduction(max : status)
#endif
    for (int64_t r = 0; r < rows; r++) {
        for (int64_t b = 0; b < nb; b++) {
            double xb[BDO_MAX_BLOCK];
            uint8_t nib[BDO_MAX_BLOCK];
            int id, e;
            for (int k = 0; k < bs; k++) xb[k] = load_elem(x, dtype, r * ld + b * bs + k);
            int st = quantize_block(xb, select, bs, nib, &id, &e);
            if (st != BDO_OK) {
                status = st;
                continue;
            }
            for (int k = 0; k < bs; k += 2)
                codes[r * (K / 2) + b * (bs / 2) + k / 2] = (uint8_t)(nib[k] | nib[k + 1] << 4);
            ids[r * nb + b] = (uint8_t)id;
            scales[r * nb + b] = (uint8_t)(e + 127);
        }
    }
    return status;
}

int bdo_quantize(const void *x, int dtype, int64_t rows, int64_t K, int64_t ld, int select,
                 uint8_t *codes, uint8_t *ids, uint8_t *scales) {
    return bdo_quantize_bs(x, dtype, rows, K, ld, select, BDO_BLOCK, codes, ids, scales);
}

/* Dequantisation (Sec. 3.3, Fig. 6): index -> 4-bit unsigned integer through
 * the dialect's table, times 0.5, times 2^e, with the stored sign. */
int bdo_dequantize_bs(const uint8_t *codes, const uint8_t *ids, const uint8_t *scales, int64_t rows,
                      int64_t K, int bs, double *out) {
    if (!block_size_ok(bs) || K % bs) return BDO_ERR_ARG;
    int64_t nb = K / bs;
    for (int64_t r = 0; r < rows; r++)
        for (int64_t k = 0; k < K; k++) {
            int64_t b = k / bs;
            uint8_t byte = codes[r * (K / 2) + k / 2];
            int nib = (k % 2) ? byte >> 4 : byte & 15;
            int h = FORMATBOOK[ids[r * nb + b]][nib & 7];
            double v = ldexp(0.5 * (double)h, (int)scales[r * nb + b] - 127);
            out[r * K + k] = (nib & 8) ? -v : v;
        }
    return BDO_OK;
}

int bdo_dequantize(const uint8_t *codes, const uint8_t *ids, const uint8_t *scales, int64_t rows,
                   int64_t K, double *out) {
    return bdo_dequantize_bs(codes, ids, scales, rows, K, BDO_BLOCK, out);
}

/* Reference product Y = dq(A) dq(B)^T in fp64 over the dequantised operands
 * (each operand value and each product is exact in fp64), together with the
 * tolerance base T[m,n] = sum_k |a_k| |b_k|.  A is [M,K], B is [N,K]. */
int bdo_gemm(const double *a, const double *b, int64_t M, int64_t N, int64_t K, double *Y,
             double *T) {
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            double y = 0.0, t = 0.0;
            for (int64_t k = 0; k < K; k++) {
                double prod = a[m * K + k] * b[n * K + k];
                y += prod;
                t += fabs(prod);
            }
            Y[m * N + n] = y;
            if (T) T[m * N + n] = t;
        }
    return BDO_OK;
}

/* The block MAC as the paper describes it (Sec. 3.3): unsigned 4-bit integer
 * products with the sign applied separately, exact integer sums inside a block,
 * one conversion per block: S_b * 2^(eA + eB - 2), accumulated in fp64.
 * Used by the tests to check that this route equals bdo_gemm. */
int bdo_gemm_blockmac_bs(const uint8_t *codesA, const uint8_t *idsA, const uint8_t *scalesA,
                         const uint8_t *codesB, const uint8_t *idsB, const uint8_t *scalesB,
                         int64_t M, int64_t N, int64_t K, int bs, double *Y) {
    if (!block_size_ok(bs) || K % bs) return BDO_ERR_ARG;
    int64_t nb = K / bs;
    for (int64_t m = 0; m < M; m++)
        for (int64_t n = 0; n < N; n++) {
            double y = 0.0;
            for (int64_t blk = 0; blk < nb; blk++) {
                int64_t s = 0;
                for (int k = 0; k < bs; k++) {
                    int64_t kk = blk * bs + k;
                    uint8_t ba = codesA[m * (K / 2) + kk / 2], bb = codesB[n * (K / 2) + kk / 2];
                    int na = (kk % 2) ? ba >> 4 : ba & 15, nbv = (kk % 2) ? bb >> 4 : bb & 15;
                    int64_t prod = (int64_t)FORMATBOOK[idsA[m * nb + blk]][na & 7] *
                                   (int64_t)FORMATBOOK[idsB[n * nb + blk]][nbv & 7];
                    s += ((na ^ nbv) & 8) ? -prod : prod;
                }
                int ea = (int)scalesA[m * nb + blk] - 127, eb = (int)scalesB[n * nb + blk] - 127;
                y += ldexp((double)s, ea + eb - 2);
            }
            Y[m * N + n] = y;
        }
    return BDO_OK;
}

int bdo_gemm_blockmac(const uint8_t *codesA, const uint8_t *idsA, const uint8_t *scalesA,
                      const uint8_t *codesB, const uint8_t *idsB, const uint8_t *scalesB,
                      int64_t M, int64_t N, int64_t K, double *Y) {
    return bdo_gemm_blockmac_bs(codesA, idsA, scalesA, codesB, idsB, scalesB, M, N, K, BDO_BLOCK, Y);
}

/* Number of threads the row loops above run on (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
int bdo_threads(void) { return omp_get_max_threads(); }
#else
int bdo_threads(void) { return 1; }
#endif
