// Block sizes 16 and 64 (the block-size study of Sec. 4.2, Table 3) on top of the 32-element machinery.
//
// The tensor-core product applies one power-of-two scale per 32 elements of K (that is the MMA's own
// granularity), so operands of another block size are stored in the library's ordinary 32-block form:
//   block 64: each block becomes two neighbouring 32-blocks that carry the same scale and dialect id;
//   block 16: each block becomes one 32-block whose second half is zero codes (index 0 = value 0), i.e. the
//             physical operand has K' = 2 K.  Zeros add nothing to a block sum, so a product of two such
//             operands equals the product of the 16-element blocks exactly.
// Every product kernel then serves them unchanged and exactly; block 16 pays twice the MMA work and twice the
// code bytes.  The quantizer below does the selection over the real block: for 64 two neighbouring lanes own
// the halves and share maximum and range counts through shuffles (the exact-MSE sums run through both lanes
// in element order); for 16 the padded block is quantised as it stands (zeros never enter the maximum, a
// beneficial range or a squared error).
#pragma once
#include "bd_common.cuh"
#include "quantize.cuh"

namespace bd {

__host__ __device__ inline int64_t physical_k(int64_t K, int block) { return block == 16 ? 2 * K : K; }
inline bool block_size_ok(int block) { return block == 16 || block == 32 || block == 64; }

// 32 fp32 bit patterns of physical block pb of a row: the real elements, zero-padded for block 16.
template <int DT, int BS>
__device__ __forceinline__ void load_physical_block(const void *row, int pb, uint32_t (&bits)[32]) {
    if (BS == 16) {
        const char *p = (const char *)row + (int64_t)pb * 16 * Loader<DT>::kElemBytes;
#pragma unroll
        for (int k = 0; k < 16; k++) bits[k] = Loader<DT>::one(p + k * Loader<DT>::kElemBytes);
#pragma unroll
        for (int k = 16; k < 32; k++) bits[k] = 0;
    } else {
        Loader<DT>::contiguous((const char *)row + (int64_t)pb * 32 * Loader<DT>::kElemBytes, bits);
    }
}

// Two-stage rule (Sec. 3.2) on a 32-element half whose block may span PAIR = 2 neighbouring lanes: maximum and
// range counts are shared before they decide anything.  All lanes of the warp must call this.
template <int PAIR>
__device__ __forceinline__ void two_stage_shared(const uint32_t (&bits)[32], const SmemTables &tab, BlockResult &res, bool &nonfinite) {
    uint32_t amax = 0;
#pragma unroll
    for (int k = 0; k < 32; k++) amax = max(amax, bits[k] & 0x7fffffffu);
    if (PAIR == 2) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    nonfinite = amax >= 0x7f800000u;
    const uint32_t eadj = max(amax >> 23, 2u);
    const Scaler sc(eadj);
    const uint32_t m5 = sc.q5(amax);
    const uint32_t pair = min(7u, 15u - min(15u, (m5 + 1u) >> 1));
    const uint32_t even_mask = tab.even_mask[pair], odd_mask = tab.odd_mask[pair];
    uint32_t cnt_even = 0, cnt_odd = 0;
#pragma unroll
    for (int k = 0; k < 32; k++) {
        const uint32_t q = sc.q5(bits[k] & 0x7fffffffu);
        cnt_even += (even_mask >> q) & 1u;
        cnt_odd += (odd_mask >> q) & 1u;
    }
    if (PAIR == 2) {
        cnt_even += __shfl_xor_sync(0xffffffffu, cnt_even, 1);
        cnt_odd += __shfl_xor_sync(0xffffffffu, cnt_odd, 1);
    }
    res.id = 2u * pair + (cnt_odd > cnt_even ? 1u : 0u);          // equal counts: the even member
    res.scale = eadj - 2u;
    encode_block(bits, sc, tab.round_mask[res.id], res.words);
}

// Exact-MSE rule over a block that spans PAIR lanes: per dialect the fp64 sum of squared errors runs through the
// lanes in element order (the odd lane continues the even lane's sum), the lowest id wins equal sums.
template <int PAIR>
__device__ __forceinline__ void mse_shared(const uint32_t (&bits)[32], const SmemTables &tab, BlockResult &res, bool &nonfinite) {
    uint32_t amax = 0;
#pragma unroll
    for (int k = 0; k < 32; k++) amax = max(amax, bits[k] & 0x7fffffffu);
    if (PAIR == 2) amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
    nonfinite = amax >= 0x7f800000u;
    const uint32_t eadj = max(amax >> 23, 2u);
    const Scaler sc(eadj);
    const double inv = __longlong_as_double((long long)(1023 + 129 - (int)eadj) << 52);   // 2^-e
    const bool second = PAIR == 2 && (threadIdx.x & 1u);
    uint32_t best = 0;
    double best_err = __longlong_as_double(0x7ff0000000000000LL);
    for (uint32_t d = 0; d < 16; d++) {
        const uint32_t mask = tab.round_mask[d];
        const uint64_t lut = (uint64_t)c_tables.int_hi[d] << 32 | c_tables.int_lo[d];
        double err = 0.0;
        if (PAIR == 2) {                                          // the second half starts from the first half's sum
            double first_half = 0.0;
            if (!second) {
#pragma unroll
                for (int k = 0; k < 32; k++) {
                    const uint32_t a = bits[k] & 0x7fffffffu;
                    const double h = (double)((lut >> (8 * __popc(mask & ((2u << sc.q5(a)) - 1u)))) & 0xff);
                    const double t = __dsub_rn(__dmul_rn((double)__uint_as_float(a), inv), __dmul_rn(0.5, h));
                    first_half = __dadd_rn(first_half, __dmul_rn(t, t));
                }
            }
            err = __shfl_xor_sync(0xffffffffu, first_half, 1);    // the odd lane receives the even lane's sum
            if (!second) err = first_half;
        }
        if (PAIR == 1 || second) {
#pragma unroll
            for (int k = 0; k < 32; k++) {
                const uint32_t a = bits[k] & 0x7fffffffu;
                const double h = (double)((lut >> (8 * __popc(mask & ((2u << sc.q5(a)) - 1u)))) & 0xff);
                const double t = __dsub_rn(__dmul_rn((double)__uint_as_float(a), inv), __dmul_rn(0.5, h));
                err = __dadd_rn(err, __dmul_rn(t, t));
            }
        }
        if (PAIR == 2) err = __shfl_sync(0xffffffffu, err, (threadIdx.x & 31u) | 1u);   // both lanes: the whole block's sum
        if (err < best_err) {
            best_err = err;
            best = d;
        }
    }
    res.id = best;
    res.scale = eadj - 2u;
    encode_block(bits, sc, tab.round_mask[best], res.words);
}

// Thread t owns physical block (r, pb) over the padded grid [rows_pad][nbp_pad] (pb fastest), as the other
// quantizers do: threads past the operand write the zero padding of the scale and id atoms.
template <int DT, int BS, int SELECT>
__global__ void __launch_bounds__(256) quantize_bs_kernel(const void *__restrict__ X, int64_t ld, QView out, int64_t rows_pad,
                                                          int nbp, int nbp_pad) {
    __shared__ SmemTables tab;
    load_tables(tab);
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;    // (the grid covers whole warps of the padded range)
    const int64_t r = t / nbp_pad;
    const int pb = (int)(t - r * nbp_pad);
    const bool valid = r < out.rows && pb < nbp;
    uint32_t bits[32];
    if (valid) {
        load_physical_block<DT, BS>((const char *)X + r * ld * Loader<DT>::kElemBytes, pb, bits);
    } else {
#pragma unroll
        for (int k = 0; k < 32; k++) bits[k] = 0;
    }
    BlockResult res;
    bool nonfinite;
    constexpr int PAIR = BS == 64 ? 2 : 1;
    if (SELECT == BD_SELECT_MSE) mse_shared<PAIR>(bits, tab, res, nonfinite);
    else two_stage_shared<PAIR>(bits, tab, res, nonfinite);
    if (valid && nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
    if (!valid) { res.id = 0; res.scale = 0; }
    if (valid)
        *(uint4 *)(out.codes + r * out.ldc + (int64_t)pb * 16) = make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
    uint32_t scw = res.scale << (8 * (pb & 3)), idn = res.id << (4 * (pb & 3));
    scw |= __shfl_xor_sync(0xffffffffu, scw, 1);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 1);
    scw |= __shfl_xor_sync(0xffffffffu, scw, 2);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 2);
    if ((pb & 3) == 0 && r < rows_pad) {
        *(uint32_t *)(out.scales + scale_offset(out.rows, r, pb)) = scw;
        *(uint16_t *)(out.ids + id_byte_offset(out.rows, r, pb)) = (uint16_t)idn;
    }
}

// Canonical view of an operand stored for block size BS: codes [rows][K/2], ids and scales [rows][K/BS].
// Thread = physical block.
template <int BS>
__global__ void export_canonical_bs_kernel(QView q, uint8_t *__restrict__ codes, uint8_t *__restrict__ ids,
                                           uint8_t *__restrict__ scales, int nbp) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= q.rows * nbp) return;
    const int64_t r = t / nbp;
    const int pb = (int)(t - r * nbp);
    const uint4 u = *(const uint4 *)(q.codes + r * q.ldc + (int64_t)pb * 16);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        uint32_t c = 0;
#pragma unroll
        for (int j = 0; j < 8; j++) c |= (word_sign(w[i], j) << 3 | word_index(w[i], j)) << (4 * j);
        o[i] = c;
    }
    const uint32_t id = (q.ids[id_byte_offset(q.rows, r, pb)] >> (4 * (pb & 1))) & 15, sc = q.scales[scale_offset(q.rows, r, pb)];
    if (BS == 16) {                                               // the first 16 elements are the block; K = q.K / 2
        *(uint2 *)(codes + r * (q.K / 4) + (int64_t)pb * 8) = make_uint2(o[0], o[1]);
        ids[r * nbp + pb] = (uint8_t)id;
        scales[r * nbp + pb] = (uint8_t)sc;
    } else {                                                      // 64: two physical blocks per block, same id and scale
        *(uint4 *)(codes + r * (q.K / 2) + (int64_t)pb * 16) = make_uint4(o[0], o[1], o[2], o[3]);
        if ((pb & 1) == 0) {
            ids[r * (nbp / 2) + pb / 2] = (uint8_t)id;
            scales[r * (nbp / 2) + pb / 2] = (uint8_t)sc;
        }
    }
}

}  // namespace bd
