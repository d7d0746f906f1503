// CUDA-core GEMM over packed operands: the block MAC exactly as Sec. 3.3 states it.
// Indices are decoded to signed 8-bit integers in half-units, the 32 products of a
// block are summed as integers (dp4a), and each block contributes
// S_b * 2^(eA + eB - 2) to a double accumulator.  Any shape; used for small M, as a
// cross-check of the tensor-core kernel, and wherever that kernel does not apply.
#pragma once
#include "bd_common.cuh"
#include "quantize.cuh"

namespace bd {

constexpr int kSimtTile = 64;

// Each byte of the result is 0xff if bit 7 of the same byte of x is set, else 0
// (prmt in its default mode replicates the byte's top bit when the selector's bit 3 is set).
__device__ __forceinline__ uint32_t sign_bytes(uint32_t x) {
    uint32_t r;
    asm("prmt.b32 %0, %1, %1, 0xba98;" : "=r"(r) : "r"(x));
    return r;
}

__device__ __forceinline__ void simt_decode_block(const QView &q, int64_t row, int b, uint32_t (&dst)[8],
                                                  int &scale) {
    if (row >= q.rows) {
#pragma unroll
        for (int i = 0; i < 8; i++) dst[i] = 0;
        scale = 0;
        return;
    }
    uint4 u = *(const uint4 *)(q.codes + row * q.ldc + (int64_t)b * 16);
    uint32_t w[4] = {u.x, u.y, u.z, u.w};
    uint32_t id = (q.ids[id_byte_offset(q.rows, row, b)] >> (4 * (b & 1))) & 15;
    uint32_t lo = c_tables.int_lo[id], hi = c_tables.int_hi[id];
#pragma unroll
    for (int i = 0; i < 4; i++) {
        uint32_t m0, m1;
        decode_word(w[i] & 0x77777777u, lo, hi, m0, m1);          // magnitudes only
        // two's-complement negate the bytes whose sign bit is set
        uint32_t s0 = sign_bytes(w[i]);                           // 0xff where elements 0..3 are negative
        uint32_t s1 = sign_bytes(w[i] << 4);                      // elements 4..7
        dst[2 * i] = __vsub4(m0 ^ s0, s0);
        dst[2 * i + 1] = __vsub4(m1 ^ s1, s1);
    }
    scale = q.scales[scale_offset(q.rows, row, b)];
}

template <typename OutT>
__global__ void __launch_bounds__(256) gemm_simt_kernel(QView A, QView B, OutT *__restrict__ Y, int64_t ldy) {
    __shared__ uint32_t sa[kSimtTile][9], sb[kSimtTile][9];
    __shared__ int sca[kSimtTile], scb[kSimtTile];
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const int64_t m0 = (int64_t)blockIdx.y * kSimtTile, n0 = (int64_t)blockIdx.x * kSimtTile;
    const int nb = (int)(A.K / kBlock);
    double acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = 0.0;

    for (int b = 0; b < nb; b++) {
        if (tid < 2 * kSimtTile) {
            uint32_t d[8];
            int sc;
            const bool isA = tid < kSimtTile;
            const int row = isA ? tid : tid - kSimtTile;
            simt_decode_block(isA ? A : B, (isA ? m0 : n0) + row, b, d, sc);
            uint32_t *dst = isA ? sa[row] : sb[row];
#pragma unroll
            for (int i = 0; i < 8; i++) dst[i] = d[i];
            (isA ? sca : scb)[row] = sc;
        }
        __syncthreads();
        uint32_t ra[4][8], rb[4][8];
#pragma unroll
        for (int i = 0; i < 4; i++)
#pragma unroll
            for (int k = 0; k < 8; k++) {
                ra[i][k] = sa[ty * 4 + i][k];
                rb[i][k] = sb[tx * 4 + i][k];
            }
#pragma unroll
        for (int i = 0; i < 4; i++)
#pragma unroll
            for (int j = 0; j < 4; j++) {
                int s = 0;
#pragma unroll
                for (int k = 0; k < 8; k++) s = __dp4a((int)ra[i][k], (int)rb[j][k], s);
                // 2^(eA + eB - 2) with e = scale - 127
                double f = __longlong_as_double((long long)(1023 - 256 + sca[ty * 4 + i] + scb[tx * 4 + j]) << 52);
                acc[i][j] += (double)s * f;
            }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) {
            int64_t m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (m < A.rows && n < B.rows) {
                if constexpr (sizeof(OutT) == 4) Y[m * ldy + n] = (float)acc[i][j];
                else Y[m * ldy + n] = __float2bfloat16_rn((float)acc[i][j]);
            }
        }
}

}  // namespace bd
