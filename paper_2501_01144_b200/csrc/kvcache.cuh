// KV cache of one KV head in DialectFP4 (appendix "Quantization Dimension", Fig. 9b).
//
// Keys are quantised sub-token-wise (blocks of 32 along head_dim): a new key vector is quantised once and becomes
// the next row of the key operand [capacity, head_dim].  Values are quantised sub-channel-wise, along the token
// axis, which is their multiplication dimension in score x V: the value operand is [head_dim, capacity] and a
// block is 32 consecutive tokens of one channel.  A single new token cannot extend such a block, so the newest
// N mod 32 value rows wait in high precision (`recent`, the source type) and are quantised once, as a whole chunk,
// when there are 32 of them.  Nothing stored is ever requantised.
//
// Both operands keep the library's ordinary layout, so the product kernels read them through views: the first
// `length` rows of the keys, and the first 32 * (length / 32) elements of every value row (code rows keep the
// pitch of the full capacity).  With head_dim <= 128 the key operand has one scale atom along K and the value
// operand one row tile, so the atom order of both does not depend on the capacity.
#pragma once
#include <cuda_fp16.h>

#include "bd_common.cuh"
#include "quantize.cuh"

namespace bd {

// The KV heads of a layer in one launch: blockIdx.y picks the head's operand and its high-precision rows; the sources
// advance by a stride per head.  (kernels launched with BATCH = false ignore it.)
constexpr int kKvMaxBatch = 64;
struct KvBatch {
    uint8_t *codes[kKvMaxBatch], *ids[kKvMaxBatch], *scales[kKvMaxBatch];
    void *recent[kKvMaxBatch];
};
template <bool BATCH>
__device__ __forceinline__ void kv_pick(QView &q, const KvBatch &batch) {
    if (BATCH) {
        q.codes = batch.codes[blockIdx.y];
        q.ids = batch.ids[blockIdx.y];
        q.scales = batch.scales[blockIdx.y];
    }
}

// New key rows: thread = (new row i, block b of 4); the four lanes of a row merge scale bytes and id nibbles.
template <int DT, bool BATCH>
__global__ void __launch_bounds__(256) kv_append_keys_kernel(const void *__restrict__ Knew, int64_t ldk, int64_t t_new, QView k,
                                                             int64_t row0, int nb, const __grid_constant__ KvBatch batch, int64_t src_stride) {
    __shared__ SmemTables tab;
    load_tables(tab);
    kv_pick<BATCH>(k, batch);
    if (BATCH) Knew = (const char *)Knew + (int64_t)blockIdx.y * src_stride * Loader<DT>::kElemBytes;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t i = t / kBlocksPerAtom;
    const int b = (int)(t % kBlocksPerAtom);
    const bool valid = i < t_new && b < nb;
    BlockResult res;
    res.id = 0; res.scale = 0;
    res.words[0] = res.words[1] = res.words[2] = res.words[3] = 0;
    const int64_t r = row0 + i;
    if (valid) {
        uint32_t bits[32], unused[8];
        Loader<DT>::contiguous((const char *)Knew + (i * ldk + (int64_t)b * 32) * Loader<DT>::kElemBytes, bits);
        bool nonfinite;
        quantize_two_stage_f32<false>(bits, tab, res, unused, nonfinite);
        if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
        *(uint4 *)(k.codes + r * k.ldc + (int64_t)b * 16) = make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
    }
    uint32_t scw = res.scale << (8 * b), idn = res.id << (4 * b);
    scw |= __shfl_xor_sync(0xffffffffu, scw, 1);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 1);
    scw |= __shfl_xor_sync(0xffffffffu, scw, 2);
    idn |= __shfl_xor_sync(0xffffffffu, idn, 2);
    if (b == 0 && i < t_new) {
        *(uint32_t *)(k.scales + scale_offset(k.rows, r, 0)) = scw;
        *(uint16_t *)(k.ids + id_byte_offset(k.rows, r, 0)) = (uint16_t)idn;
    }
}

// Value rows that do not complete a chunk: copied as they are into the high-precision slots.
template <bool BATCH>
__global__ void kv_store_recent_kernel(const void *__restrict__ Vnew, int64_t ldv_bytes, int rows, int row_bytes, uint8_t *__restrict__ recent,
                                       int slot0, const __grid_constant__ KvBatch batch, int64_t src_stride_bytes) {
    if (BATCH) {
        recent = (uint8_t *)batch.recent[blockIdx.y];
        Vnew = (const char *)Vnew + (int64_t)blockIdx.y * src_stride_bytes;
    }
    const int t = blockIdx.x * blockDim.x + threadIdx.x;          // one 2-byte unit each
    const int units = row_bytes / 2;
    if (t >= rows * units) return;
    const int i = t / units, u = t % units;
    ((uint16_t *)(recent + (int64_t)(slot0 + i) * row_bytes))[u] = ((const uint16_t *)((const char *)Vnew + i * ldv_bytes))[u];
}

// Whole chunks of 32 value rows -> one block per channel.  Thread = (channel c, pair of chunks p): the chunks 2p and
// 2p + 1 of a channel share an id byte, so one thread writes both nibbles; a nibble of an earlier call is kept.
// src: [32 * n_chunks, ld] elements, the rows of chunks chunk0 .. chunk0 + n_chunks - 1.
// BATCH: src is nullptr for "the head's own high-precision rows", else the new rows, src_stride elements per head.
template <int DT, bool BATCH>
__global__ void __launch_bounds__(256) kv_quantize_chunks_kernel(const void *__restrict__ src, int64_t ld, int n_chunks, QView v, int chunk0,
                                                                 const __grid_constant__ KvBatch batch, int64_t src_stride) {
    __shared__ SmemTables tab;
    load_tables(tab);
    kv_pick<BATCH>(v, batch);
    if (BATCH) src = src ? (const void *)((const char *)src + (int64_t)blockIdx.y * src_stride * Loader<DT>::kElemBytes) : batch.recent[blockIdx.y];
    const int d = (int)v.rows;
    const int pair0 = chunk0 / 2, n_pairs = (chunk0 + n_chunks + 1) / 2 - pair0;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= (int64_t)d * n_pairs) return;
    const int c = (int)(t % d), p = pair0 + (int)(t / d);          // neighbouring lanes = neighbouring channels
    uint32_t idbyte = 0;
    for (int h = 0; h < 2; h++) {
        const int chunk = 2 * p + h;
        if (chunk < chunk0) {                                     // stored by an earlier call: keep its nibble
            idbyte |= v.ids[id_byte_offset(v.rows, c, chunk)] & 0x0fu;
            continue;
        }
        if (chunk >= chunk0 + n_chunks) continue;
        uint32_t bits[32], unused[8];
        const char *base = (const char *)src + ((int64_t)(chunk - chunk0) * 32 * ld + c) * Loader<DT>::kElemBytes;
#pragma unroll
        for (int k = 0; k < 32; k++) bits[k] = Loader<DT>::one(base + (int64_t)k * ld * Loader<DT>::kElemBytes);
        BlockResult res;
        bool nonfinite;
        quantize_two_stage_f32<false>(bits, tab, res, unused, nonfinite);
        if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
        *(uint4 *)(v.codes + (int64_t)c * v.ldc + (int64_t)chunk * 16) = make_uint4(res.words[0], res.words[1], res.words[2], res.words[3]);
        v.scales[scale_offset(v.rows, c, chunk)] = (uint8_t)res.scale;
        idbyte |= res.id << (4 * h);
    }
    v.ids[id_byte_offset(v.rows, c, 2 * p)] = (uint8_t)idbyte;
}

// O[q, c] = (product over the stored chunks, fp32, or nothing) + sum over the recent tokens of P[q, n_q + k] * V_recent[k, c],
// the latter in fp32 on the source values ("maintained in high precision").  Thread = one output.
// blockIdx.y = head of a batch: `recent` then is an array of the heads' pointers, part / P / Y advance by their strides.
struct RecentBatch {
    const void *ptr[64];
};
template <int DT, typename OutT, bool BATCH>
__global__ void kv_pv_finish_kernel(const float *__restrict__ part, int64_t ld_part, const float *__restrict__ P, int64_t ldp, int64_t n_q,
                                    int n_recent, const void *__restrict__ recent, int d, int64_t q_rows, OutT *__restrict__ Y, int64_t ldy,
                                    const __grid_constant__ RecentBatch batch, int64_t part_stride, int64_t p_stride, int64_t y_stride) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= q_rows * d) return;
    if (BATCH) {
        recent = batch.ptr[blockIdx.y];
        if (part) part += (int64_t)blockIdx.y * part_stride;
        P += (int64_t)blockIdx.y * p_stride;
        Y += (int64_t)blockIdx.y * y_stride;
    }
    const int64_t q = t / d;
    const int c = (int)(t % d);
    float acc = 0.0f;
    for (int k = 0; k < n_recent; k++)
        acc = fmaf(P[q * ldp + n_q + k], __uint_as_float(Loader<DT>::one((const char *)recent + ((int64_t)k * d + c) * Loader<DT>::kElemBytes)), acc);
    const float y = (part ? part[q * ld_part + c] : 0.0f) + acc;
    if (sizeof(OutT) == 2) ((__nv_bfloat16 *)Y)[q * ldy + c] = __float2bfloat16_rn(y);
    else ((float *)Y)[q * ldy + c] = y;
}

// Softmax between the two products of a decode step, in high precision (Sec. 3.3): row r of S [rows, length]
// (fp32, pitch ld) becomes exp(scale * (s - max)) / sum in place, through exp2 of the scores in units of log2 e as
// in the prefill kernel.  One CTA per row; three sweeps over the row (maximum, sum, store), which for the few
// rows of a decode step sit in L1/L2.  Columns from `length` to the pitch are left alone.
__global__ void __launch_bounds__(256) kv_softmax_rows_kernel(float *__restrict__ S, int64_t ld, int64_t length, float scale) {
    __shared__ float red[8];
    float *row = S + (int64_t)blockIdx.x * ld;
    const float sl2 = scale * 1.4426950408889634f;
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    auto block_reduce = [&](float v, bool take_max) {
#pragma unroll
        for (int d = 16; d; d >>= 1) {
            const float o = __shfl_xor_sync(0xffffffffu, v, d);
            v = take_max ? fmaxf(v, o) : v + o;
        }
        __syncthreads();                                          // the previous reduction's readers are done
        if (lane == 0) red[warp] = v;
        __syncthreads();
        float r = red[0];
        for (int w = 1; w < 8; w++) r = take_max ? fmaxf(r, red[w]) : r + red[w];     // fixed order
        return r;
    };
    float m = -INFINITY;
    for (int64_t k = threadIdx.x; k < length; k += blockDim.x) m = fmaxf(m, row[k] * sl2);
    m = block_reduce(m, true);
    float l = 0.0f;
    for (int64_t k = threadIdx.x; k < length; k += blockDim.x) l += exp2f(row[k] * sl2 - m);
    l = block_reduce(l, false);
    const float inv = 1.0f / l;
    for (int64_t k = threadIdx.x; k < length; k += blockDim.x) row[k] = exp2f(row[k] * sl2 - m) * inv;
}

// The same softmax followed by the two-stage quantisation of the row's probabilities over the stored chunks (the first
// n_q columns) into the warp-level product kernel's records (gemm_warp.cuh: [block][group of 8 rows][row][32 fp16] and
// a factor per row and block; blocks from n_q / 32 up to `padded_blocks` are zeros).  Grid: (8 * nt row slots, heads);
// row slots past q_rows only write zero records.  The probabilities are stored (fp32) first and the blocks are
// quantised from what was stored, so the codes are those of the two-kernel route bit for bit.
__global__ void __launch_bounds__(256) kv_softmax_records_kernel(float *__restrict__ S, int64_t ld, int64_t s_stride, int64_t length, float scale,
                                                                 int q_rows, int nt, int n_q, int padded_blocks, uint8_t *__restrict__ rec16,
                                                                 float *__restrict__ recs, int64_t rec_stride) {
    __shared__ float red[8];
    __shared__ SmemTables tab;
    load_tables(tab);
    asm volatile("griddepcontrol.wait;" ::: "memory");           // the scores
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int m = blockIdx.x;                                     // row slot
    rec16 += (int64_t)blockIdx.y * rec_stride;
    recs = (float *)((uint8_t *)recs + (int64_t)blockIdx.y * rec_stride);
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    float *row = S + (int64_t)blockIdx.y * s_stride + (int64_t)m * ld;
    if (m < q_rows) {
        const float sl2 = scale * 1.4426950408889634f;
        auto block_reduce = [&](float v, bool take_max) {
#pragma unroll
            for (int d = 16; d; d >>= 1) {
                const float o = __shfl_xor_sync(0xffffffffu, v, d);
                v = take_max ? fmaxf(v, o) : v + o;
            }
            __syncthreads();
            if (lane == 0) red[warp] = v;
            __syncthreads();
            float r = red[0];
            for (int w = 1; w < 8; w++) r = take_max ? fmaxf(r, red[w]) : r + red[w];
            return r;
        };
        float mx = -INFINITY;
        for (int64_t k = threadIdx.x; k < length; k += blockDim.x) mx = fmaxf(mx, row[k] * sl2);
        mx = block_reduce(mx, true);
        float l = 0.0f;
        for (int64_t k = threadIdx.x; k < length; k += blockDim.x) l += exp2f(row[k] * sl2 - mx);
        l = block_reduce(l, false);
        const float inv = 1.0f / l;
        for (int64_t k = threadIdx.x; k < length; k += blockDim.x) row[k] = exp2f(row[k] * sl2 - mx) * inv;
        __syncthreads();                                          // the blocks below read what other threads stored
    }
    const int nb = n_q / kBlock;
    for (int b = threadIdx.x; b < padded_blocks; b += blockDim.x) {
        uint4 out[4];
#pragma unroll
        for (int i = 0; i < 4; i++) out[i] = make_uint4(0, 0, 0, 0);
        float factor = 1.0f;
        if (m < q_rows && b < nb) {
            uint32_t bits[32], unused[8];
            const uint4 *src = (const uint4 *)(row + (int64_t)b * 32);   // plain loads: this kernel wrote the row
#pragma unroll
            for (int i = 0; i < 8; i++) {
                const uint4 u = src[i];
                bits[4 * i] = u.x; bits[4 * i + 1] = u.y; bits[4 * i + 2] = u.z; bits[4 * i + 3] = u.w;
            }
            BlockResult res;
            bool nonfinite;
            quantize_two_stage_f32<false>(bits, tab, res, unused, nonfinite);
            if (nonfinite) atomicOr(&g_status_word, kStatusNonfinite);
            factor = __uint_as_float(min(res.scale + 22u, 254u) << 23);
            const uint32_t tlo = c_tables.int_lo[res.id], thi = c_tables.int_hi[res.id];
#pragma unroll
            for (int w = 0; w < 4; w++) {
                uint32_t v[4];
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    uint32_t pair = 0;
#pragma unroll
                    for (int j = 0; j < 2; j++) {
                        const int e = 2 * i + j;
                        const uint32_t idx = word_index(res.words[w], e);
                        const uint32_t mag = ((idx < 4 ? tlo : thi) >> (8 * (idx & 3))) & 0xffu;
                        pair |= ((uint32_t)__half_as_ushort(__int2half_rn((int)mag)) | word_sign(res.words[w], e) << 15) << (16 * j);
                    }
                    v[i] = pair;
                }
                out[w] = make_uint4(v[0], v[1], v[2], v[3]);
            }
        }
        const size_t slot = (size_t)(b * nt + m / 8) * 8 + m % 8;
        uint4 *dst = (uint4 *)(rec16 + slot * (kBlock * 2));
#pragma unroll
        for (int i = 0; i < 4; i++) dst[i] = out[i];
        recs[slot] = factor;
    }
}

}  // namespace bd
