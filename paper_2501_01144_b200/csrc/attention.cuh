// Full-path attention on DialectFP4 operands in one kernel (Sec. 4.1, scope "all": the products Q K^T and score x V
// are quantised too; Sec. 3.3: softmax stays in high precision; appendix "Quantization Dimension": Q and K are cut
// into blocks along head_dim, the scores along the keys, V along the tokens).
//
//   S = dq(Q) dq(K)^T * scale            (per head; Q [Sq, d] and K [Sk, d] quantised along d)
//   P = softmax(S) row by row, fp32
//   O = dq(quantise(P)) dq(V)^T          (P quantised online along the keys with the two-stage rule of Sec. 3.2,
//                                         V [d, Sk] quantised along the tokens)
// Neither S nor P is written to memory (unless the caller asks for them, for checking).  The probabilities a block
// of P is quantised from must be the final, normalised ones (the rule is not invariant under the rescaling an
// "online" softmax would apply afterwards), so a CTA walks over the keys twice: first for the row maxima and sums,
// then again for S -> P -> quantise -> accumulate.  Q K^T has only d = 128 deep sums, so the second pass over it is
// cheap next to what writing and re-reading S and P costs.
//
// Arithmetic: warp-level bf16 tensor-core instructions with fp32 accumulators.  Every DialectFP4 value is
// 0.5 * h * 2^e with h <= 15, which bf16 holds exactly, and every product of two of them is exact in fp32, so the
// only rounding is the fp32 accumulation (as in the other product kernels).  A CTA of eight warps owns 128 queries
// of one head; keys come in tiles of 64: their codes are expanded to bf16 tiles in shared memory (K as [key][d],
// V as [channel][key]) and the warps read their operand fragments from there.
//
// Operand fragments use the freedom that the 16 positions of an instruction's K dimension may be any 16 elements
// as long as both operands agree: a thread's positions map to eight consecutive elements of a 32-element block
// (8 t .. 8 t + 7 for lane t of a quad, four per instruction), so one 16-byte shared-memory load feeds two
// instructions, and the keys of a score tile are ordered so that the accumulator a thread ends up with holds
// exactly the eight probabilities (keys 8 t .. 8 t + 7 of a block) it needs as the next product's operand.
#pragma once
#include <cuda_bf16.h>

#include "bd_common.cuh"
#include "quantize.cuh"

namespace bd {
namespace attn {

constexpr int kQTile = 128, kKTile = 64, kWarps = 8, kThreads = 32 * kWarps;

template <int HD>
struct Layout {
    static constexpr int row_stride = HD * 2 + 64;               // bytes between rows of the Q / K tiles: the two rows a
    static constexpr int v_stride = kKTile * 2 + 64;             // quarter-warp reads lie 16 banks apart (same for V)
    static constexpr int q = 0;
    static constexpr int k = q + kQTile * row_stride;
    static constexpr int v = k + kKTile * row_stride;
    static constexpr int total = v + HD * v_stride;
};

constexpr int kMaxHeads = 64, kMaxKvHeads = 32;                // per launch: the operand pointers travel as kernel arguments

struct Params {
    const uint8_t *q_codes[kMaxHeads], *q_ids[kMaxHeads], *q_scales[kMaxHeads];
    const uint8_t *k_codes[kMaxKvHeads], *k_ids[kMaxKvHeads], *k_scales[kMaxKvHeads];
    const uint8_t *v_codes[kMaxKvHeads], *v_ids[kMaxKvHeads], *v_scales[kMaxKvHeads];
    int64_t sq, sk;
    int head0;                 // first head of this launch (results and dumps are indexed by head0 + blockIdx.y)
    int group;                 // query heads per KV head
    float scale;               // softmax scale (1 / sqrt(d) usually)
    void *O;                   // [heads][sq][ldo]
    int64_t ldo, stride_o;
    int out_bf16;
    const uint8_t *k_exp, *v_exp;   // PRE: the KV heads' operands already expanded to bf16 (K [sk][d], V [d][sk]), exp_stride
    int64_t exp_stride;             // bytes from one KV head of this launch to the next
    float *dump_S, *dump_P;    // optional [heads][sq][sk] fp32 (nullptr: not written)
    uint8_t *dump_codes, *dump_ids, *dump_scales;   // optional canonical form of quantise(P): [heads][sq][sk/2], [..][sk/32]
};

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Four E4M3 operand bytes (0.5 * h with the sign in bit 7) -> two registers of bf16 pairs holding the same values
// times 2^-120 (the exponent fields differ by that bias), then scaled to 0.5 * h * 2^e by two exact multiplications.
__device__ __forceinline__ void bytes_to_bf16(uint32_t bytes, __nv_bfloat162 m1, __nv_bfloat162 m2, uint32_t &lo, uint32_t &hi) {
    const uint32_t v0 = __byte_perm(bytes, 0u, 0x1404u), v1 = __byte_perm(bytes, 0u, 0x3424u);   // b0,b1 / b2,b3 into the high bytes
    uint32_t r0 = (v0 & 0x80008000u) | ((v0 >> 4) & 0x07f007f0u), r1 = (v1 & 0x80008000u) | ((v1 >> 4) & 0x07f007f0u);
    __nv_bfloat162 x0 = *(__nv_bfloat162 *)&r0, x1 = *(__nv_bfloat162 *)&r1;
    x0 = __hmul2(__hmul2(x0, m1), m2);
    x1 = __hmul2(__hmul2(x1, m1), m2);
    lo = *(uint32_t *)&x0;
    hi = *(uint32_t *)&x1;
}

// A block of an operand as it comes from memory: its 16 bytes of codes, dialect id and scale byte.  Fetching and
// expanding are separate steps so that a thread's loads of a tile are all issued before the first is used.
struct RawBlock {
    uint4 codes;
    uint32_t id, scale;
    bool valid;
};
__device__ __forceinline__ RawBlock fetch_block(const uint8_t *codes, const uint8_t *ids, const uint8_t *scales, int64_t rows, int64_t ldc,
                                                int64_t nb, int64_t r, int64_t b) {
    RawBlock raw;
    raw.valid = r < rows && b < nb;
    if (raw.valid) {
        raw.codes = __ldg((const uint4 *)(codes + r * ldc + b * 16));
        raw.id = (__ldg(ids + id_byte_offset(rows, r, b)) >> (4 * (b & 1))) & 15u;
        raw.scale = __ldg(scales + scale_offset(rows, r, b));
    }
    return raw;
}
// Expands a block into 32 bf16 values at dst (64 bytes, 16-byte aligned); blocks outside the operand give zeros.
__device__ __forceinline__ void expand_block(const RawBlock &raw, const SmemTables &tab, uint8_t *dst) {
    uint4 out[4];
    if (raw.valid) {
        const uint4 u = raw.codes;
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
        const uint32_t id = raw.id;
        const int e = (int)raw.scale - 127;
        // 2^(e + 120) as two bf16 factors, each inside the normal range
        const int e1 = (e + 120) / 2, e2 = e + 120 - e1;
        const __nv_bfloat162 m1 = __float2bfloat162_rn(__uint_as_float((uint32_t)(e1 + 127) << 23));
        const __nv_bfloat162 m2 = __float2bfloat162_rn(__uint_as_float((uint32_t)(e2 + 127) << 23));
        const uint32_t lut_lo = tab.e4m3_lo[id], lut_hi = tab.e4m3_hi[id];
#pragma unroll
        for (int i = 0; i < 4; i++) {
            uint32_t lo, hi, p0, p1, p2, p3;
            decode_word(w[i], lut_lo, lut_hi, lo, hi);
            bytes_to_bf16(lo, m1, m2, p0, p1);
            bytes_to_bf16(hi, m1, m2, p2, p3);
            out[i] = make_uint4(p0, p1, p2, p3);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 4; i++) out[i] = make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int i = 0; i < 4; i++) *(uint4 *)(dst + 16 * i) = out[i];
}

// The K and V operands of a launch's KV heads expanded once to bf16 (exact: 0.5 h 2^e), for the kernel instantiation
// that copies its key tiles instead of expanding them again for every tile of 128 queries (32 tiles x 4 heads of a
// group share each KV head at the benchmark's shapes).  blockIdx.y = KV head, blockIdx.z = 0: K, 1: V.
template <int HD>
__global__ void __launch_bounds__(256) expand_kv_kernel(const __grid_constant__ Params p, uint8_t *__restrict__ k_exp, uint8_t *__restrict__ v_exp) {
    __shared__ SmemTables tab;
    load_tables(tab);
    const int kvh = blockIdx.y;
    const bool is_v = blockIdx.z != 0;
    const int64_t rows = is_v ? HD : p.sk, nb = is_v ? p.sk / kBlock : HD / kBlock;
    const int64_t task = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (task >= rows * nb) return;
    const int64_t r = task / nb, b = task % nb;
    const uint8_t *codes = is_v ? p.v_codes[kvh] : p.k_codes[kvh], *ids = is_v ? p.v_ids[kvh] : p.k_ids[kvh],
                  *scales = is_v ? p.v_scales[kvh] : p.k_scales[kvh];
    uint8_t *dst = (is_v ? v_exp : k_exp) + (int64_t)kvh * p.exp_stride + (r * nb + b) * 64;
    expand_block(fetch_block(codes, ids, scales, rows, nb * 16, nb, r, b), tab, dst);
}

// Key of accumulator column n (0..7) of score tile j (0..3) inside a block of 32 keys: chosen so that lane t of a quad,
// which owns columns 2 t and 2 t + 1 of every tile, ends up with the keys 8 t .. 8 t + 7 in order.
__device__ __forceinline__ int key_of(int j, int n) { return 8 * (n >> 1) + 2 * j + (n & 1); }

// PRE: the key and value tiles are copied from the bf16 operands expand_kv_kernel wrote, instead of expanded from codes.
template <int HD, bool PRE>
__global__ void __launch_bounds__(kThreads, 2) attention_kernel(const __grid_constant__ Params p) {
    using L = Layout<HD>;
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ SmemTables tab;
    __shared__ uint32_t int_lut[32];                              // half-unit values of a dialect's eight indices, two words per dialect
    load_tables(tab);
    if (threadIdx.x < 32) int_lut[threadIdx.x] = (threadIdx.x & 1) ? c_tables.int_hi[threadIdx.x >> 1] : c_tables.int_lo[threadIdx.x >> 1];
    constexpr int NB = HD / kBlock;                               // blocks along head_dim
    const int hl = blockIdx.y, kvh = hl / p.group, head = p.head0 + hl;   // (a launch starts at a KV-group boundary)
    const int64_t q0 = (int64_t)blockIdx.x * kQTile;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32, g = lane >> 2, t = lane & 3;
    const uint8_t *qc = p.q_codes[hl], *qi = p.q_ids[hl], *qs = p.q_scales[hl];
    const uint8_t *kc = p.k_codes[kvh], *ki = p.k_ids[kvh], *ks = p.k_scales[kvh];
    const uint8_t *vc = p.v_codes[kvh], *vi = p.v_ids[kvh], *vs = p.v_scales[kvh];
    const int64_t nbk = p.sk / kBlock;                            // key blocks of the value operand

    // ---- the CTA's 64 query rows as bf16 ----
    for (int task = threadIdx.x; task < kQTile * NB; task += kThreads) {
        const int r = task / NB, b = task % NB;
        expand_block(fetch_block(qc, qi, qs, p.sq, HD / 2, NB, q0 + r, b), tab, smem + L::q + r * L::row_stride + b * 64);
    }
    // A tile of 64 keys is kKTile * NB key blocks and HD * 2 value blocks: with 256 threads one of each per thread
    // (head_dim 128; half as many key blocks for head_dim 64).
    constexpr int kKTasks = (kKTile * NB + kThreads - 1) / kThreads, kVTasks = (HD * (kKTile / kBlock) + kThreads - 1) / kThreads;
    RawBlock raw_k[kKTasks], raw_v[kVTasks];
    const uint8_t *k_exp = PRE ? p.k_exp + (int64_t)kvh * p.exp_stride : nullptr, *v_exp = PRE ? p.v_exp + (int64_t)kvh * p.exp_stride : nullptr;
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem);
    auto copy16 = [&](uint32_t dst, const uint8_t *src, bool ok) {
        if (ok) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
        else asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
    };
    // PRE: 64 keys x HD bf16 = 16-byte pieces, HD / 8 per key; keys past sk become zeros
    auto copy_k_tile = [&](int64_t key0) {
        for (int c = threadIdx.x; c < kKTile * (HD / 8); c += kThreads) {
            const int r = c / (HD / 8), piece = c % (HD / 8);
            copy16(smem_s + L::k + r * L::row_stride + piece * 16, k_exp + ((key0 + r) * HD + piece * 8) * 2, key0 + r < p.sk);
        }
    };
    // PRE: HD channels x 64 keys bf16 = 8 pieces per channel
    auto copy_v_tile = [&](int64_t key0) {
        for (int c = threadIdx.x; c < HD * (kKTile / 8); c += kThreads) {
            const int ch = c / (kKTile / 8), piece = c % (kKTile / 8);
            copy16(smem_s + L::v + ch * L::v_stride + piece * 16, v_exp + ((int64_t)ch * p.sk + key0 + piece * 8) * 2, key0 + piece * 8 < p.sk);
        }
    };
    auto copies_done = [&]() { asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory"); };
    auto fetch_k_tile = [&](int64_t key0) {
#pragma unroll
        for (int i = 0; i < kKTasks; i++) {
            const int task = threadIdx.x + i * kThreads, r = task / NB, b = task % NB;
            raw_k[i] = fetch_block(kc, ki, ks, task < kKTile * NB ? p.sk : 0, HD / 2, NB, key0 + r, b);
        }
    };
    auto expand_k_tile = [&]() {
#pragma unroll
        for (int i = 0; i < kKTasks; i++) {
            const int task = threadIdx.x + i * kThreads, r = task / NB, b = task % NB;
            if (task < kKTile * NB) expand_block(raw_k[i], tab, smem + L::k + r * L::row_stride + b * 64);
        }
    };
    auto fetch_v_tile = [&](int64_t key0) {
#pragma unroll
        for (int i = 0; i < kVTasks; i++) {
            const int task = threadIdx.x + i * kThreads, ch = task % HD, b = task / HD;   // neighbouring lanes = neighbouring channels
            raw_v[i] = fetch_block(vc, vi, vs, task < HD * (kKTile / kBlock) ? HD : 0, p.sk / 2, nbk, ch, key0 / kBlock + b);
        }
    };
    auto expand_v_tile = [&]() {
#pragma unroll
        for (int i = 0; i < kVTasks; i++) {
            const int task = threadIdx.x + i * kThreads, ch = task % HD, b = task / HD;
            if (task < HD * (kKTile / kBlock)) expand_block(raw_v[i], tab, smem + L::v + ch * L::v_stride + b * 64);
        }
    };
    // ---- scores of this warp's 16 queries against the 32 keys of block kb of the tile in shared memory ----
    // s[j][0..3]: (row g, keys 8t+2j, 8t+2j+1), (row g+8, same keys)
    const uint8_t *my_q = smem + L::q + (warp * 16 + g) * L::row_stride + t * 16;
    auto scores = [&](int kb, float (&s)[4][4]) {
#pragma unroll
        for (int j = 0; j < 4; j++) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.0f;
#pragma unroll
        for (int b = 0; b < NB; b++) {
            const uint4 a_lo = *(const uint4 *)(my_q + b * 64), a_hi = *(const uint4 *)(my_q + 8 * L::row_stride + b * 64);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                const uint4 kf = *(const uint4 *)(smem + L::k + (kb * 32 + key_of(j, g)) * L::row_stride + b * 64 + t * 16);
                mma_bf16(s[j], a_lo.x, a_hi.x, a_lo.y, a_hi.y, kf.x, kf.y);
                mma_bf16(s[j], a_lo.z, a_hi.z, a_lo.w, a_hi.w, kf.z, kf.w);
            }
        }
    };
    const float sl2 = p.scale * 1.4426950408889634f;             // scores in units of log2 e: exp(x) = exp2(x * log2 e)
    const int64_t row_lo = q0 + warp * 16 + g, row_hi = row_lo + 8;

    // ---- first walk over the keys: row maxima and sums ----
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.0f, l_hi = 0.0f;
    for (int64_t key0 = 0; key0 < p.sk; key0 += kKTile) {
        __syncthreads();                                          // the previous tile has been used
        if (PRE) {
            copy_k_tile(key0);
            copies_done();
        } else {
            fetch_k_tile(key0);
            expand_k_tile();
        }
        __syncthreads();
#pragma unroll
        for (int kb = 0; kb < kKTile / kBlock; kb++) {
            if (key0 + kb * 32 >= p.sk) break;                    // (whole blocks: sk is a multiple of 32)
            float s[4][4];
            scores(kb, s);
            float mx_lo = m_lo, mx_hi = m_hi;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                mx_lo = fmaxf(mx_lo, fmaxf(s[j][0], s[j][1]) * sl2);
                mx_hi = fmaxf(mx_hi, fmaxf(s[j][2], s[j][3]) * sl2);
            }
            float add_lo = 0.0f, add_hi = 0.0f;
#pragma unroll
            for (int j = 0; j < 4; j++) {
                add_lo += exp2f(s[j][0] * sl2 - mx_lo) + exp2f(s[j][1] * sl2 - mx_lo);
                add_hi += exp2f(s[j][2] * sl2 - mx_hi) + exp2f(s[j][3] * sl2 - mx_hi);
            }
            l_lo = l_lo * exp2f(m_lo - mx_lo) + add_lo;
            l_hi = l_hi * exp2f(m_hi - mx_hi) + add_hi;
            m_lo = mx_lo;
            m_hi = mx_hi;
        }
    }
    // the four lanes of a quad saw different keys of the same rows
#pragma unroll
    for (int d = 1; d <= 2; d <<= 1) {
        const float om_lo = __shfl_xor_sync(0xffffffffu, m_lo, d), ol_lo = __shfl_xor_sync(0xffffffffu, l_lo, d);
        const float om_hi = __shfl_xor_sync(0xffffffffu, m_hi, d), ol_hi = __shfl_xor_sync(0xffffffffu, l_hi, d);
        const float nm_lo = fmaxf(m_lo, om_lo), nm_hi = fmaxf(m_hi, om_hi);
        l_lo = l_lo * exp2f(m_lo - nm_lo) + ol_lo * exp2f(om_lo - nm_lo);
        l_hi = l_hi * exp2f(m_hi - nm_hi) + ol_hi * exp2f(om_hi - nm_hi);
        m_lo = nm_lo;
        m_hi = nm_hi;
    }
    const float inv_lo = 1.0f / l_lo, inv_hi = 1.0f / l_hi;

    // ---- second walk: S -> P -> quantise along the keys -> O += P V ----
    float o[HD / 8][4];
#pragma unroll
    for (int n = 0; n < HD / 8; n++) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.0f;
    const int64_t dump_row_lo = ((int64_t)head * p.sq + row_lo), dump_row_hi = dump_row_lo + 8;
    for (int64_t key0 = 0; key0 < p.sk; key0 += kKTile) {
        __syncthreads();
        if (PRE) {
            copy_k_tile(key0);
            copy_v_tile(key0);
            copies_done();
        } else {
            fetch_k_tile(key0);                                   // (keeping the next tile's blocks in registers through the
            fetch_v_tile(key0);                                   // products, to hide this latency, costs more in spills)
            expand_k_tile();
            expand_v_tile();
        }
        __syncthreads();
#pragma unroll
        for (int kb = 0; kb < kKTile / kBlock; kb++) {
            if (key0 + kb * 32 >= p.sk) break;
            float s[4][4];
            scores(kb, s);
            const int64_t kbase = key0 + kb * 32 + 8 * t;         // this lane's eight keys
            // probabilities of this lane's eight keys, both rows
            float pr[2][8];
#pragma unroll
            for (int j = 0; j < 4; j++) {
                pr[0][2 * j] = exp2f(s[j][0] * sl2 - m_lo) * inv_lo;
                pr[0][2 * j + 1] = exp2f(s[j][1] * sl2 - m_lo) * inv_lo;
                pr[1][2 * j] = exp2f(s[j][2] * sl2 - m_hi) * inv_hi;
                pr[1][2 * j + 1] = exp2f(s[j][3] * sl2 - m_hi) * inv_hi;
            }
            if (p.dump_S) {
#pragma unroll
                for (int j = 0; j < 4; j++) {
                    if (row_lo < p.sq) *(float2 *)(p.dump_S + dump_row_lo * p.sk + kbase + 2 * j) = make_float2(s[j][0] * p.scale, s[j][1] * p.scale);
                    if (row_hi < p.sq) *(float2 *)(p.dump_S + dump_row_hi * p.sk + kbase + 2 * j) = make_float2(s[j][2] * p.scale, s[j][3] * p.scale);
                }
            }
            // two-stage rule (Sec. 3.2) on the block of 32 probabilities of each row, eight per lane of the quad
            uint32_t a_frag[2][4];                                // operand registers of the next product, per row
#pragma unroll
            for (int h = 0; h < 2; h++) {
                uint32_t amax = 0;
#pragma unroll
                for (int i = 0; i < 8; i++) amax = max(amax, __float_as_uint(pr[h][i]));      // probabilities are >= 0
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
                amax = max(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
                const uint32_t eadj = max(amax >> 23, 2u);
                // The quantizer's packed arithmetic on this lane's eight elements (one code word of the block): the
                // number of merged thresholds of the dialect pair above each 5-bit code, as nibbles; range counts by
                // byte-permute lookup, summed over the quad; indices by nibble-parallel arithmetic (finish_two_stage).
                float pv8[8];
                uint32_t eadj_eff = eadj;
                float amax_f = __uint_as_float(amax);
#pragma unroll
                for (int i = 0; i < 8; i++) pv8[i] = pr[h][i];
                if (eadj < 4u) {                                  // block at the exponent clamp: 2^(131 - eadj) is no fp32
#pragma unroll
                    for (int i = 0; i < 8; i++) pv8[i] *= 18446744073709551616.0f;
                    amax_f *= 18446744073709551616.0f;
                    eadj_eff = eadj + 64u;
                }
                const float q_scale = __uint_as_float((258u - eadj_eff) << 23);      // 2^(2 - e), e = eadj - 129
                const uint32_t m5 = __float_as_uint(__fmaf_rz(amax_f, q_scale, 8388608.0f)) & 63u;
                const uint32_t pair = min(7u, 15u - min(15u, (m5 + 1u) >> 1));
                const uint32_t above = tab.merged_above[pair];
                uint32_t v = 0;
#pragma unroll
                for (int i = 0; i < 8; i++) {
                    const uint32_t tq = __float_as_uint(__fmaf_rz(pv8[i], q_scale, 8388608.0f));
                    v = (uint32_t)__popc(__funnelshift_r(above, 0u, tq)) * (1u << (4 * i)) + v;
                }
                const uint32_t acc = prmt_b32(0x10010100u, 0x00000010u, v) + prmt_b32(0x10010100u, 0x00000010u, v >> 16);
                uint32_t cnt = byte_sum(acc & 0x0f0f0f0fu) | byte_sum((acc >> 4) & 0x0f0f0f0fu) << 16;   // even | odd << 16
                cnt += __shfl_xor_sync(0xffffffffu, cnt, 1);
                cnt += __shfl_xor_sync(0xffffffffu, cnt, 2);
                const uint32_t odd = (cnt >> 16) > (cnt & 0xffffu) ? 1u : 0u;                  // equal counts: the even member
                const uint32_t id = 2u * pair + odd;
                const uint32_t first_step = odd ? 0x11111111u : 0x22222222u, odd_mask = 0u - odd;
                const uint32_t u = 0xaaaaaaaau - v;
                const uint32_t b3 = (u >> 3) & 0x11111111u, b1 = (u >> 1) & 0x11111111u, b0 = u & 0x11111111u;
                const uint32_t f = ((u + first_step) >> 3) & 0x11111111u;
                const uint32_t top = b3 & (b1 | (b0 & ~odd_mask));
                const uint32_t codes = u - f - b3 - top;           // index of element i in nibble i (probabilities carry no sign)
                // values 0.5 h 2^e = h * unit as bf16: the half-unit integers through the dialect's byte table, each
                // byte under the high byte 0x43 is the bf16 number 128 + h, and (128 + h) * unit - 128 * unit is exact
                const uint32_t h_lo = prmt_b32(int_lut[2 * id], int_lut[2 * id + 1], codes), h_hi = prmt_b32(int_lut[2 * id], int_lut[2 * id + 1], codes >> 16);
                const float unit = __uint_as_float((uint32_t)max((int)eadj - 130 + 127, 0) << 23);
                const __nv_bfloat162 unit2 = __float2bfloat162_rn(unit), off2 = __float2bfloat162_rn(-128.0f * unit);
                const uint32_t raw4[4] = {prmt_b32(h_lo, 0x43434343u, 0x4140u), prmt_b32(h_lo, 0x43434343u, 0x4342u),
                                          prmt_b32(h_hi, 0x43434343u, 0x4140u), prmt_b32(h_hi, 0x43434343u, 0x4342u)};
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    const __nv_bfloat162 pk = __hfma2(*(const __nv_bfloat162 *)&raw4[i], unit2, off2);
                    a_frag[h][i] = *(const uint32_t *)&pk;
                }
                const int64_t drow = h ? dump_row_hi : dump_row_lo;
                if ((h ? row_hi : row_lo) < p.sq) {
                    if (p.dump_P) {
#pragma unroll
                        for (int i = 0; i < 8; i += 2) *(float2 *)(p.dump_P + drow * p.sk + kbase + i) = make_float2(pr[h][i], pr[h][i + 1]);
                    }
                    if (p.dump_codes) {
                        *(uint32_t *)(p.dump_codes + drow * (p.sk / 2) + kbase / 2) = codes;
                        if (t == 0) {
                            p.dump_ids[drow * nbk + (key0 / 32 + kb)] = (uint8_t)id;
                            p.dump_scales[drow * nbk + (key0 / 32 + kb)] = (uint8_t)(eadj - 2u);
                        }
                    }
                }
            }
            // O[16 queries][HD] += P[16 x 32 keys] V^T: two instructions per eight channels
#pragma unroll
            for (int n = 0; n < HD / 8; n++) {
                const uint4 vf = *(const uint4 *)(smem + L::v + (8 * n + g) * L::v_stride + kb * 64 + t * 16);
                mma_bf16(o[n], a_frag[0][0], a_frag[1][0], a_frag[0][1], a_frag[1][1], vf.x, vf.y);
                mma_bf16(o[n], a_frag[0][2], a_frag[1][2], a_frag[0][3], a_frag[1][3], vf.z, vf.w);
            }
        }
    }
    // ---- result: rows g and g + 8 of the warp's 16 queries, channels 8 n + 2 t, + 1 ----
    uint8_t *out = (uint8_t *)p.O;
    const int esz = p.out_bf16 ? 2 : 4;
#pragma unroll
    for (int n = 0; n < HD / 8; n++) {
        const int ch = 8 * n + 2 * t;
        if (row_lo < p.sq) {
            uint8_t *dst = out + ((int64_t)head * p.stride_o + row_lo * p.ldo + ch) * esz;
            if (p.out_bf16) *(__nv_bfloat162 *)dst = __floats2bfloat162_rn(o[n][0], o[n][1]);
            else *(float2 *)dst = make_float2(o[n][0], o[n][1]);
        }
        if (row_hi < p.sq) {
            uint8_t *dst = out + ((int64_t)head * p.stride_o + row_hi * p.ldo + ch) * esz;
            if (p.out_bf16) *(__nv_bfloat162 *)dst = __floats2bfloat162_rn(o[n][2], o[n][3]);
            else *(float2 *)dst = make_float2(o[n][2], o[n][3]);
        }
    }
}

}  // namespace attn
}  // namespace bd
