/*
 * libblockdialect: BlockDialect W4A4 quantized linear layer for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every tensor pointer is a DEVICE pointer owned by the caller unless a
 * parameter says "host".  `stream` is a cudaStream_t passed as void* (NULL = the
 * legacy default stream).  Calls enqueue work on the stream and return; argument
 * errors are reported synchronously through the return value and nothing is
 * enqueued.  Device-side conditions (non-finite input, an expired bounded wait)
 * are recorded in a device status word that bd_poll_status reads.  The library
 * never allocates or frees device memory on these paths: scratch is passed in as
 * `workspace` (sizes from the *_workspace_size calls).  There is no CPU fallback.
 *
 * Threads: the library keeps a few unsynchronised host-side globals (launch counter,
 * last CUDA error, implementation choice, per-device caches filled on first use), so
 * it is NOT thread-safe: serialise calls into it, or make every call from one thread.
 * bd_get_formatbook reports the table of the last successful bd_set_formatbook of the
 * process; the device tables are per device, so set the same table on every device
 * that is used.
 *
 * The method (arXiv 2501.01144, "BlockDialect"):
 *   - operands are cut into blocks of 32 consecutive elements along the
 *     multiplication dimension K (Sec. 3.1; Appendix "Quantization Dimension");
 *   - each block stores a shared power-of-two exponent e = floor(log2 max|x|) - 2
 *     (Sec. 3.1), a 4-bit dialect id into the 16-entry DialectFP4 formatbook
 *     (Sec. 3.1, Fig. 4) and, per element, a sign bit and a 3-bit index into the
 *     dialect's eight magnitudes 0.5 * {0..15} (Sec. 3.1, Sec. 3.3);
 *   - a product of two operands sums 4-bit integer products exactly inside a
 *     block and rescales once per block by 2^(eA + eB - 2) (Sec. 3.3, Fig. 6).
 */
#ifndef BD_H
#define BD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BD_OK = 0,
    BD_ERR_INVALID_ARG = 1, /* null pointer, negative size, bad enum                      */
    BD_ERR_SHAPE = 2,       /* K not a multiple of 32, operand shapes disagree, ld < K    */
    BD_ERR_ALIGN = 3,       /* pointer or leading dimension not 16-byte aligned           */
    BD_ERR_UNSUPPORTED = 4, /* combination not implemented                                */
    BD_ERR_CUDA = 5,        /* a CUDA call failed; bd_last_cuda_error gives the code      */
    BD_ERR_NONFINITE = 6,   /* Inf/NaN met by a quantizer (from bd_poll_status)           */
    BD_ERR_TIMEOUT = 7,     /* a bounded device-side wait expired (from bd_poll_status)   */
    BD_ERR_WORKSPACE = 8,   /* workspace missing or too small                             */
    BD_ERR_SCRATCH_LIMIT = 9 /* bd_linear_noalloc: the problem needs more scratch than the
                                library's built-in buffer holds                             */
} bd_status;

typedef enum { BD_F32 = 0, BD_BF16 = 1, BD_F16 = 2 } bd_dtype;

/* Dialect selection rule.
 * BD_SELECT_TWO_STAGE: the online rule of Sec. 3.2 (Fig. 5): stage 1 picks the
 *   dialect pair whose maximum equals the block maximum rounded to the 0.5 grid,
 *   stage 2 the member of the pair with more block elements inside its beneficial
 *   range (equal counts: the even-numbered dialect).
 * BD_SELECT_MSE: the offline rule for weights (Sec. 3.2 first paragraph, Sec. 4.3):
 *   the dialect with the smallest exact squared error over all 16, lowest id on
 *   equal error; errors are summed in fp64 in element order.                        */
typedef enum { BD_SELECT_TWO_STAGE = 0, BD_SELECT_MSE = 1 } bd_select;

/* Which axis of the source the blocks run along.
 * BD_AXIS_CONTIG:  source is [rows, K] with K contiguous (activations per token,
 *                  weights per output channel, Q and K per head dimension).
 * BD_AXIS_STRIDED: source is [K, rows] with `rows` contiguous and blocks made of 32
 *                  consecutive source rows (the value matrix V, quantised along the
 *                  token axis; Appendix "Quantization Dimension").  The result is the
 *                  quantised TRANSPOSE: a [rows, K] operand.                         */
typedef enum { BD_AXIS_CONTIG = 0, BD_AXIS_STRIDED = 1 } bd_axis;

/* GEMM implementation choice (bd_set_gemm_impl). */
typedef enum {
    BD_GEMM_AUTO = 0,   /* by shape                                                    */
    BD_GEMM_SIMT = 1,   /* CUDA-core kernel: exact integer in-block sums, any shape     */
    BD_GEMM_TCGEN05 = 2, /* tensor-core kernel (block-scaled E4M3 MMA, TMEM accumulators) */
    BD_GEMM_WARP = 3    /* products with at most 16 rows on the activation side (bd_linear of at most 16
                           tokens, bd_gemm with A->rows <= 16, the KV-cache calls): warp-level fp16 MMA
                           straight from the packed B operand, one launch after the kernel that prepares
                           A, no partial sums in memory; BD_ERR_UNSUPPORTED for more rows */
} bd_gemm_impl;

/* A quantised [rows, K] operand in the library's physical layout.  All three
 * buffers are caller-allocated device memory of the sizes bd_qtensor_sizes
 * returns; the library never frees them.  The layout is opaque (it is arranged
 * for bulk copies into shared memory and for the tensor-core scale-factor
 * format); bd_export_canonical converts it to the documented canonical layout. */
typedef struct {
    void *codes;   /* 4 bits per element                                  */
    void *ids;     /* 4 bits per block                                    */
    void *scales;  /* 8 bits per block: e + 127                           */
    int64_t rows;
    int64_t K;
} bd_qtensor;

/* Buffer sizes in bytes for a [rows, K] operand.  K must be a multiple of 32. */
bd_status bd_qtensor_sizes(int64_t rows, int64_t K, size_t *codes_bytes, size_t *ids_bytes,
                           size_t *scales_bytes);

/* Offline weight quantisation (Sec. 3.3 "the optimal dialect for each block is
 * precomputed").  W: [N, K] of `dtype`, row stride ldw elements, blocks along K.
 * out->rows must be N and out->K must be K. */
bd_status bd_quantize_weights(const void *W, bd_dtype dtype, int64_t N, int64_t K, int64_t ldw,
                              bd_select select, bd_qtensor *out, void *stream);

/* Online activation quantisation with the two-stage rule (Sec. 3.2, Sec. 3.3):
 * per block absmax -> shared exponent, 5-bit truncated magnitudes, pair by rounded
 * block maximum, dialect by beneficial-range counts, round-to-nearest (ties to the
 * larger magnitude) onto the dialect's grid, 4-bit codes.
 * BD_AXIS_CONTIG:  X is [M, K], row stride ldx.  out is [M, K].
 * BD_AXIS_STRIDED: X is [K, M], row stride ldx.  out is [M, K] (the transpose).
 * X and ldx*sizeof(element) must be 16-byte aligned. */
bd_status bd_quantize_act(const void *X, bd_dtype dtype, int64_t M, int64_t K, int64_t ldx,
                          bd_axis axis, bd_qtensor *out, void *stream);

/* Y[M,N] = dq(A)[M,K] * dq(B)[N,K]^T (Sec. 3.3, Fig. 6).  ydtype is BD_F32 or BD_BF16
 * (bf16 = round-to-nearest-even of the fp32 accumulator); ldy = row stride of Y in
 * elements.  workspace: bd_gemm_workspace_size bytes, 256-byte aligned, or NULL when
 * that size is 0.
 *
 * Accuracy of the fp32 result against the exact product, per output element, with
 * S = sum_k |a_k| |b_k| over the dequantised operands (bd_gemm, bd_gemm_batched and
 * bd_linear alike):
 *   BD_GEMM_SIMT      in-block sums are exact integers and blocks are added in fp64:
 *                     |err| <= 2^-24 * |y| (the final rounding to fp32) for any input.
 *   BD_GEMM_TCGEN05   one block-scaled tensor-core instruction per block of 32; each
 *                     aligns its 32 products and the running fp32 sum to the largest
 *                     exponent among them, drops bits below 2^-25 of it and truncates
 *                     the sum to fp32.  When the block scales met along a row of K lie
 *                     within a factor 2^24 of each other, as activations and weights
 *                     of a layer do, the result is exact or within about 1e-8 * S;
 *                     the guaranteed bound for ANY input is (K / 32) * 2^-21 * S (an
 *                     operand with blocks 2^28 apart and opposite signs gets close to
 *                     it).  Callers who need 1e-6 * S on such inputs select BD_GEMM_SIMT.
 *   BD_GEMM_WARP      (at most 16 rows of A) in-block sums are exact (fp16 tensor-core
 *                     products of 4-bit integers, fp32 sums of 32 of them); each block's sum is
 *                     multiplied by its two power-of-two scales one after the other and the blocks
 *                     are added in fp32, the warps' shares of K in a fixed order: |err| <=
 *                     (K / 32 + 16) * 2^-24 * S.  Blocks whose scale lies below 2^-100 or above
 *                     2^100 may be flushed or overflow in the intermediate product.
 *   BD_GEMM_AUTO      picks BD_GEMM_TCGEN05 except for tiny problems, and BD_GEMM_WARP for at most
 *                     8 rows of A (at most 16 against up to 2^25 elements of B); the chosen
 *                     implementation's bound applies. */
bd_status bd_gemm_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes);
bd_status bd_gemm(const bd_qtensor *A, const bd_qtensor *B, void *Y, bd_dtype ydtype, int64_t ldy,
                  void *workspace, size_t workspace_bytes, void *stream);

/* Batched product for attention (Appendix "Quantization Dimension"): `batch`
 * independent products; operand b of A uses operand b / b_group of B (grouped-query
 * attention shares one K/V head among b_group query heads).  A points to `batch`
 * descriptors, B to batch / b_group descriptors (host arrays); Y + b * stride_y
 * elements is product b.  All operands of A share one shape, all of B another
 * (checked: BD_ERR_SHAPE otherwise).
 * With a workspace of bd_gemm_batched_workspace_size bytes, results of a group that
 * are contiguous in Y (stride_y == M * ldy) and M a multiple of 128, the b_group
 * products of a group run as one stacked launch; otherwise (any workspace of at
 * least bd_gemm_workspace_size bytes) one launch per product.  With at most 16 rows
 * per A operand (where BD_GEMM_WARP serves the call) all products share launches of
 * up to 64, whatever the strides; no workspace is touched then. */
bd_status bd_gemm_batched_workspace_size(int64_t M, int64_t N, int64_t K, int64_t b_group, size_t *bytes);
bd_status bd_gemm_batched(const bd_qtensor *A, const bd_qtensor *B, int64_t batch, int64_t b_group,
                          void *Y, bd_dtype ydtype, int64_t ldy, int64_t stride_y, void *workspace,
                          size_t workspace_bytes, void *stream);

/* The quantised linear layer: quantise X [M,K] online (two-stage rule), then
 * Y = dq(X) * dq(Wq)^T.  The quantised activation lives only in `workspace`.
 * The call is two or three kernel launches on `stream` (quantizer, product, and for
 * short calls with few weight rows a kernel that adds partial sums kept in the
 * workspace), linked by programmatic dependent launch: each starts while its
 * predecessor drains and waits for it before touching its results; work queued
 * behind the call in the usual way sees it complete.  After one call per device
 * (which sets function attributes) further calls can be captured into a CUDA graph. */
bd_status bd_linear_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes);
bd_status bd_linear(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx,
                    const bd_qtensor *Wq, void *Y, bd_dtype ydtype, int64_t ldy, void *workspace,
                    size_t workspace_bytes, void *stream);

/* Products whose result stays in DialectFP4 (Sec. 3.3, last paragraph: the accumulated
 * partial sums are "requantized into 4-bit DialectFP4 format for the next matrix
 * multiplication").  Instead of Y [M, N] the call writes Yq, the quantised operand
 * [M rows, N along its K axis] that quantising the fp32 result row by row with the online
 * two-stage rule (bd_quantize_act, BD_AXIS_CONTIG) would give: bit for bit the same codes,
 * ids and scales.  N must be a multiple of 32; Yq->rows = M, Yq->K = N.  Yq then feeds the
 * next layer through bd_gemm / bd_gemm_requant, and no high-precision Y is written.
 * With more than 128 tokens on the tensor-core route the requantisation runs in the
 * product kernel's epilogue on the fp32 accumulators; otherwise the fp32 result is parked
 * in the workspace and the quantizer kernel follows (same result).  The workspace sizes
 * depend on the implementation chosen with bd_set_gemm_impl: ask after choosing. */
bd_status bd_linear_requant_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes);
bd_status bd_linear_requant(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx,
                            const bd_qtensor *Wq, bd_qtensor *Yq, void *workspace,
                            size_t workspace_bytes, void *stream);
bd_status bd_gemm_requant_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes);
bd_status bd_gemm_requant(const bd_qtensor *A, const bd_qtensor *B, bd_qtensor *Yq, void *workspace,
                          size_t workspace_bytes, void *stream);

/* Block sizes 16 and 64 beside the default 32 (the block-size study of Sec. 4.2 and its
 * Table 3, including per-sublayer mixes such as block 16 for the down projection: the block
 * size is chosen per call).  `block` is 16, 32 or 64 and must divide K; both operands of a
 * product use the same block size.  The tensor-core product scales per 32 elements, so other
 * block sizes are STORED in the ordinary 32-block form and every product entry point
 * (bd_gemm, bd_gemm_batched, bd_gemm_requant) takes such operands as they are, exactly:
 *   block 64: two neighbouring 32-blocks with the same scale and id; physical K' = K;
 *   block 16: one 32-block per block, its second half zero codes; physical K' = 2 K
 *             (twice the code bytes and twice the MMA work of the same K at block 32).
 * bd_qtensor_sizes_bs gives the buffer sizes; out->K must be the physical K'.
 * bd_export_canonical_bs gives the canonical view: codes [rows][K/2], ids and scales
 * [rows][K/block].  bd_linear_bs = two-stage quantisation of X with that block size
 * (into the workspace) followed by the product with Wq (quantised with the same block size). */
bd_status bd_qtensor_sizes_bs(int64_t rows, int64_t K, int block, size_t *codes_bytes, size_t *ids_bytes,
                              size_t *scales_bytes);
bd_status bd_quantize_bs(const void *X, bd_dtype dtype, int64_t rows, int64_t K, int64_t ld, bd_select select,
                         int block, bd_qtensor *out, void *stream);
bd_status bd_export_canonical_bs(const bd_qtensor *q, int block, uint8_t *codes, uint8_t *ids, uint8_t *scales,
                                 void *stream);
bd_status bd_linear_bs_workspace_size(int64_t M, int64_t N, int64_t K, int block, size_t *bytes);
bd_status bd_linear_bs(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, int block,
                       const bd_qtensor *Wq, void *Y, bd_dtype ydtype, int64_t ldy, void *workspace,
                       size_t workspace_bytes, void *stream);

/* KV cache of one KV head (appendix "Quantization Dimension", Fig. 9b).  Keys are quantised
 * sub-token-wise (along head_dim) when they arrive and appended as rows of the key operand
 * k [capacity, head_dim].  Values are quantised sub-channel-wise, along the token axis: the
 * value operand is v [head_dim, capacity] with blocks of 32 consecutive tokens per channel.
 * Such a block cannot take a single new token, so the newest (length mod 32) value rows are
 * kept in high precision in v_recent (the source type, [32, head_dim]) and are quantised
 * once, as a whole chunk, when 32 are there; nothing stored is requantised.
 * All buffers are caller-allocated device memory: k and v as bd_qtensor_sizes(capacity,
 * head_dim) and (head_dim, capacity) say, v_recent as bd_kvcache_recent_bytes.  head_dim is
 * a multiple of 32, at most 128; capacity a multiple of 32.  `length` is host state that
 * bd_kvcache_append advances (the struct is not thread-safe).  Call bd_kvcache_reset once
 * before the first append (it clears scales and ids and sets length = 0).
 *   bd_kvcache_append   t new tokens: Knew, Vnew [t, head_dim] of the cache's dtype.
 *   bd_kvcache_scores   S [q, length] = dq(Q) dq(K)^T for a quantised query operand Q [q, head_dim].
 *   bd_kvcache_pv       O [q, head_dim] = P V for fp32 probabilities P [q, length]: the columns
 *                       over stored chunks are quantised online along the keys and multiplied with
 *                       the 4-bit values; the columns of the recent tokens are multiplied in fp32
 *                       with the high-precision rows.  Once a chunk is stored, P and its row
 *                       pitch (ldp * 4 bytes) must be 16-byte aligned.
 * workspace: bd_kvcache_workspace_size(capacity, head_dim, q) bytes, 256-byte aligned. */
typedef struct {
    bd_qtensor k;       /* [capacity, head_dim]                      */
    bd_qtensor v;       /* [head_dim, capacity]                      */
    void *v_recent;     /* [32, head_dim] elements of `dtype`        */
    bd_dtype dtype;     /* type of the key / value rows handed in    */
    int64_t capacity, head_dim, length;
} bd_kvcache;
bd_status bd_kvcache_recent_bytes(int64_t head_dim, bd_dtype dtype, size_t *bytes);
bd_status bd_kvcache_reset(bd_kvcache *c, void *stream);
bd_status bd_kvcache_append(bd_kvcache *c, const void *Knew, const void *Vnew, int64_t t, int64_t ldk, int64_t ldv,
                            void *stream);
bd_status bd_kvcache_workspace_size(int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes);
bd_status bd_kvcache_scores(const bd_kvcache *c, const bd_qtensor *Q, void *S, bd_dtype sdtype, int64_t lds,
                            void *workspace, size_t workspace_bytes, void *stream);
bd_status bd_kvcache_pv(const bd_kvcache *c, const float *P, int64_t q_rows, int64_t ldp, void *Y, bd_dtype ydtype,
                        int64_t ldy, void *workspace, size_t workspace_bytes, void *stream);
/* The same two calls for the n KV heads of a layer in one decode step (n >= 1): c[i] all of one capacity,
 * head_dim, dtype and length; Q[i] [q, head_dim] with the same q; head i reads P + i * stride_p and writes
 * S + i * stride_s / Y + i * stride_y, and takes its t new tokens from Knew + i * stride_k, Vnew + i * stride_v
 * (strides in elements; every head's length advances by t).  With q <= 16 and n <= 64 (and the library's own
 * choice of product kernel) the heads share one (scores) or two (P x V) launches; otherwise the calls
 * above run head by head.  BD_ERR_SHAPE when the heads differ in capacity, head_dim, dtype or length, or the strides
 * are shorter than a head's rows; otherwise the errors of the one-head calls.  workspace:
 * bd_kvcache_batched_workspace_size bytes, 256-byte aligned. */
bd_status bd_kvcache_append_batched(bd_kvcache *c, int64_t n, const void *Knew, const void *Vnew, int64_t t, int64_t ldk,
                                    int64_t ldv, int64_t stride_k, int64_t stride_v, void *stream);
bd_status bd_kvcache_batched_workspace_size(int64_t n, int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes);
bd_status bd_kvcache_scores_batched(const bd_kvcache *c, int64_t n, const bd_qtensor *Q, void *S, bd_dtype sdtype,
                                    int64_t lds, int64_t stride_s, void *workspace, size_t workspace_bytes, void *stream);
bd_status bd_kvcache_pv_batched(const bd_kvcache *c, int64_t n, const float *P, int64_t q_rows, int64_t ldp,
                                int64_t stride_p, void *Y, bd_dtype ydtype, int64_t ldy, int64_t stride_y,
                                void *workspace, size_t workspace_bytes, void *stream);
/* Attention of one decode step over the cached heads (Sec. 4.1 scope "all", Sec. 3.3): per head i
 *     S = dq(Q[i]) dq(K_i)^T,  P = softmax(scale * S) row by row in fp32,  O_i = P V_i as in bd_kvcache_pv.
 * O + i * stride_o is [q, head_dim] with row pitch ldo.  P_out, when not NULL, receives the fp32 probabilities
 * (head i at P_out + i * stride_p_out, pitch ldp_out >= length; 16-byte aligned pointer and pitches) and is the
 * buffer the second product reads; with NULL they stay in the workspace.  Three launches where the batched calls
 * above share theirs (scores; softmax, which also prepares the second product's operand; P x V), else those calls
 * and a softmax kernel.  workspace: bd_kvcache_attention_workspace_size bytes, 256-byte aligned. */
bd_status bd_kvcache_attention_workspace_size(int64_t n, int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes);
bd_status bd_kvcache_attention(const bd_kvcache *c, int64_t n, const bd_qtensor *Q, float scale, void *O, bd_dtype odtype,
                               int64_t ldo, int64_t stride_o, float *P_out, int64_t ldp_out, int64_t stride_p_out,
                               void *workspace, size_t workspace_bytes, void *stream);

/* Full-path attention in one kernel (Sec. 4.1, scope "all": Q K^T and score x V are quantised
 * like the linear layers; Sec. 3.3: softmax stays in high precision; appendix "Quantization
 * Dimension": Q and K are cut into blocks along head_dim, the probabilities along the keys, V
 * along the tokens).  Per head h:
 *     S = dq(Q[h]) dq(K[h / group])^T * scale
 *     P = softmax(S) row by row in fp32
 *     O[h] = dq(quantise(P)) dq(V[h / group])^T     (P quantised with the online two-stage rule)
 * Q: `heads` operands [Sq, d] (bd_quantize_act, BD_AXIS_CONTIG); K: heads / group operands
 * [Sk, d]; V: heads / group operands [d, Sk] (bd_quantize_act of V [Sk, d] with BD_AXIS_STRIDED).
 * Q, K, V are host arrays of descriptors.  d is 64 or 128; Sk a multiple of 32.  O is
 * [heads][Sq][ldo] with stride_o elements between heads, BD_F32 or BD_BF16.  No mask.
 * Neither S nor P goes to memory; the keys are walked twice (row maxima and sums first), because
 * the blocks of P must be quantised from the final probabilities.  With `dump` (for checking;
 * any member may be NULL) the kernel also writes S and P as fp32 [heads][Sq][Sk] and the
 * canonical codes [heads][Sq][Sk/2], ids and scales [heads][Sq][Sk/32] of the quantised P.
 * With a workspace (bd_attention_workspace_size bytes, 256-byte aligned; NULL: none) the K and V operands of
 * the launch's KV heads are first expanded to bf16 there, once, and the kernel copies its key tiles from that
 * instead of expanding the codes again for every tile of 128 queries; the results are the same bit for bit.
 * Accuracy: as the tensor-core product (fp32 accumulation of exact products). */
typedef struct {
    float *S, *P;
    uint8_t *codes, *ids, *scales;
} bd_attention_dump;
bd_status bd_attention_workspace_size(int64_t heads, int64_t group, int64_t sk, int64_t head_dim, size_t *bytes);
bd_status bd_attention(const bd_qtensor *Q, const bd_qtensor *K, const bd_qtensor *V, int64_t heads, int64_t group,
                       float scale, void *O, bd_dtype odtype, int64_t ldo, int64_t stride_o,
                       const bd_attention_dump *dump, void *workspace, size_t workspace_bytes, void *stream);

/* bd_linear for callers that can neither allocate device memory nor hand in a
 * workspace (the paper has no counterpart; this is a convenience of the library).
 * Think of code that runs where cudaMalloc is off limits: inside a region whose
 * memory plan is already frozen, in a plugin that was given only its input and
 * output tensors, or under a memory pool that forbids side allocations.  The
 * scratch that bd_linear takes as `workspace` lives here in a fixed device array
 * of BD_NOALLOC_SCRATCH_BYTES that is part of the library image: every GPU whose
 * context loads the library carries those bytes until the process exits.
 *
 * Same arguments, results and errors as bd_linear, minus the workspace pair.
 * Problems with bd_linear_workspace_size(M, N, K) > BD_NOALLOC_SCRATCH_BYTES are
 * refused with BD_ERR_SCRATCH_LIMIT and nothing is enqueued.  The call performs no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *
 * The first call on each device looks up the array's device address (a symbol
 * query, with that device current) and caches it; make that first call outside
 * any stream capture.  All calls on a device share the one array: it keeps
 * whatever the previous call left there, which is harmless because every byte a
 * call reads it has written earlier in the same call, so nothing needs clearing.
 * Two calls that overlap on the GPU (different streams, or one stream per thread)
 * race on the array; serialise them. */
#define BD_NOALLOC_SCRATCH_BYTES (32u << 20)
bd_status bd_linear_noalloc(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx,
                            const bd_qtensor *Wq, void *Y, bd_dtype ydtype, int64_t ldy, void *stream);

/* Canonical layout (what is compared bit for bit with a reference):
 *   codes  [rows][K/2]   byte j of a row: element 2j in bits 3:0, element 2j+1 in
 *                        bits 7:4; nibble = sign << 3 | index (index ascending in
 *                        magnitude, Sec. 3.3: the example value 10 has index 110b)
 *   ids    [rows][K/32]  one byte per block, 0..15
 *   scales [rows][K/32]  one byte per block, e + 127                               */
bd_status bd_export_canonical(const bd_qtensor *q, uint8_t *codes, uint8_t *ids, uint8_t *scales,
                              void *stream);
bd_status bd_import_canonical(const uint8_t *codes, const uint8_t *ids, const uint8_t *scales,
                              bd_qtensor *q, void *stream);

/* out[rows][ld] (fp32) = sign * 0.5 * value[id][index] * 2^e (Sec. 3.3, Fig. 6). */
bd_status bd_dequantize(const bd_qtensor *q, float *out, int64_t ld, void *stream);

/* The DialectFP4 formatbook (Sec. 3.1, Fig. 4) as a HOST table: magnitudes in units
 * of 0.5, ascending. */
bd_status bd_get_formatbook(uint8_t out[16][8]);

/* Replaces the formatbook (HOST table, same form; NULL restores the built-in one) on the
 * current device.  The paper shows its table only as a figure (Fig. 4); the built-in table
 * is reconstructed from the rules of Sec. 3.1 and the printed values of dialects 4 and 5,
 * so this call is how a caller supplies other values.  Accepted tables keep the structure
 * the two-stage selection relies on (Sec. 3.2): every row strictly ascending from 0, values
 * <= 15; rows 2p and 2p + 1 share all values but the one at index 6, the even row holding
 * the larger; the pair's maximum is 15 - p.  Anything else returns BD_ERR_INVALID_ARG and
 * changes nothing.  Synchronises the device first; operands quantised under another table
 * keep their codes but decode through the new one, so requantise them.  Not thread-safe
 * against other calls of the library. */
bd_status bd_set_formatbook(const uint8_t in[16][8]);

/* Synchronises `stream`, then returns and clears the device status word:
 * BD_OK, BD_ERR_NONFINITE or BD_ERR_TIMEOUT (or BD_ERR_CUDA). */
bd_status bd_poll_status(void *stream);

/* Test hook for the bounded device-side waits (every wait on a barrier inside the kernels gives up
 * after a number of polls, records BD_ERR_TIMEOUT in the status word and lets the kernel drain and
 * return).  poll_limit > 0 replaces the built-in limit (about a second) on the current device, rounded
 * up to 1024 polls; skip_first_code_stage != 0 makes the tensor-core product leave out the first copy
 * of packed weights of every CTA, so that the wait for it runs out: the call then writes no result and
 * bd_poll_status returns BD_ERR_TIMEOUT.  (0, 0) restores normal operation.  Synchronises the device. */
bd_status bd_debug_fault(uint32_t poll_limit, int skip_first_code_stage);

bd_status bd_set_gemm_impl(bd_gemm_impl impl);
/* Number of kernels this library has launched in this process (host counter). */
uint64_t bd_launch_count(void);
int bd_last_cuda_error(void);
const char *bd_status_string(bd_status s);
int bd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BD_H */
