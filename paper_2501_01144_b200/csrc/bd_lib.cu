// libblockdialect: the extern "C" entry points declared in include/bd.h.
// Host-side validation and kernel dispatch only; all arithmetic is in the kernels.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdlib.h>

#include <algorithm>

#include "bd_common.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_warp.cuh"
#include "blocksize.cuh"
#include "kvcache.cuh"
#include "attention.cuh"
#include "quantize.cuh"

using namespace bd;

namespace {

int g_last_cuda_error = 0;
uint64_t g_launches = 0;
bd_gemm_impl g_gemm_impl = BD_GEMM_AUTO;
constexpr int kMaxDevices = 64;
Formatbook g_book = kBook;            // the table bd_get_formatbook reports (host copy of what the device uses)

bd_status cuda_result(cudaError_t e) {
    if (e == cudaSuccess) return BD_OK;
    g_last_cuda_error = (int)e;
    return BD_ERR_CUDA;
}
bd_status launch_result(int kernels = 1) {
    g_launches += (uint64_t)kernels;
    return cuda_result(cudaGetLastError());
}

bool aligned16(const void *p) { return ((uintptr_t)p & 15u) == 0; }

bd_status check_qtensor(const bd_qtensor *q) {
    if (!q || !q->codes || !q->ids || !q->scales) return BD_ERR_INVALID_ARG;
    if (q->rows <= 0 || q->K <= 0) return BD_ERR_INVALID_ARG;
    if (q->K % kBlock) return BD_ERR_SHAPE;
    if (!aligned16(q->codes) || !aligned16(q->ids) || !aligned16(q->scales)) return BD_ERR_ALIGN;
    return BD_OK;
}

int elem_bytes(bd_dtype dt) { return dt == BD_F32 ? 4 : 2; }

unsigned grid_for(int64_t threads, int block) { return (unsigned)((threads + block - 1) / block); }

// Resident CTAs of the bf16 quantizer on the current device (it loops over its chunks).
unsigned quant_bf16_grid_limit() {
    static unsigned limit[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) return 148u * BD_QUANT_MIN_BLOCKS;
    if (!limit[dev]) {
        int sms = 0;
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        limit[dev] = (unsigned)(sms > 0 ? sms : 148) * BD_QUANT_MIN_BLOCKS;
    }
    return limit[dev];
}

// Launch with programmatic stream serialisation: the blocks may be scheduled while the previous kernel of the
// stream drains; such a kernel waits for that kernel's results before it touches global memory.
template <typename... Params, typename... Args>
void launch_serialized(void (*kernel)(Params...), dim3 grid, unsigned block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaLaunchKernelEx(&cfg, kernel, Params(args)...);
}

template <int SELECT, bool WC, bool WE>
bd_status launch_contig(const void *X, bd_dtype dt, int64_t ld, const QView &out, uint8_t *e4m3, cudaStream_t st) {
    const int nb = (int)(out.K / kBlock), nb_pad = (int)k_groups(out.K) * kBlocksPerAtom;
    const int64_t rows_pad = row_tiles(out.rows) * kRowTile;
    const unsigned chunks = (unsigned)(rows_pad / 64) * (unsigned)(nb_pad / kBlocksPerAtom);     // 64 rows x one k-group
    // generic kernel: its CTAs loop over the chunks; three per SM fit with the fp32 staging buffers, and the
    // other source types are served well enough by the same number
    const unsigned gen_grid = std::min(chunks, quant_bf16_grid_limit());
    const int kgs = nb_pad / kBlocksPerAtom;
    const FastDiv div_kgs = make_fast_div((uint32_t)kgs);
    const bool regular = out.rows % kRowTile == 0 && nb % kBlocksPerAtom == 0;
    switch (dt) {
        case BD_F32: {
            static bool configured[64] = {};                      // per instantiation and device
            int dev = 0;
            cudaGetDevice(&dev);
            if (dev >= 0 && dev < 64 && !configured[dev]) {
                if (cudaFuncSetAttribute(quantize_contig_kernel<BD_F32, SELECT, WC, WE, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kContigStageBytes) != cudaSuccess ||
                    cudaFuncSetAttribute(quantize_contig_kernel<BD_F32, SELECT, WC, WE, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kContigStageBytes) != cudaSuccess)
                    return launch_result();
                configured[dev] = true;
            }
            if (regular)
                launch_serialized(quantize_contig_kernel<BD_F32, SELECT, WC, WE, true>, gen_grid, 256, kContigStageBytes, st, X, ld, out, e4m3, nb, kgs, chunks, div_kgs);
            else
                launch_serialized(quantize_contig_kernel<BD_F32, SELECT, WC, WE, false>, gen_grid, 256, kContigStageBytes, st, X, ld, out, e4m3, nb, kgs, chunks, div_kgs);
            break;
        }
        case BD_BF16:
            if (SELECT == BD_SELECT_TWO_STAGE && rows_pad * nb_pad < (1ll << 31))
            {
                const unsigned grid = std::min(chunks, quant_bf16_grid_limit());
                if (regular)
                    launch_serialized(quantize_bf16_kernel<WC, WE, true>, grid, 256, 0, st, (const uint16_t *)X, ld, out, e4m3, chunks,
                                      (uint32_t)nb, (uint32_t)kgs, div_kgs);
                else
                    launch_serialized(quantize_bf16_kernel<WC, WE, false>, grid, 256, 0, st, (const uint16_t *)X, ld, out, e4m3, chunks,
                                      (uint32_t)nb, (uint32_t)kgs, div_kgs);
            }
            else
                launch_serialized(quantize_contig_kernel<BD_BF16, SELECT, WC, WE, false>, gen_grid, 256, 0, st, X, ld, out, e4m3, nb, kgs, chunks, div_kgs);
            break;
        case BD_F16: launch_serialized(quantize_contig_kernel<BD_F16, SELECT, WC, WE, false>, gen_grid, 256, 0, st, X, ld, out, e4m3, nb, kgs, chunks, div_kgs); break;
        default: return BD_ERR_INVALID_ARG;
    }
    return launch_result();
}

bd_status check_source(const void *X, bd_dtype dt, int64_t rows, int64_t K, int64_t ld, int64_t min_ld) {
    if (!X || rows <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (dt != BD_F32 && dt != BD_BF16 && dt != BD_F16) return BD_ERR_INVALID_ARG;
    if (K % kBlock || ld < min_ld) return BD_ERR_SHAPE;
    if (!aligned16(X) || (ld * elem_bytes(dt)) % 16) return BD_ERR_ALIGN;
    return BD_OK;
}

template <typename OutT>
bd_status launch_simt(const QView &A, const QView &B, void *Y, int64_t ldy, cudaStream_t st) {
    dim3 grid((unsigned)((B.rows + kSimtTile - 1) / kSimtTile), (unsigned)((A.rows + kSimtTile - 1) / kSimtTile));
    gemm_simt_kernel<OutT><<<grid, 256, 0, st>>>(A, B, (OutT *)Y, ldy);
    return launch_result();
}

bool use_tc(int64_t M, int64_t N, int64_t K) {
    if (g_gemm_impl == BD_GEMM_SIMT) return false;
    if (g_gemm_impl == BD_GEMM_TCGEN05) return true;
    return tc_supported(M, N, K) && (M >= 16 || (int64_t)N * K >= (1 << 22));
}

bd_status check_gemm(const bd_qtensor *A, const bd_qtensor *B, const void *Y, bd_dtype ydt, int64_t ldy) {
    bd_status s = check_qtensor(A);
    if (s) return s;
    s = check_qtensor(B);
    if (s) return s;
    if (!Y || (ydt != BD_F32 && ydt != BD_BF16)) return BD_ERR_INVALID_ARG;
    if (A->K != B->K || ldy < B->rows) return BD_ERR_SHAPE;
    return BD_OK;
}

// The warp-level kernel (gemm_warp.cuh) serves up to 16 activation rows.  The library's own choice takes it for up to 8
// (one token group per MMA), where it measured faster than the tensor-core path with its three launches at every
// size, and for 9 to 16 rows against at most 2^25 weights, where a call is mostly fixed cost and this kernel has
// less of it (9.5 against 12.8 us at 4096 x 4096); against more weights the two token groups make it the slower one
// (22 against 17 us at 4096 x 14336).
bool use_warp(int64_t M, int64_t N, int64_t K) {
    if (g_gemm_impl == BD_GEMM_WARP) return true;
    if (g_gemm_impl != BD_GEMM_AUTO || !wk::supported(M, N, K) || (int64_t)N * K < (1 << 18)) return false;
    return M <= wk::kTokTile || (int64_t)N * K <= (1 << 25);
}
unsigned sm_count() {
    static int sms[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= kMaxDevices) return 148;
    if (!sms[dev]) {
        cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev);
        if (sms[dev] <= 0) sms[dev] = 148;
    }
    return (unsigned)sms[dev];
}
// Warps per CTA = shares of K of a row tile: as many as keep about 32 warps on every SM with all CTAs resident
// at once, at most one per unit of K.
int warp_kernel_warps(int64_t N, int64_t K) {
    const int64_t tiles = N / wk::kRows, units = K / wk::kUnitK;
    const int64_t per_sm = (tiles + sm_count() - 1) / sm_count();
    int64_t w = 32 / per_sm;
    return (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(w, units), wk::kMaxWarps));
}
// The product kernel over records at `workspace` (rec16, then the factors).  batch: n problems with the operands
// of `batch`, records rec_stride bytes apart and results y_stride elements apart.
bd_status launch_warp_main(int64_t M, int64_t K, const QView &W, void *Y, bd_dtype ydtype, int64_t ldy, void *workspace, cudaStream_t st,
                           const wk::OperandBatch *batch = nullptr, int n = 1, int64_t rec_stride = 0, int64_t y_stride = 0) {
    const int nt = M > wk::kTokTile ? 2 : 1;
    const uint8_t *rec16 = (const uint8_t *)workspace;
    const float *recs = (const float *)(rec16 + (size_t)wk::padded_blocks(K) * nt * wk::kRecBytes);
    wk::Params p{W.codes, W.ids, W.scales, W.ldc, row_tiles(W.rows), rec16, recs, Y, ldy, W.rows, rec_stride, y_stride, (int)M,
                 (int)((K + wk::kUnitK - 1) / wk::kUnitK), (int)(K / kBlock % wk::kUnitBlocks), ydtype == BD_BF16};
    const int64_t tiles = (W.rows + wk::kRows - 1) / wk::kRows;
    const int warps = warp_kernel_warps(tiles * n * wk::kRows, (K + wk::kUnitK - 1) / wk::kUnitK * wk::kUnitK);
    const size_t smem = (size_t)warps * (wk::kStages * wk::kStageBytes + nt * 512);
    const dim3 grid((unsigned)tiles, (unsigned)n);
    const bool ragged = W.rows % wk::kRows != 0 || K % wk::kUnitK != 0;
    using Kernel = void (*)(const wk::Params, const wk::OperandBatch);
    static const Kernel kernels[8] = {wk::gemm_warp_kernel<1, false, false>, wk::gemm_warp_kernel<1, false, true>, wk::gemm_warp_kernel<1, true, false>,
                                      wk::gemm_warp_kernel<1, true, true>,   wk::gemm_warp_kernel<2, false, false>, wk::gemm_warp_kernel<2, false, true>,
                                      wk::gemm_warp_kernel<2, true, false>,  wk::gemm_warp_kernel<2, true, true>};
    static bool smem_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < kMaxDevices && !smem_set[dev]) {
        const int most = wk::kMaxWarps * (wk::kStages * wk::kStageBytes + 2 * 512);
        for (Kernel k : kernels)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess) return cuda_result(cudaGetLastError());
        smem_set[dev] = true;
    }
    const wk::OperandBatch none{};
    launch_serialized(kernels[(nt - 1) * 4 + (batch ? 2 : 0) + (ragged ? 1 : 0)], grid, 32u * warps, smem, st, p, batch ? *batch : none);
    return launch_result(1);
}
// X: n problems x_stride elements apart (n = 1: one).
bd_status launch_warp_records(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, void *workspace, cudaStream_t st, int n = 1,
                              int64_t x_stride = 0, int64_t rec_stride = 0) {
    const int nt = M > wk::kTokTile ? 2 : 1, nb = (int)(K / kBlock);
    uint8_t *rec16 = (uint8_t *)workspace;
    float *recs = (float *)(rec16 + (size_t)wk::padded_blocks(K) * nt * wk::kRecBytes);
    const dim3 qgrid(grid_for(wk::padded_blocks(K) * wk::kTokTile * nt, 128), (unsigned)n);
    switch (xdtype) {
    case BD_F32: launch_serialized(wk::quantize_records_kernel<BD_F32>, qgrid, 128, 0, st, X, ldx, (int)M, nb, nt, rec16, recs, x_stride, rec_stride); break;
    case BD_BF16: launch_serialized(wk::quantize_records_kernel<BD_BF16>, qgrid, 128, 0, st, X, ldx, (int)M, nb, nt, rec16, recs, x_stride, rec_stride); break;
    default: launch_serialized(wk::quantize_records_kernel<BD_F16>, qgrid, 128, 0, st, X, ldx, (int)M, nb, nt, rec16, recs, x_stride, rec_stride); break;
    }
    return launch_result(1);
}
bd_status launch_warp_linear(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, const QView &W, void *Y,
                             bd_dtype ydtype, int64_t ldy, void *workspace, cudaStream_t st) {
    bd_status s = launch_warp_records(X, xdtype, M, K, ldx, workspace, st);
    if (s) return s;
    return launch_warp_main(M, K, W, Y, ydtype, ldy, workspace, st);
}
// The two products of a decode step's attention over n heads (gemm_warp.cuh, MODE 1 and 2): W is the view of head 0's
// cached operand (shape, pitch), `ops` the heads' operand pointers, x the mode's extras.
bd_status launch_warp_attn(int mode, int64_t M, int64_t K, const QView &W, void *Y, bd_dtype ydtype, int64_t ldy, int64_t y_stride,
                           const void *records, int64_t rec_stride, const wk::OperandBatch &ops, const wk::Extra &x, int n, cudaStream_t st) {
    const int nt = M > wk::kTokTile ? 2 : 1;
    const uint8_t *rec16 = (const uint8_t *)records;
    const float *recs = (const float *)(rec16 + (size_t)wk::padded_blocks(K) * nt * wk::kRecBytes);
    wk::Params p{W.codes, W.ids, W.scales, W.ldc, row_tiles(W.rows), rec16, recs, Y, ldy, W.rows, rec_stride, y_stride, (int)M,
                 (int)((K + wk::kUnitK - 1) / wk::kUnitK), (int)(K / kBlock % wk::kUnitBlocks), ydtype == BD_BF16};
    const int64_t tiles = (W.rows + wk::kRows - 1) / wk::kRows;
    const int warps = warp_kernel_warps(tiles * n * wk::kRows, (K + wk::kUnitK - 1) / wk::kUnitK * wk::kUnitK);
    const size_t smem = (size_t)warps * (wk::kStages * wk::kStageBytes + nt * 512);
    using Kernel = void (*)(const wk::Params, const wk::OperandBatch, const wk::Extra);
    static const Kernel kernels[4] = {wk::gemm_warp_attn_kernel<1, 1>, wk::gemm_warp_attn_kernel<2, 1>, wk::gemm_warp_attn_kernel<1, 2>,
                                      wk::gemm_warp_attn_kernel<2, 2>};
    static bool smem_set[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < kMaxDevices && !smem_set[dev]) {
        const int most = wk::kMaxWarps * (wk::kStages * wk::kStageBytes + 2 * 512);
        for (Kernel k : kernels)
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, most) != cudaSuccess) return cuda_result(cudaGetLastError());
        smem_set[dev] = true;
    }
    launch_serialized(kernels[(mode - 1) * 2 + (nt - 1)], dim3((unsigned)tiles, (unsigned)n), 32u * warps, smem, st, p, ops, x);
    return launch_result(1);
}
// bd_gemm with a few rows of A: records from the quantised A, then the same product kernel.
bd_status launch_warp_gemm(const QView &A, const QView &B, void *Y, bd_dtype ydtype, int64_t ldy, void *workspace, cudaStream_t st) {
    const int nt = A.rows > wk::kTokTile ? 2 : 1;
    uint8_t *rec16 = (uint8_t *)workspace;
    float *recs = (float *)(rec16 + (size_t)wk::padded_blocks(A.K) * nt * wk::kRecBytes);
    const wk::OperandBatch none{};
    launch_serialized(wk::records_from_qtensor_kernel<false>, dim3(grid_for(wk::padded_blocks(A.K) * wk::kTokTile * nt, 128)), 128, 0, st, A, nt, rec16,
                      recs, none, (int64_t)0);
    bd_status s = launch_result(1);
    if (s) return s;
    return launch_warp_main(A.rows, A.K, B, Y, ydtype, ldy, workspace, st);
}

bd_status gemm_dispatch(const QView &A, const QView &B, void *Y, bd_dtype ydt, int64_t ldy, void *ws, size_t ws_bytes,
                        cudaStream_t st) {
    if (use_warp(A.rows, B.rows, A.K)) {
        if (!wk::supported(A.rows, B.rows, A.K)) return BD_ERR_UNSUPPORTED;
        if (!ws || ws_bytes < wk::record_bytes(A.K, 2)) return BD_ERR_WORKSPACE;
        if ((uintptr_t)ws & 255u) return BD_ERR_ALIGN;
        return launch_warp_gemm(A, B, Y, ydt, ldy, ws, st);
    }
    if (use_tc(A.rows, B.rows, A.K)) {
        if (!tc_supported(A.rows, B.rows, A.K)) return BD_ERR_UNSUPPORTED;
        size_t need = tc_gemm_workspace(A.rows, B.rows, A.K);
        if (!ws || ws_bytes < need) return BD_ERR_WORKSPACE;
        if ((uintptr_t)ws & 255u) return BD_ERR_ALIGN;
        // A is expanded to operand bytes by a kernel; B stays packed and is expanded inside the GEMM
        uint8_t *a8 = (uint8_t *)ws;
        const int nb = (int)(A.K / kBlock);
        decode_e4m3_kernel<<<grid_for(A.rows * nb, 256), 256, 0, st>>>(A, a8, nb);
        bd_status s = launch_result(1);
        if (s) return s;
        int kernels = 1;
        s = cuda_result(tc::launch(a8, A.scales, A.rows, B, A.K, Y, ydt == BD_BF16, ldy, st,
                                   a8 + tc_operand_bytes(A.rows, A.K), tc::splitk_workspace(A.rows, B.rows, A.K), &kernels));
        g_launches += (uint64_t)kernels;
        return s;
    }
    if (ydt == BD_F32) return launch_simt<float>(A, B, Y, ldy, st);
    return launch_simt<__nv_bfloat16>(A, B, Y, ldy, st);
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

// Built-in scratch of bd_linear_noalloc.  In host code this name is only a handle
// for symbol queries, never a device address: the entry point asks the runtime for
// the address once per device and passes that pointer on.
static __device__ __align__(256) uint8_t g_noalloc_scratch[BD_NOALLOC_SCRATCH_BYTES];

namespace {
void *g_noalloc_ptr[kMaxDevices] = {};
}  // namespace

// launchers of the KV-cache kernels per source type
template <int DT>
void launch_kv_keys(const void *Knew, int64_t ldk, int64_t t, const QView &k, int64_t row0, cudaStream_t st, const KvBatch *batch = nullptr,
                    int n = 1, int64_t src_stride = 0) {
    const dim3 grid(grid_for(t * kBlocksPerAtom, 256), (unsigned)n);
    const KvBatch none{};
    if (batch) kv_append_keys_kernel<DT, true><<<grid, 256, 0, st>>>(Knew, ldk, t, k, row0, (int)(k.K / kBlock), *batch, src_stride);
    else kv_append_keys_kernel<DT, false><<<grid, 256, 0, st>>>(Knew, ldk, t, k, row0, (int)(k.K / kBlock), none, 0);
}
template <int DT>
void launch_kv_chunks(const void *src, int64_t ld, int n_chunks, const QView &v, int chunk0, cudaStream_t st, const KvBatch *batch = nullptr,
                      int n = 1, int64_t src_stride = 0) {
    const int pairs = (chunk0 + n_chunks + 1) / 2 - chunk0 / 2;
    const dim3 grid(grid_for(v.rows * pairs, 256), (unsigned)n);
    const KvBatch none{};
    if (batch) kv_quantize_chunks_kernel<DT, true><<<grid, 256, 0, st>>>(src, ld, n_chunks, v, chunk0, *batch, src_stride);
    else kv_quantize_chunks_kernel<DT, false><<<grid, 256, 0, st>>>(src, ld, n_chunks, v, chunk0, none, 0);
}
void launch_kv_recent(const void *Vnew, int64_t ldv_bytes, int rows, int row_bytes, void *recent, int slot0, cudaStream_t st,
                      const KvBatch *batch = nullptr, int n = 1, int64_t src_stride_bytes = 0) {
    const dim3 grid(grid_for((int64_t)rows * row_bytes / 2, 256), (unsigned)n);
    const KvBatch none{};
    if (batch) kv_store_recent_kernel<true><<<grid, 256, 0, st>>>(Vnew, ldv_bytes, rows, row_bytes, (uint8_t *)recent, slot0, *batch, src_stride_bytes);
    else kv_store_recent_kernel<false><<<grid, 256, 0, st>>>(Vnew, ldv_bytes, rows, row_bytes, (uint8_t *)recent, slot0, none, 0);
}
template <int DT>
void launch_kv_finish(const float *part, int64_t ld_part, const float *P, int64_t ldp, int64_t n_q, int n_recent, const void *recent,
                      int d, int64_t q_rows, void *Y, bd_dtype ydt, int64_t ldy, cudaStream_t st) {
    const unsigned grid = grid_for(q_rows * d, 256);
    const RecentBatch none{};
    if (ydt == BD_BF16)
        kv_pv_finish_kernel<DT, __nv_bfloat16, false><<<grid, 256, 0, st>>>(part, ld_part, P, ldp, n_q, n_recent, recent, d, q_rows, (__nv_bfloat16 *)Y, ldy, none, 0, 0, 0);
    else
        kv_pv_finish_kernel<DT, float, false><<<grid, 256, 0, st>>>(part, ld_part, P, ldp, n_q, n_recent, recent, d, q_rows, (float *)Y, ldy, none, 0, 0, 0);
}
#define BD_KV_DISPATCH(dt, fn, ...)                          \
    switch (dt) {                                            \
        case BD_F32: fn<BD_F32>(__VA_ARGS__); break;         \
        case BD_BF16: fn<BD_BF16>(__VA_ARGS__); break;       \
        default: fn<BD_F16>(__VA_ARGS__); break;             \
    }

// launchers of the quantizer for block sizes 16 and 64
namespace {
template <int DT, int BS>
void launch_quantize_bs(const void *X, int64_t ld, bd_select select, const QView &v, cudaStream_t st) {
    const int nbp = (int)(v.K / kBlock), nbp_pad = (int)k_groups(v.K) * kBlocksPerAtom;
    const int64_t rows_pad = row_tiles(v.rows) * kRowTile;
    const unsigned grid = grid_for(rows_pad * nbp_pad, 256);
    if (select == BD_SELECT_MSE) quantize_bs_kernel<DT, BS, BD_SELECT_MSE><<<grid, 256, 0, st>>>(X, ld, v, rows_pad, nbp, nbp_pad);
    else quantize_bs_kernel<DT, BS, BD_SELECT_TWO_STAGE><<<grid, 256, 0, st>>>(X, ld, v, rows_pad, nbp, nbp_pad);
}
template <int BS>
bd_status quantize_bs_dtype(const void *X, bd_dtype dt, int64_t ld, bd_select select, const QView &v, cudaStream_t st) {
    switch (dt) {
        case BD_F32: launch_quantize_bs<BD_F32, BS>(X, ld, select, v, st); break;
        case BD_BF16: launch_quantize_bs<BD_BF16, BS>(X, ld, select, v, st); break;
        default: launch_quantize_bs<BD_F16, BS>(X, ld, select, v, st); break;
    }
    return launch_result();
}
}  // namespace

extern "C" {

bd_status bd_qtensor_sizes(int64_t rows, int64_t K, size_t *codes_bytes, size_t *ids_bytes, size_t *scales_bytes) {
    if (rows <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (K % kBlock) return BD_ERR_SHAPE;
    const size_t atoms = (size_t)(row_tiles(rows) * k_groups(K));
    if (codes_bytes) *codes_bytes = (size_t)rows * (size_t)(K / 2);
    if (ids_bytes) *ids_bytes = atoms * kIdAtomBytes;
    if (scales_bytes) *scales_bytes = atoms * kScaleAtomBytes;
    return BD_OK;
}

bd_status bd_quantize_weights(const void *W, bd_dtype dtype, int64_t N, int64_t K, int64_t ldw, bd_select select,
                              bd_qtensor *out, void *stream) {
    bd_status s = check_source(W, dtype, N, K, ldw, K);
    if (s) return s;
    s = check_qtensor(out);
    if (s) return s;
    if (out->rows != N || out->K != K) return BD_ERR_SHAPE;
    QView v = view_of(out);
    cudaStream_t st = (cudaStream_t)stream;
    if (select == BD_SELECT_MSE) return launch_contig<BD_SELECT_MSE, true, false>(W, dtype, ldw, v, nullptr, st);
    if (select == BD_SELECT_TWO_STAGE) return launch_contig<BD_SELECT_TWO_STAGE, true, false>(W, dtype, ldw, v, nullptr, st);
    return BD_ERR_INVALID_ARG;
}

bd_status bd_quantize_act(const void *X, bd_dtype dtype, int64_t M, int64_t K, int64_t ldx, bd_axis axis,
                          bd_qtensor *out, void *stream) {
    if (axis != BD_AXIS_CONTIG && axis != BD_AXIS_STRIDED) return BD_ERR_INVALID_ARG;
    bd_status s = check_source(X, dtype, M, K, ldx, axis == BD_AXIS_CONTIG ? K : M);
    if (s) return s;
    s = check_qtensor(out);
    if (s) return s;
    if (out->rows != M || out->K != K) return BD_ERR_SHAPE;
    QView v = view_of(out);
    cudaStream_t st = (cudaStream_t)stream;
    if (axis == BD_AXIS_CONTIG) return launch_contig<BD_SELECT_TWO_STAGE, true, false>(X, dtype, ldx, v, nullptr, st);
    const int nb = (int)(K / kBlock), nb_pad = (int)k_groups(K) * kBlocksPerAtom;
    const int64_t rows_pad = row_tiles(M) * kRowTile;
    const unsigned grid = grid_for(rows_pad * (nb_pad / 2), 256);
    switch (dtype) {
        case BD_F32: quantize_strided_kernel<BD_F32><<<grid, 256, 0, st>>>(X, ldx, v, rows_pad, nb, nb_pad); break;
        case BD_BF16: quantize_strided_kernel<BD_BF16><<<grid, 256, 0, st>>>(X, ldx, v, rows_pad, nb, nb_pad); break;
        default: quantize_strided_kernel<BD_F16><<<grid, 256, 0, st>>>(X, ldx, v, rows_pad, nb, nb_pad); break;
    }
    return launch_result();
}

bd_status bd_gemm_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes) {
    if (!bytes || M <= 0 || N <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (K % kBlock) return BD_ERR_SHAPE;
    *bytes = tc_supported(M, N, K) ? tc_gemm_workspace(M, N, K) : 0;
    if (wk::supported(M, N, K)) *bytes = std::max(*bytes, (size_t)((wk::record_bytes(K, 2) + 255) & ~(size_t)255));
    return BD_OK;
}

bd_status bd_gemm(const bd_qtensor *A, const bd_qtensor *B, void *Y, bd_dtype ydtype, int64_t ldy, void *workspace,
                  size_t workspace_bytes, void *stream) {
    bd_status s = check_gemm(A, B, Y, ydtype, ldy);
    if (s) return s;
    return gemm_dispatch(view_of(A), view_of(B), Y, ydtype, ldy, workspace, workspace_bytes, (cudaStream_t)stream);
}

bd_status bd_gemm_batched_workspace_size(int64_t M, int64_t N, int64_t K, int64_t b_group, size_t *bytes) {
    if (!bytes || M <= 0 || N <= 0 || K <= 0 || b_group <= 0) return BD_ERR_INVALID_ARG;
    if (K % kBlock) return BD_ERR_SHAPE;
    size_t single = 0;
    bd_status s = bd_gemm_workspace_size(M, N, K, &single);
    if (s) return s;
    const int64_t count = std::min<int64_t>(b_group, kStackMax);
    size_t c, i, sc;
    bd_qtensor_sizes(M * count, K, &c, &i, &sc);
    const size_t stacked = b_group > 1 ? align256(sc) + tc_operand_bytes(M * count, K) : 0;
    *bytes = std::max(single, stacked);
    return BD_OK;
}

bd_status bd_gemm_batched(const bd_qtensor *A, const bd_qtensor *B, int64_t batch, int64_t b_group, void *Y,
                          bd_dtype ydtype, int64_t ldy, int64_t stride_y, void *workspace, size_t workspace_bytes,
                          void *stream) {
    if (!A || !B || batch <= 0 || b_group <= 0 || batch % b_group) return BD_ERR_INVALID_ARG;
    for (int64_t i = 0; i < batch; i++) {
        bd_status s = check_gemm(&A[i], &B[i / b_group], Y, ydtype, ldy);
        if (s) return s;
        // one shape per side: the stacked route reads A[0]'s row count and K from every operand
        if (A[i].rows != A[0].rows || A[i].K != A[0].K || B[i / b_group].rows != B[0].rows) return BD_ERR_SHAPE;
    }
    const int ysz = ydtype == BD_F32 ? 4 : 2;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t M = A[0].rows, N = B[0].rows, K = A[0].K;
    size_t stacked_need = 0;
    bd_gemm_batched_workspace_size(M, N, K, b_group, &stacked_need);
    // Grouped products share their B operand: when the group's results are contiguous in Y and the operands are
    // whole row tiles, the group's A operands are decoded into one stacked matrix and the group is one launch.
    // A few rows of A per product (decode-shaped attention without the cache object): the warp-level kernel takes the
    // whole batch through grid.y, 64 products per launch, and expands the A operands' code words itself.
    if (use_warp(M, N, K) && wk::supported(M, N, K)) {
        for (int64_t i0 = 0; i0 < batch; i0 += wk::kMaxBatch) {
            const int count = (int)std::min<int64_t>(wk::kMaxBatch, batch - i0);
            wk::OperandBatch ops{};
            wk::Extra x{};
            for (int h = 0; h < count; h++) {
                const bd_qtensor &a = A[i0 + h], &b = B[(i0 + h) / b_group];
                x.a_codes[h] = (const uint8_t *)a.codes; x.a_ids[h] = (const uint8_t *)a.ids; x.a_scales[h] = (const uint8_t *)a.scales;
                ops.codes[h] = (const uint8_t *)b.codes; ops.ids[h] = (const uint8_t *)b.ids; ops.scales[h] = (const uint8_t *)b.scales;
            }
            x.a_ldc = K / 2;
            bd_status s = launch_warp_attn(1, M, K, view_of(&B[0]), (uint8_t *)Y + i0 * stride_y * ysz, ydtype, ldy, stride_y, nullptr, 0, ops, x, count, st);
            if (s) return s;
        }
        return BD_OK;
    }
    const bool stack = b_group > 1 && M % kRowTile == 0 && stride_y == M * ldy && use_tc(M * b_group, N, K) &&
                       tc_supported(M * b_group, N, K) && workspace && workspace_bytes >= stacked_need &&
                       !((uintptr_t)workspace & 255u);
    if (stack) {
        const int nb = (int)(K / kBlock);
        for (int64_t g0 = 0; g0 < batch; g0 += b_group) {
            uint8_t *y = (uint8_t *)Y + g0 * stride_y * ysz;
            for (int64_t c0 = 0; c0 < b_group; c0 += kStackMax) {            // at most kStackMax operands per launch
                const int count = (int)std::min<int64_t>(kStackMax, b_group - c0);
                size_t sc_bytes, dummy_c, dummy_i;
                bd_qtensor_sizes(M * count, K, &dummy_c, &dummy_i, &sc_bytes);
                uint8_t *sf = (uint8_t *)workspace, *a8 = sf + align256(sc_bytes);
                StackedViews v = {};
                for (int h = 0; h < count; h++) {
                    const bd_qtensor &a = A[g0 + c0 + h];
                    v.codes[h] = (const uint8_t *)a.codes;
                    v.ids[h] = (const uint8_t *)a.ids;
                    v.scales[h] = (const uint8_t *)a.scales;
                }
                dim3 grid(grid_for(M * nb, 256), (unsigned)count);
                decode_e4m3_stacked_kernel<<<grid, 256, 0, st>>>(v, count, M, K, a8, sf, nb);
                bd_status s = launch_result(1);
                if (s) return s;
                g_launches += 1;
                s = cuda_result(tc::launch(a8, sf, M * count, view_of(&B[g0 / b_group]), K, y + c0 * stride_y * ysz,
                                           ydtype == BD_BF16, ldy, st));
                if (s) return s;
            }
        }
        return BD_OK;
    }
    for (int64_t i = 0; i < batch; i++) {
        bd_status s = gemm_dispatch(view_of(&A[i]), view_of(&B[i / b_group]), (char *)Y + i * stride_y * ysz, ydtype,
                                    ldy, workspace, workspace_bytes, (cudaStream_t)stream);
        if (s) return s;
    }
    return BD_OK;
}

bd_status bd_linear_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes) {
    if (!bytes || M <= 0 || N <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (K % kBlock) return BD_ERR_SHAPE;
    size_t c, i, s;
    bd_qtensor_sizes(M, K, &c, &i, &s);
    // tensor-core path: scale atoms + operand bytes of X; CUDA-core path: a packed X
    const size_t tc_bytes = tc_supported(M, N, K) ? align256(s) + tc_gemm_workspace(M, N, K) : 0;
    const size_t simt_bytes = align256(c) + align256(i) + align256(s);
    *bytes = tc_bytes > simt_bytes ? tc_bytes : simt_bytes;
    if (wk::supported(M, N, K)) *bytes = std::max(*bytes, align256(wk::record_bytes(K, 2)));
    return BD_OK;
}

bd_status bd_linear(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, const bd_qtensor *Wq, void *Y,
                    bd_dtype ydtype, int64_t ldy, void *workspace, size_t workspace_bytes, void *stream) {
    bd_status s = check_source(X, xdtype, M, K, ldx, K);
    if (s) return s;
    s = check_qtensor(Wq);
    if (s) return s;
    if (Wq->K != K || ldy < Wq->rows) return BD_ERR_SHAPE;
    if (!Y || (ydtype != BD_F32 && ydtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    size_t need;
    bd_linear_workspace_size(M, Wq->rows, K, &need);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    size_t c, i, sc;
    bd_qtensor_sizes(M, K, &c, &i, &sc);
    char *p = (char *)workspace;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t N = Wq->rows;
    if (use_warp(M, N, K)) {
        if (!wk::supported(M, N, K)) return BD_ERR_UNSUPPORTED;
        return launch_warp_linear(X, xdtype, M, K, ldx, view_of(Wq), Y, ydtype, ldy, workspace, st);
    }
    if (use_tc(M, N, K)) {
        if (!tc_supported(M, N, K)) return BD_ERR_UNSUPPORTED;
        // tensor-core path: the quantizer writes the operand bytes and the scale atoms directly
        // (no codes, no ids); the weights stay packed and are expanded inside the GEMM
        uint8_t *sfa = (uint8_t *)p;
        uint8_t *a8 = sfa + align256(sc);
        bd_qtensor xq{nullptr, nullptr, sfa, M, K};
        s = launch_contig<BD_SELECT_TWO_STAGE, false, true>(X, xdtype, ldx, view_of(&xq), a8, st);
        if (s) return s;
        int kernels = 1;
        s = cuda_result(tc::launch(a8, sfa, M, view_of(Wq), K, Y, ydtype == BD_BF16, ldy, st,
                                   a8 + tc_operand_bytes(M, K), tc::splitk_workspace(M, N, K), &kernels));
        g_launches += (uint64_t)kernels;
        return s;
    }
    bd_qtensor xq{p, p + align256(c), p + align256(c) + align256(i), M, K};
    s = launch_contig<BD_SELECT_TWO_STAGE, true, false>(X, xdtype, ldx, view_of(&xq), nullptr, st);
    if (s) return s;
    return gemm_dispatch(view_of(&xq), view_of(Wq), Y, ydtype, ldy, nullptr, 0, st);
}

// ---- products whose result is requantised for the next product (Sec. 3.3, last paragraph) ----
namespace {
bool requant_fused(int64_t M, int64_t N, int64_t K) {
    // the tensor-core kernel's requantising epilogue serves items of 128 or 256 tokens
    return g_gemm_impl != BD_GEMM_SIMT && tc_supported(M, N, K) && M > tc::kSplitMaxTokens;
}
size_t requant_extra(int64_t M, int64_t N, int64_t K) {            // fp32 result in scratch when the epilogue cannot requantise
    return requant_fused(M, N, K) ? 0 : align256((size_t)M * (size_t)N * sizeof(float));
}
bd_status check_requant_out(const bd_qtensor *Yq, int64_t M, int64_t N) {
    bd_status s = check_qtensor(Yq);
    if (s) return s;
    if (Yq->rows != M || Yq->K != N) return BD_ERR_SHAPE;          // (N % 32 is part of check_qtensor)
    return BD_OK;
}
}  // namespace

bd_status bd_linear_requant_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes) {
    bd_status s = bd_linear_workspace_size(M, N, K, bytes);
    if (s) return s;
    if (N % kBlock) return BD_ERR_SHAPE;
    *bytes = align256(*bytes) + requant_extra(M, N, K);
    return BD_OK;
}

bd_status bd_gemm_requant_workspace_size(int64_t M, int64_t N, int64_t K, size_t *bytes) {
    bd_status s = bd_gemm_workspace_size(M, N, K, bytes);
    if (s) return s;
    if (N % kBlock) return BD_ERR_SHAPE;
    *bytes = align256(*bytes) + requant_extra(M, N, K);
    return BD_OK;
}

bd_status bd_linear_requant(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, const bd_qtensor *Wq,
                            bd_qtensor *Yq, void *workspace, size_t workspace_bytes, void *stream) {
    bd_status s = check_source(X, xdtype, M, K, ldx, K);
    if (s) return s;
    s = check_qtensor(Wq);
    if (s) return s;
    if (Wq->K != K) return BD_ERR_SHAPE;
    const int64_t N = Wq->rows;
    s = check_requant_out(Yq, M, N);
    if (s) return s;
    size_t need, base;
    bd_linear_requant_workspace_size(M, N, K, &need);
    bd_linear_workspace_size(M, N, K, &base);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (requant_fused(M, N, K)) {
        size_t c, i, sc;
        bd_qtensor_sizes(M, K, &c, &i, &sc);
        uint8_t *sfa = (uint8_t *)workspace, *a8 = sfa + align256(sc);
        bd_qtensor xq{nullptr, nullptr, sfa, M, K};
        s = launch_contig<BD_SELECT_TWO_STAGE, false, true>(X, xdtype, ldx, view_of(&xq), a8, st);
        if (s) return s;
        const QView out = view_of(Yq);
        s = cuda_result(tc::launch(a8, sfa, M, view_of(Wq), K, nullptr, false, N, st, nullptr, 0, nullptr, &out));
        g_launches += 1;
        return s;
    }
    // short calls and the CUDA-core route: the fp32 result goes to scratch and the quantizer reads it from there
    float *y32 = (float *)((char *)workspace + align256(base));
    s = bd_linear(X, xdtype, M, K, ldx, Wq, y32, BD_F32, N, workspace, base, stream);
    if (s) return s;
    return launch_contig<BD_SELECT_TWO_STAGE, true, false>(y32, BD_F32, N, view_of(Yq), nullptr, st);
}

bd_status bd_gemm_requant(const bd_qtensor *A, const bd_qtensor *B, bd_qtensor *Yq, void *workspace, size_t workspace_bytes,
                          void *stream) {
    bd_status s = check_qtensor(A);
    if (s) return s;
    s = check_qtensor(B);
    if (s) return s;
    if (A->K != B->K) return BD_ERR_SHAPE;
    const int64_t M = A->rows, N = B->rows, K = A->K;
    s = check_requant_out(Yq, M, N);
    if (s) return s;
    size_t need, base;
    bd_gemm_requant_workspace_size(M, N, K, &need);
    bd_gemm_workspace_size(M, N, K, &base);
    if (need && (!workspace || workspace_bytes < need)) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (requant_fused(M, N, K)) {
        const QView a = view_of(A), out = view_of(Yq);
        uint8_t *a8 = (uint8_t *)workspace;
        const int nb = (int)(K / kBlock);
        decode_e4m3_kernel<<<grid_for(M * nb, 256), 256, 0, st>>>(a, a8, nb);
        s = launch_result(1);
        if (s) return s;
        s = cuda_result(tc::launch(a8, a.scales, M, view_of(B), K, nullptr, false, N, st, nullptr, 0, nullptr, &out));
        g_launches += 1;
        return s;
    }
    float *y32 = (float *)((char *)workspace + align256(base));
    s = gemm_dispatch(view_of(A), view_of(B), y32, BD_F32, N, workspace, base, st);
    if (s) return s;
    return launch_contig<BD_SELECT_TWO_STAGE, true, false>(y32, BD_F32, N, view_of(Yq), nullptr, st);
}

bd_status bd_linear_noalloc(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, const bd_qtensor *Wq,
                            void *Y, bd_dtype ydtype, int64_t ldy, void *stream) {
    if (!Wq || M <= 0 || K <= 0 || Wq->rows <= 0) return BD_ERR_INVALID_ARG;
    size_t need = 0;
    bd_status s = bd_linear_workspace_size(M, Wq->rows, K, &need);
    if (s) return s;
    if (need > (size_t)BD_NOALLOC_SCRATCH_BYTES) return BD_ERR_SCRATCH_LIMIT;
    int dev = -1;
    s = cuda_result(cudaGetDevice(&dev));
    if (s) return s;
    if (dev < 0 || dev >= kMaxDevices) return BD_ERR_UNSUPPORTED;
    if (!g_noalloc_ptr[dev]) {                       // first call on this device: resolve the symbol
        void *p = nullptr;
        s = cuda_result(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (s) return s;
        g_noalloc_ptr[dev] = p;
    }
    return bd_linear(X, xdtype, M, K, ldx, Wq, Y, ydtype, ldy, g_noalloc_ptr[dev], BD_NOALLOC_SCRATCH_BYTES, stream);
}

// ---- block sizes 16 and 64 (Sec. 4.2, Table 3) ----
bd_status bd_qtensor_sizes_bs(int64_t rows, int64_t K, int block, size_t *codes_bytes, size_t *ids_bytes, size_t *scales_bytes) {
    if (!block_size_ok(block)) return BD_ERR_INVALID_ARG;
    if (rows <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (K % block) return BD_ERR_SHAPE;
    return bd_qtensor_sizes(rows, physical_k(K, block), codes_bytes, ids_bytes, scales_bytes);
}

bd_status bd_quantize_bs(const void *X, bd_dtype dtype, int64_t rows, int64_t K, int64_t ld, bd_select select, int block,
                         bd_qtensor *out, void *stream) {
    if (!block_size_ok(block) || (select != BD_SELECT_TWO_STAGE && select != BD_SELECT_MSE)) return BD_ERR_INVALID_ARG;
    if (!X || rows <= 0 || K <= 0 || (dtype != BD_F32 && dtype != BD_BF16 && dtype != BD_F16)) return BD_ERR_INVALID_ARG;
    if (K % block || ld < K) return BD_ERR_SHAPE;
    if (!aligned16(X) || (ld * elem_bytes(dtype)) % 16) return BD_ERR_ALIGN;
    bd_status s = check_qtensor(out);
    if (s) return s;
    if (out->rows != rows || out->K != physical_k(K, block)) return BD_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (block == 32) {
        if (select == BD_SELECT_MSE) return launch_contig<BD_SELECT_MSE, true, false>(X, dtype, ld, view_of(out), nullptr, st);
        return launch_contig<BD_SELECT_TWO_STAGE, true, false>(X, dtype, ld, view_of(out), nullptr, st);
    }
    if (block == 16) return quantize_bs_dtype<16>(X, dtype, ld, select, view_of(out), st);
    return quantize_bs_dtype<64>(X, dtype, ld, select, view_of(out), st);
}

bd_status bd_export_canonical_bs(const bd_qtensor *q, int block, uint8_t *codes, uint8_t *ids, uint8_t *scales, void *stream) {
    if (!block_size_ok(block)) return BD_ERR_INVALID_ARG;
    if (block == 32) return bd_export_canonical(q, codes, ids, scales, stream);
    bd_status s = check_qtensor(q);
    if (s) return s;
    if (!codes || !ids || !scales) return BD_ERR_INVALID_ARG;
    if (!aligned16(codes)) return BD_ERR_ALIGN;
    if (q->K % 64) return BD_ERR_SHAPE;                            // K' = 2 K with K % 16 == 0 ... K % 64 == 0 for block 64
    const int nbp = (int)(q->K / kBlock);
    const unsigned grid = grid_for(q->rows * nbp, 256);
    if (block == 16) export_canonical_bs_kernel<16><<<grid, 256, 0, (cudaStream_t)stream>>>(view_of(q), codes, ids, scales, nbp);
    else export_canonical_bs_kernel<64><<<grid, 256, 0, (cudaStream_t)stream>>>(view_of(q), codes, ids, scales, nbp);
    return launch_result();
}

bd_status bd_linear_bs_workspace_size(int64_t M, int64_t N, int64_t K, int block, size_t *bytes) {
    if (!bytes || !block_size_ok(block) || M <= 0 || N <= 0 || K <= 0) return BD_ERR_INVALID_ARG;
    if (K % block) return BD_ERR_SHAPE;
    const int64_t Kp = physical_k(K, block);
    if (block == 32) return bd_linear_workspace_size(M, N, K, bytes);
    size_t c, i, s, g;
    bd_qtensor_sizes(M, Kp, &c, &i, &s);
    bd_gemm_workspace_size(M, N, Kp, &g);
    *bytes = align256(c) + align256(i) + align256(s) + g;
    return BD_OK;
}

bd_status bd_linear_bs(const void *X, bd_dtype xdtype, int64_t M, int64_t K, int64_t ldx, int block, const bd_qtensor *Wq, void *Y,
                       bd_dtype ydtype, int64_t ldy, void *workspace, size_t workspace_bytes, void *stream) {
    if (!block_size_ok(block)) return BD_ERR_INVALID_ARG;
    if (block == 32) return bd_linear(X, xdtype, M, K, ldx, Wq, Y, ydtype, ldy, workspace, workspace_bytes, stream);
    if (K <= 0 || K % block) return BD_ERR_SHAPE;
    bd_status s = check_qtensor(Wq);
    if (s) return s;
    const int64_t Kp = physical_k(K, block), N = Wq->rows;
    if (Wq->K != Kp || ldy < N) return BD_ERR_SHAPE;
    if (!Y || (ydtype != BD_F32 && ydtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    size_t need;
    s = bd_linear_bs_workspace_size(M, N, K, block, &need);
    if (s) return s;
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    size_t c, i, sc, g;
    bd_qtensor_sizes(M, Kp, &c, &i, &sc);
    bd_gemm_workspace_size(M, N, Kp, &g);
    char *p = (char *)workspace;
    bd_qtensor xq{p, p + align256(c), p + align256(c) + align256(i), M, Kp};
    s = bd_quantize_bs(X, xdtype, M, K, ldx, BD_SELECT_TWO_STAGE, block, &xq, stream);
    if (s) return s;
    return gemm_dispatch(view_of(&xq), view_of(Wq), Y, ydtype, ldy, p + align256(c) + align256(i) + align256(sc), g, (cudaStream_t)stream);
}

// ---- KV cache (appendix "Quantization Dimension", Fig. 9b) ----
static bd_status check_kvcache(const bd_kvcache *c) {
    if (!c || !c->v_recent) return BD_ERR_INVALID_ARG;
    bd_status s = check_qtensor(&c->k);
    if (s) return s;
    s = check_qtensor(&c->v);
    if (s) return s;
    if (c->dtype != BD_F32 && c->dtype != BD_BF16 && c->dtype != BD_F16) return BD_ERR_INVALID_ARG;
    if (c->head_dim <= 0 || c->head_dim % kBlock || c->head_dim > 128 || c->capacity <= 0 || c->capacity % kBlock) return BD_ERR_SHAPE;
    if (c->k.rows != c->capacity || c->k.K != c->head_dim || c->v.rows != c->head_dim || c->v.K != c->capacity) return BD_ERR_SHAPE;
    if (c->length < 0 || c->length > c->capacity) return BD_ERR_SHAPE;
    if (!aligned16(c->v_recent)) return BD_ERR_ALIGN;
    return BD_OK;
}

bd_status bd_kvcache_recent_bytes(int64_t head_dim, bd_dtype dtype, size_t *bytes) {
    if (!bytes || head_dim <= 0) return BD_ERR_INVALID_ARG;
    *bytes = (size_t)kBlock * (size_t)head_dim * (size_t)elem_bytes(dtype);
    return BD_OK;
}

bd_status bd_kvcache_reset(bd_kvcache *c, void *stream) {
    bd_status s = check_kvcache(c);
    if (s) return s;
    size_t cb, ib, sb;
    cudaStream_t st = (cudaStream_t)stream;
    bd_qtensor_sizes(c->capacity, c->head_dim, &cb, &ib, &sb);
    if ((s = cuda_result(cudaMemsetAsync(c->k.ids, 0, ib, st)))) return s;
    if ((s = cuda_result(cudaMemsetAsync(c->k.scales, 0, sb, st)))) return s;
    bd_qtensor_sizes(c->head_dim, c->capacity, &cb, &ib, &sb);
    if ((s = cuda_result(cudaMemsetAsync(c->v.ids, 0, ib, st)))) return s;
    if ((s = cuda_result(cudaMemsetAsync(c->v.scales, 0, sb, st)))) return s;
    c->length = 0;
    return BD_OK;
}

namespace {
// t new tokens for n heads (n = 1: `c` alone, no batch): the same launches, grid.y = head.
bd_status kv_append(bd_kvcache *c, int64_t n, const void *Knew, const void *Vnew, int64_t t, int64_t ldk, int64_t ldv, int64_t stride_k,
                    int64_t stride_v, cudaStream_t st) {
    const int64_t d = c->head_dim;
    const int esz = elem_bytes(c->dtype);
    KvBatch kb{}, vb{};
    const KvBatch *pk = nullptr, *pv = nullptr;
    if (n > 1) {
        for (int64_t i = 0; i < n; i++) {
            kb.codes[i] = (uint8_t *)c[i].k.codes; kb.ids[i] = (uint8_t *)c[i].k.ids; kb.scales[i] = (uint8_t *)c[i].k.scales;
            vb.codes[i] = (uint8_t *)c[i].v.codes; vb.ids[i] = (uint8_t *)c[i].v.ids; vb.scales[i] = (uint8_t *)c[i].v.scales;
            kb.recent[i] = vb.recent[i] = c[i].v_recent;
        }
        pk = &kb;
        pv = &vb;
    }
    const QView kq = view_of(&c->k), vq = view_of(&c->v);
    int kernels = 0;
    // keys: one quantisation per new token, appended as rows
    BD_KV_DISPATCH(c->dtype, launch_kv_keys, Knew, ldk, t, kq, c->length, st, pk, (int)n, stride_k);
    kernels++;
    // values: complete the waiting chunk, then whole chunks straight from the source, then the new remainder
    int64_t done = 0, len = c->length;
    const int waiting = (int)(len % kBlock);
    if (waiting) {
        const int fill = (int)std::min<int64_t>(kBlock - waiting, t);
        launch_kv_recent(Vnew, ldv * esz, fill, (int)(d * esz), c->v_recent, waiting, st, pv, (int)n, stride_v * esz);
        kernels++;
        if (waiting + fill == kBlock) {
            BD_KV_DISPATCH(c->dtype, launch_kv_chunks, n > 1 ? nullptr : c->v_recent, d, 1, vq, (int)(len / kBlock), st, pv, (int)n, (int64_t)0);
            kernels++;
        }
        done = fill;
        len += fill;
    }
    const int64_t whole = (t - done) / kBlock;
    if (whole) {
        BD_KV_DISPATCH(c->dtype, launch_kv_chunks, (const char *)Vnew + done * ldv * esz, ldv, (int)whole, vq, (int)(len / kBlock), st, pv, (int)n, stride_v);
        kernels++;
        done += whole * kBlock;
    }
    if (done < t) {
        const int rest = (int)(t - done);
        launch_kv_recent((const char *)Vnew + done * ldv * esz, ldv * esz, rest, (int)(d * esz), c->v_recent, 0, st, pv, (int)n, stride_v * esz);
        kernels++;
    }
    for (int64_t i = 0; i < n; i++) c[i].length += t;
    return launch_result(kernels);
}
bd_status check_append(const bd_kvcache *c, const void *Knew, const void *Vnew, int64_t t, int64_t ldk, int64_t ldv) {
    if (!Knew || !Vnew || t <= 0) return BD_ERR_INVALID_ARG;
    const int64_t d = c->head_dim;
    const int esz = elem_bytes(c->dtype);
    if (ldk < d || ldv < d || c->length + t > c->capacity) return BD_ERR_SHAPE;
    if (!aligned16(Knew) || !aligned16(Vnew) || (ldk * esz) % 16 || (ldv * esz) % 16) return BD_ERR_ALIGN;
    return BD_OK;
}
}  // namespace

bd_status bd_kvcache_append(bd_kvcache *c, const void *Knew, const void *Vnew, int64_t t, int64_t ldk, int64_t ldv, void *stream) {
    bd_status s = check_kvcache(c);
    if (s) return s;
    s = check_append(c, Knew, Vnew, t, ldk, ldv);
    if (s) return s;
    return kv_append(c, 1, Knew, Vnew, t, ldk, ldv, 0, 0, (cudaStream_t)stream);
}

bd_status bd_kvcache_workspace_size(int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes) {
    if (!bytes || capacity <= 0 || head_dim <= 0 || q_rows <= 0) return BD_ERR_INVALID_ARG;
    if (capacity % kBlock || head_dim % kBlock) return BD_ERR_SHAPE;
    size_t g1, g2, cb, ib, sb;
    bd_gemm_workspace_size(q_rows, capacity, head_dim, &g1);       // scores
    bd_gemm_workspace_size(q_rows, head_dim, capacity, &g2);       // P x V over the stored chunks
    bd_qtensor_sizes(q_rows, capacity, &cb, &ib, &sb);            // the quantised probabilities
    const size_t pv = align256(cb) + align256(ib) + align256(sb) + align256(g2) + align256((size_t)q_rows * head_dim * sizeof(float));
    *bytes = std::max(align256(g1), pv);
    return BD_OK;
}

namespace {
bool kv_batch_fused(int64_t n, int64_t q_rows, int64_t N, int64_t K);   // (with the batched calls below)
}

bd_status bd_kvcache_scores(const bd_kvcache *c, const bd_qtensor *Q, void *S, bd_dtype sdtype, int64_t lds, void *workspace,
                            size_t workspace_bytes, void *stream) {
    bd_status s = check_kvcache(c);
    if (s) return s;
    s = check_qtensor(Q);
    if (s) return s;
    if (Q->K != c->head_dim || c->length == 0 || lds < c->length) return BD_ERR_SHAPE;
    if (!S || (sdtype != BD_F32 && sdtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    if (kv_batch_fused(1, Q->rows, c->length, c->head_dim))       // a few query rows: the batched route with one head
        return bd_kvcache_scores_batched(c, 1, Q, S, sdtype, lds, Q->rows * lds, workspace, workspace_bytes, stream);
    QView keys = view_of(&c->k);
    keys.rows = c->length;                                        // the rows stored so far (one scale atom along K: the
    return gemm_dispatch(view_of(Q), keys, S, sdtype, lds, workspace, workspace_bytes, (cudaStream_t)stream);   // atom order ignores the row count)
}

bd_status bd_kvcache_pv(const bd_kvcache *c, const float *P, int64_t q_rows, int64_t ldp, void *Y, bd_dtype ydtype, int64_t ldy,
                        void *workspace, size_t workspace_bytes, void *stream) {
    bd_status s = check_kvcache(c);
    if (s) return s;
    if (!P || !Y || q_rows <= 0 || (ydtype != BD_F32 && ydtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    if (c->length == 0 || ldp < c->length || ldy < c->head_dim) return BD_ERR_SHAPE;
    if (c->length >= kBlock && (!aligned16(P) || (ldp * 4) % 16)) return BD_ERR_ALIGN;   // the quantizer reads P in 16-byte pieces
    if (kv_batch_fused(1, q_rows, c->head_dim, c->length >= kBlock ? c->length / kBlock * kBlock : kBlock))
        return bd_kvcache_pv_batched(c, 1, P, q_rows, ldp, q_rows * ldp, Y, ydtype, ldy, q_rows * ldy, workspace, workspace_bytes, stream);
    size_t need;
    bd_kvcache_workspace_size(c->capacity, c->head_dim, q_rows, &need);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t d = c->head_dim, n_q = c->length / kBlock * kBlock;
    const int n_recent = (int)(c->length - n_q);
    float *part = nullptr;
    if (n_q) {
        // probabilities over the stored chunks: quantised online along the keys, then the block-scaled product
        size_t cb, ib, sb, g2;
        bd_qtensor_sizes(q_rows, n_q, &cb, &ib, &sb);
        bd_gemm_workspace_size(q_rows, d, n_q, &g2);
        char *p = (char *)workspace;
        bd_qtensor pq{p, p + align256(cb), p + align256(cb) + align256(ib), q_rows, n_q};
        char *gws = p + align256(cb) + align256(ib) + align256(sb);
        part = (float *)(gws + align256(g2));
        QView vals = view_of(&c->v);
        vals.K = n_q;                                             // the first n_q tokens of every channel; the pitch stays
        if (use_warp(q_rows, d, n_q) && wk::supported(q_rows, d, n_q)) {
            // a few query rows: the probabilities go straight into the warp-level kernel's records
            s = launch_warp_linear(P, BD_F32, q_rows, n_q, ldp, vals, part, BD_F32, d, gws, st);
        } else {
            s = launch_contig<BD_SELECT_TWO_STAGE, true, false>(P, BD_F32, ldp, view_of(&pq), nullptr, st);
            if (s) return s;
            s = gemm_dispatch(view_of(&pq), vals, part, BD_F32, d, gws, g2, st);
        }
        if (s) return s;
    }
    BD_KV_DISPATCH(c->dtype, launch_kv_finish, part, d, P, ldp, n_q, n_recent, c->v_recent, (int)d, q_rows, Y, ydtype, ldy, st);
    return launch_result();
}

// ---- the same two calls for the KV heads of a layer at once ----
namespace {
bd_status check_kvcache_batch(const bd_kvcache *c, int64_t n) {
    if (!c || n <= 0) return BD_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; i++) {
        bd_status s = check_kvcache(&c[i]);
        if (s) return s;
        if (c[i].capacity != c[0].capacity || c[i].head_dim != c[0].head_dim || c[i].length != c[0].length || c[i].dtype != c[0].dtype)
            return BD_ERR_SHAPE;
    }
    return BD_OK;
}
// P x V of n heads with the probabilities' records at `records` (rec_stride bytes per head): the product over the stored
// chunks and, in its epilogue, the recent tokens in high precision.
bd_status kv_pv_product(const bd_kvcache *c, int64_t n, const float *P, int64_t q_rows, int64_t ldp, int64_t stride_p, int64_t n_q, int n_recent,
                        const void *records, int64_t rec_stride, void *Y, bd_dtype ydtype, int64_t ldy, int64_t stride_y, cudaStream_t st) {
    wk::OperandBatch vb{};
    wk::Extra x{};
    for (int64_t i = 0; i < n; i++) {
        vb.codes[i] = (const uint8_t *)c[i].v.codes; vb.ids[i] = (const uint8_t *)c[i].v.ids; vb.scales[i] = (const uint8_t *)c[i].v.scales;
        x.recent[i] = c[i].v_recent;
    }
    x.P = P; x.ldp = ldp; x.p_stride = stride_p; x.n_q = (int)n_q; x.n_recent = n_recent; x.recent_dt = (int)c[0].dtype;
    QView vals = view_of(&c[0].v);
    vals.K = n_q;
    return launch_warp_attn(2, q_rows, n_q, vals, Y, ydtype, ldy, stride_y, records, rec_stride, vb, x, (int)n, st);
}
bool kv_batch_fused(int64_t n, int64_t q_rows, int64_t N, int64_t K) {
    return n <= wk::kMaxBatch && g_gemm_impl != BD_GEMM_SIMT && g_gemm_impl != BD_GEMM_TCGEN05 && wk::supported(q_rows, N, K);
}
}  // namespace

bd_status bd_kvcache_append_batched(bd_kvcache *c, int64_t n, const void *Knew, const void *Vnew, int64_t t, int64_t ldk, int64_t ldv,
                                    int64_t stride_k, int64_t stride_v, void *stream) {
    bd_status s = check_kvcache_batch(c, n);
    if (s) return s;
    s = check_append(c, Knew, Vnew, t, ldk, ldv);
    if (s) return s;
    const int esz = elem_bytes(c->dtype);
    if (n > 1 && ((stride_k * esz) % 16 || (stride_v * esz) % 16)) return BD_ERR_ALIGN;
    if (n > kKvMaxBatch) {                                        // more heads than a launch takes: head by head
        for (int64_t i = 0; i < n; i++) {
            s = kv_append(&c[i], 1, (const char *)Knew + i * stride_k * esz, (const char *)Vnew + i * stride_v * esz, t, ldk, ldv, 0, 0, (cudaStream_t)stream);
            if (s) return s;
        }
        return BD_OK;
    }
    return kv_append(c, n, Knew, Vnew, t, ldk, ldv, stride_k, stride_v, (cudaStream_t)stream);
}

bd_status bd_kvcache_batched_workspace_size(int64_t n, int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes) {
    if (n <= 0) return BD_ERR_INVALID_ARG;
    size_t one;
    bd_status s = bd_kvcache_workspace_size(capacity, head_dim, q_rows, &one);
    if (s) return s;
    *bytes = (size_t)n * align256(one);
    return BD_OK;
}

bd_status bd_kvcache_scores_batched(const bd_kvcache *c, int64_t n, const bd_qtensor *Q, void *S, bd_dtype sdtype, int64_t lds,
                                    int64_t stride_s, void *workspace, size_t workspace_bytes, void *stream) {
    bd_status s = check_kvcache_batch(c, n);
    if (s) return s;
    if (!Q || !S || (sdtype != BD_F32 && sdtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    for (int64_t i = 0; i < n; i++) {
        s = check_qtensor(&Q[i]);
        if (s) return s;
        if (Q[i].K != c[0].head_dim || Q[i].rows != Q[0].rows) return BD_ERR_SHAPE;
    }
    const int64_t len = c[0].length, q_rows = Q[0].rows, hd = c[0].head_dim;
    if (len == 0 || lds < len || (n > 1 && stride_s < q_rows * lds)) return BD_ERR_SHAPE;
    size_t one, need;
    bd_kvcache_workspace_size(c[0].capacity, hd, q_rows, &one);
    bd_kvcache_batched_workspace_size(n, c[0].capacity, hd, q_rows, &need);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t esz = sdtype == BD_F32 ? 4 : 2;
    if (!kv_batch_fused(n, q_rows, len, hd)) {
        for (int64_t i = 0; i < n; i++) {
            s = bd_kvcache_scores(&c[i], &Q[i], (char *)S + i * stride_s * esz, sdtype, lds, (char *)workspace + i * align256(one), one, stream);
            if (s) return s;
        }
        return BD_OK;
    }
    // one launch, grid.y = head: the product kernel builds its B fragments from the queries' codes
    wk::OperandBatch kb{};
    wk::Extra x{};
    for (int64_t i = 0; i < n; i++) {
        x.a_codes[i] = (const uint8_t *)Q[i].codes; x.a_ids[i] = (const uint8_t *)Q[i].ids; x.a_scales[i] = (const uint8_t *)Q[i].scales;
        kb.codes[i] = (const uint8_t *)c[i].k.codes; kb.ids[i] = (const uint8_t *)c[i].k.ids; kb.scales[i] = (const uint8_t *)c[i].k.scales;
    }
    x.a_ldc = hd / 2;
    QView keys = view_of(&c[0].k);
    keys.rows = len;
    return launch_warp_attn(1, q_rows, hd, keys, S, sdtype, lds, stride_s, workspace, 0, kb, x, (int)n, st);
}

bd_status bd_kvcache_pv_batched(const bd_kvcache *c, int64_t n, const float *P, int64_t q_rows, int64_t ldp, int64_t stride_p, void *Y,
                                bd_dtype ydtype, int64_t ldy, int64_t stride_y, void *workspace, size_t workspace_bytes, void *stream) {
    bd_status s = check_kvcache_batch(c, n);
    if (s) return s;
    if (!P || !Y || q_rows <= 0 || (ydtype != BD_F32 && ydtype != BD_BF16)) return BD_ERR_INVALID_ARG;
    const int64_t len = c[0].length, d = c[0].head_dim;
    if (len == 0 || ldp < len || ldy < d || (n > 1 && (stride_p < q_rows * ldp || stride_y < q_rows * ldy))) return BD_ERR_SHAPE;
    if (len >= kBlock && (!aligned16(P) || (ldp * 4) % 16 || (stride_p * 4) % 16)) return BD_ERR_ALIGN;
    size_t one, need;
    bd_kvcache_workspace_size(c[0].capacity, d, q_rows, &one);
    bd_kvcache_batched_workspace_size(n, c[0].capacity, d, q_rows, &need);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t esz = ydtype == BD_F32 ? 4 : 2;
    const int64_t n_q = len / kBlock * kBlock;
    const int n_recent = (int)(len - n_q);
    if (!kv_batch_fused(n, q_rows, d, n_q ? n_q : kBlock)) {
        for (int64_t i = 0; i < n; i++) {
            s = bd_kvcache_pv(&c[i], P + i * stride_p, q_rows, ldp, (char *)Y + i * stride_y * esz, ydtype, ldy, (char *)workspace + i * align256(one), one, stream);
            if (s) return s;
        }
        return BD_OK;
    }
    // records of all heads' probabilities over the stored chunks, then one product kernel whose epilogue adds the
    // recent tokens in high precision and writes the result: two launches, grid.y = head
    const int64_t rec_stride = n_q ? (int64_t)align256(wk::record_bytes(n_q, q_rows > wk::kTokTile ? 2 : 1)) : 0;
    if (n_q) {
        s = launch_warp_records(P, BD_F32, q_rows, n_q, ldp, workspace, st, (int)n, stride_p, rec_stride);
        if (s) return s;
    }
    return kv_pv_product(c, n, P, q_rows, ldp, stride_p, n_q, n_recent, workspace, rec_stride, Y, ydtype, ldy, stride_y, st);
}

// ---- a decode step's attention over the cached heads: scores, softmax in high precision, P x V ----
bd_status bd_kvcache_attention_workspace_size(int64_t n, int64_t capacity, int64_t head_dim, int64_t q_rows, size_t *bytes) {
    size_t kv;
    bd_status s = bd_kvcache_batched_workspace_size(n, capacity, head_dim, q_rows, &kv);
    if (s) return s;
    *bytes = align256(kv) + align256((size_t)n * (size_t)q_rows * (size_t)capacity * sizeof(float));   // + the scores / probabilities
    return BD_OK;
}

bd_status bd_kvcache_attention(const bd_kvcache *c, int64_t n, const bd_qtensor *Q, float scale, void *O, bd_dtype odtype, int64_t ldo,
                               int64_t stride_o, float *P_out, int64_t ldp_out, int64_t stride_p_out, void *workspace,
                               size_t workspace_bytes, void *stream) {
    bd_status s = check_kvcache_batch(c, n);
    if (s) return s;
    if (!Q || !O) return BD_ERR_INVALID_ARG;
    const int64_t q_rows = Q[0].rows, len = c[0].length, cap = c[0].capacity, d = c[0].head_dim;
    if (q_rows <= 0 || len == 0) return BD_ERR_SHAPE;
    size_t need, kv;
    bd_kvcache_attention_workspace_size(n, cap, d, q_rows, &need);
    bd_kvcache_batched_workspace_size(n, cap, d, q_rows, &kv);
    if (!workspace || workspace_bytes < need) return BD_ERR_WORKSPACE;
    if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
    // the probabilities live in the caller's buffer when one is given (then it is also an output), else in the workspace
    float *P = P_out ? P_out : (float *)((char *)workspace + align256(kv));
    const int64_t ldp = P_out ? ldp_out : cap, stride_p = P_out ? stride_p_out : q_rows * cap;
    if (P_out && (ldp < len || (n > 1 && stride_p < q_rows * ldp))) return BD_ERR_SHAPE;
    if (P_out && (!aligned16(P_out) || (ldp * 4) % 16 || (stride_p * 4) % 16)) return BD_ERR_ALIGN;
    s = bd_kvcache_scores_batched(c, n, Q, P, BD_F32, ldp, stride_p, workspace, kv, stream);
    if (s) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n_q = len / kBlock * kBlock;
    if (kv_batch_fused(n, q_rows, d, n_q ? n_q : kBlock)) {
        // the softmax kernel also quantises its rows into the second product's records; that product's epilogue adds
        // the recent tokens: three launches for the step
        const int nt = q_rows > wk::kTokTile ? 2 : 1;
        const int64_t rec_stride = (int64_t)align256(wk::record_bytes(n_q ? n_q : kBlock, nt));
        uint8_t *rec16 = (uint8_t *)workspace;
        float *recs = (float *)(rec16 + (size_t)wk::padded_blocks(n_q) * nt * wk::kRecBytes);
        launch_serialized(kv_softmax_records_kernel, dim3((unsigned)(wk::kTokTile * nt), (unsigned)n), 256, 0, st, P, ldp, stride_p, len, scale,
                          (int)q_rows, nt, (int)n_q, (int)wk::padded_blocks(n_q), rec16, recs, rec_stride);
        s = launch_result(1);
        if (s) return s;
        return kv_pv_product(c, n, P, q_rows, ldp, stride_p, n_q, (int)(len - n_q), workspace, rec_stride, O, odtype, ldo, stride_o, st);
    }
    if (stride_p == q_rows * ldp) {
        kv_softmax_rows_kernel<<<(unsigned)(n * q_rows), 256, 0, st>>>(P, ldp, len, scale);
        s = launch_result(1);
        if (s) return s;
    } else {
        for (int64_t i = 0; i < n; i++) {
            kv_softmax_rows_kernel<<<(unsigned)q_rows, 256, 0, st>>>(P + i * stride_p, ldp, len, scale);
            s = launch_result(1);
            if (s) return s;
        }
    }
    return bd_kvcache_pv_batched(c, n, P, q_rows, ldp, stride_p, O, odtype, ldo, stride_o, workspace, kv, stream);
}

// ---- fused full-path attention ----
bd_status bd_attention_workspace_size(int64_t heads, int64_t group, int64_t sk, int64_t head_dim, size_t *bytes) {
    if (!bytes || heads <= 0 || group <= 0 || heads % group || sk <= 0 || head_dim <= 0) return BD_ERR_INVALID_ARG;
    // K and V of the KV heads of one launch as bf16
    const int64_t per_launch = std::min<int64_t>(heads / group, std::max<int64_t>(1, std::min<int64_t>(attn::kMaxKvHeads, attn::kMaxHeads / group)));
    *bytes = (size_t)2 * (size_t)per_launch * align256((size_t)sk * head_dim * 2);
    return BD_OK;
}

bd_status bd_attention(const bd_qtensor *Q, const bd_qtensor *K, const bd_qtensor *V, int64_t heads, int64_t group, float scale,
                       void *O, bd_dtype odtype, int64_t ldo, int64_t stride_o, const bd_attention_dump *dump, void *workspace,
                       size_t workspace_bytes, void *stream) {
    if (!Q || !K || !V || !O || heads <= 0 || group <= 0 || heads % group) return BD_ERR_INVALID_ARG;
    if (odtype != BD_F32 && odtype != BD_BF16) return BD_ERR_INVALID_ARG;
    const int64_t kv = heads / group, sq = Q[0].rows, hd = Q[0].K, sk = K[0].rows;
    if (hd != 128 && hd != 64) return BD_ERR_UNSUPPORTED;
    if (sk % kBlock || ldo < hd) return BD_ERR_SHAPE;
    if (!aligned16(O) || (ldo * (odtype == BD_F32 ? 4 : 2)) % 16) return BD_ERR_ALIGN;
    for (int64_t h = 0; h < heads; h++) {
        bd_status s = check_qtensor(&Q[h]);
        if (s) return s;
        if (Q[h].rows != sq || Q[h].K != hd) return BD_ERR_SHAPE;
    }
    for (int64_t g = 0; g < kv; g++) {
        bd_status s = check_qtensor(&K[g]);
        if (s) return s;
        s = check_qtensor(&V[g]);
        if (s) return s;
        if (K[g].rows != sk || K[g].K != hd || V[g].rows != hd || V[g].K != sk) return BD_ERR_SHAPE;
    }
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev]) {
        if (cudaFuncSetAttribute(attn::attention_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn::Layout<128>::total) != cudaSuccess ||
            cudaFuncSetAttribute(attn::attention_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn::Layout<64>::total) != cudaSuccess ||
            cudaFuncSetAttribute(attn::attention_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn::Layout<128>::total) != cudaSuccess ||
            cudaFuncSetAttribute(attn::attention_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn::Layout<64>::total) != cudaSuccess)
            return launch_result(0);
        configured[dev] = true;
    }
    // heads per launch: whole KV groups, as many as the argument block holds
    const int64_t groups_per_launch = std::max<int64_t>(1, std::min<int64_t>(attn::kMaxKvHeads, attn::kMaxHeads / group));
    if (group > attn::kMaxHeads) return BD_ERR_UNSUPPORTED;
    // with a workspace the KV heads' operands are expanded to bf16 once per launch and the kernel copies its key tiles
    bool pre = false;
    const size_t exp_bytes = align256((size_t)sk * hd * 2);
    if (workspace) {
        size_t need;
        bd_attention_workspace_size(heads, group, sk, hd, &need);
        if (workspace_bytes < need) return BD_ERR_WORKSPACE;
        if ((uintptr_t)workspace & 255u) return BD_ERR_ALIGN;
        pre = true;
    }
    uint8_t *k_exp = (uint8_t *)workspace, *v_exp = k_exp + (size_t)std::min(groups_per_launch, kv) * exp_bytes;
    int kernels = 0;
    for (int64_t g0 = 0; g0 < kv; g0 += groups_per_launch) {
        const int64_t ng = std::min(groups_per_launch, kv - g0), nh = ng * group, h0 = g0 * group;
        attn::Params p = {};
        for (int64_t h = 0; h < nh; h++) {
            p.q_codes[h] = (const uint8_t *)Q[h0 + h].codes; p.q_ids[h] = (const uint8_t *)Q[h0 + h].ids; p.q_scales[h] = (const uint8_t *)Q[h0 + h].scales;
        }
        for (int64_t g = 0; g < ng; g++) {
            p.k_codes[g] = (const uint8_t *)K[g0 + g].codes; p.k_ids[g] = (const uint8_t *)K[g0 + g].ids; p.k_scales[g] = (const uint8_t *)K[g0 + g].scales;
            p.v_codes[g] = (const uint8_t *)V[g0 + g].codes; p.v_ids[g] = (const uint8_t *)V[g0 + g].ids; p.v_scales[g] = (const uint8_t *)V[g0 + g].scales;
        }
        p.sq = sq; p.sk = sk; p.head0 = (int)h0; p.group = (int)group; p.scale = scale;
        p.O = O; p.ldo = ldo; p.stride_o = stride_o; p.out_bf16 = odtype == BD_BF16 ? 1 : 0;
        if (dump) {
            p.dump_S = dump->S; p.dump_P = dump->P; p.dump_codes = dump->codes; p.dump_ids = dump->ids; p.dump_scales = dump->scales;
        }
        dim3 grid((unsigned)((sq + attn::kQTile - 1) / attn::kQTile), (unsigned)nh);
        cudaStream_t st = (cudaStream_t)stream;
        if (pre) {
            p.k_exp = k_exp; p.v_exp = v_exp; p.exp_stride = (int64_t)exp_bytes;
            const dim3 egrid(grid_for(sk * (hd / kBlock), 256), (unsigned)ng, 2);
            if (hd == 128) attn::expand_kv_kernel<128><<<egrid, 256, 0, st>>>(p, k_exp, v_exp);
            else attn::expand_kv_kernel<64><<<egrid, 256, 0, st>>>(p, k_exp, v_exp);
            kernels++;
            if (hd == 128) attn::attention_kernel<128, true><<<grid, attn::kThreads, attn::Layout<128>::total, st>>>(p);
            else attn::attention_kernel<64, true><<<grid, attn::kThreads, attn::Layout<64>::total, st>>>(p);
        } else {
            if (hd == 128) attn::attention_kernel<128, false><<<grid, attn::kThreads, attn::Layout<128>::total, st>>>(p);
            else attn::attention_kernel<64, false><<<grid, attn::kThreads, attn::Layout<64>::total, st>>>(p);
        }
        kernels++;
    }
    return launch_result(kernels);
}

bd_status bd_export_canonical(const bd_qtensor *q, uint8_t *codes, uint8_t *ids, uint8_t *scales, void *stream) {
    bd_status s = check_qtensor(q);
    if (s) return s;
    if (!codes || !ids || !scales) return BD_ERR_INVALID_ARG;
    if (!aligned16(codes)) return BD_ERR_ALIGN;
    const int nb = (int)(q->K / kBlock);
    export_canonical_kernel<<<grid_for(q->rows * nb, 256), 256, 0, (cudaStream_t)stream>>>(view_of(q), codes, ids,
                                                                                          scales, nb);
    return launch_result();
}

bd_status bd_import_canonical(const uint8_t *codes, const uint8_t *ids, const uint8_t *scales, bd_qtensor *q,
                              void *stream) {
    bd_status s = check_qtensor(q);
    if (s) return s;
    if (!codes || !ids || !scales) return BD_ERR_INVALID_ARG;
    if (!aligned16(codes)) return BD_ERR_ALIGN;
    const int nb = (int)(q->K / kBlock), nb_pad = (int)k_groups(q->K) * kBlocksPerAtom;
    const int64_t rows_pad = row_tiles(q->rows) * kRowTile;
    import_canonical_kernel<<<grid_for(rows_pad * nb_pad, 256), 256, 0, (cudaStream_t)stream>>>(
        codes, ids, scales, view_of(q), rows_pad, nb, nb_pad);
    return launch_result();
}

bd_status bd_dequantize(const bd_qtensor *q, float *out, int64_t ld, void *stream) {
    bd_status s = check_qtensor(q);
    if (s) return s;
    if (!out) return BD_ERR_INVALID_ARG;
    if (ld < q->K) return BD_ERR_SHAPE;
    const int nb = (int)(q->K / kBlock);
    dequantize_kernel<<<grid_for(q->rows * nb, 256), 256, 0, (cudaStream_t)stream>>>(view_of(q), out, ld, nb);
    return launch_result();
}

bd_status bd_get_formatbook(uint8_t out[16][8]) {
    if (!out) return BD_ERR_INVALID_ARG;
    for (int d = 0; d < 16; d++)
        for (int i = 0; i < 8; i++) out[d][i] = g_book.v[d][i];
    return BD_OK;
}

bd_status bd_set_formatbook(const uint8_t in[16][8]) {
    Formatbook b = kBook;                                        // NULL restores the built-in table
    if (in)
        for (int d = 0; d < 16; d++)
            for (int i = 0; i < 8; i++) b.v[d][i] = in[d][i];
    if (!formatbook_ok(b)) return BD_ERR_INVALID_ARG;
    // the tables live in constant memory of the current device: nothing of the library may be in flight
    bd_status s = cuda_result(cudaDeviceSynchronize());
    if (s) return s;
    const DeviceTables t = make_tables(b);
    s = cuda_result(cudaMemcpyToSymbol(c_tables, &t, sizeof(t)));
    if (s) return s;
    g_book = b;
    return BD_OK;
}

bd_status bd_poll_status(void *stream) {
    bd_status s = cuda_result(cudaStreamSynchronize((cudaStream_t)stream));
    if (s) return s;
    uint32_t word = 0, zero = 0;
    s = cuda_result(cudaMemcpyFromSymbol(&word, g_status_word, sizeof(word)));
    if (s) return s;
    if (word) {
        s = cuda_result(cudaMemcpyToSymbol(g_status_word, &zero, sizeof(zero)));
        if (s) return s;
    }
    if (word & kStatusTimeout) return BD_ERR_TIMEOUT;
    if (word & kStatusNonfinite) return BD_ERR_NONFINITE;
    return BD_OK;
}

bd_status bd_set_gemm_impl(bd_gemm_impl impl) {
    if (impl != BD_GEMM_AUTO && impl != BD_GEMM_SIMT && impl != BD_GEMM_TCGEN05 && impl != BD_GEMM_WARP) return BD_ERR_INVALID_ARG;
    g_gemm_impl = impl;
    return BD_OK;
}

uint64_t bd_launch_count(void) { return g_launches; }

int bd_last_cuda_error(void) { return g_last_cuda_error; }

const char *bd_status_string(bd_status s) {
    switch (s) {
        case BD_OK: return "ok";
        case BD_ERR_INVALID_ARG: return "invalid argument";
        case BD_ERR_SHAPE: return "shape error (K must be a multiple of 32; operand shapes must agree)";
        case BD_ERR_ALIGN: return "pointer or leading dimension not 16-byte aligned";
        case BD_ERR_UNSUPPORTED: return "unsupported combination";
        case BD_ERR_CUDA: return "CUDA error (see bd_last_cuda_error)";
        case BD_ERR_NONFINITE: return "non-finite input met by a quantizer";
        case BD_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case BD_ERR_WORKSPACE: return "workspace missing or too small";
        case BD_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the built-in no-allocation buffer holds";
    }
    return "unknown status";
}

bd_status bd_debug_fault(uint32_t poll_limit, int skip_first_code_stage) {
    bd_status s = cuda_result(cudaDeviceSynchronize());
    if (s) return s;
    const uint32_t skip = skip_first_code_stage ? 1u : 0u;
    s = cuda_result(cudaMemcpyToSymbol(g_debug_spin_limit, &poll_limit, sizeof(poll_limit)));
    if (s) return s;
    return cuda_result(cudaMemcpyToSymbol(g_debug_skip_first_code_stage, &skip, sizeof(skip)));
}

int bd_version(void) { return 100; }

}  // extern "C"
