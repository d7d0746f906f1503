"""BlockDialect W4A4 quantized linear layer for B200: Python binding of libblockdialect.

The binding marshals arguments only; every step runs in the CUDA library.
Importing the package does not load the library; the first call does, and it
raises if the shared object has not been built (there is no fallback path).
"""
from .binding import (  # noqa: F401
    AXIS_CONTIG, AXIS_STRIDED, BF16, F16, F32, GEMM_AUTO, GEMM_SIMT, GEMM_TCGEN05, GEMM_WARP, SELECT_MSE,
    SELECT_TWO_STAGE, BdError, KVCache, QTensor, attention, attention_workspace_size, build, debug_fault, dequantize, export_canonical, gemm, gemm_batched,
    gemm_batched_workspace_size, gemm_requant, gemm_requant_workspace_size, gemm_workspace_size, get_formatbook, kvcache_append_batched, kvcache_attention, kvcache_pv_batched, kvcache_scores_batched, import_canonical, launch_count, library_path, linear, linear_noalloc, linear_requant, linear_requant_workspace_size, linear_workspace_size,
    export_canonical_bs, linear_bs, linear_bs_workspace_size, load, physical_k, poll_status, quantize_bs, quantize_act, quantize_weights, set_formatbook, set_gemm_impl, version,
)
