// Tensor-core GEMM (tcgen05, block-scaled E4M3 MMA with TMEM accumulators): interface.
#pragma once
#include "bd_common.cuh"

namespace bd {

inline bool tc_supported(int64_t, int64_t, int64_t) { return false; }
inline size_t tc_operand_bytes(int64_t rows, int64_t K) { return ((size_t)rows * (size_t)K + 255) & ~(size_t)255; }
inline size_t tc_gemm_workspace(int64_t M, int64_t N, int64_t K) { return tc_operand_bytes(M, K) + tc_operand_bytes(N, K); }
inline cudaError_t tc_gemm(const uint8_t *, const uint8_t *, int64_t, const uint8_t *, const uint8_t *, int64_t, int64_t,
                           void *, bool, int64_t, cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace bd
