"""CPU oracle of full-path attention (test infrastructure): both matrix products of attention on DialectFP4
operands with the softmax between them in high precision (Sec. 4.1, scope "all": QK^T and score x V are quantised
too; Sec. 3.3: softmax and the other non-linear operations stay in high precision; appendix "Quantization
Dimension": Q and K are cut into blocks along head_dim, the scores along the keys, V along the tokens).

The chain, one head at a time, from the package's plain pieces:
    S = dq(Q) dq(K)^T * scale            fp64 product of the dequantised operands
    P = softmax(S) row by row            fp64, then stored as fp32 (the online quantizer's source type)
    O = dq(quantise(P)) dq(V)^T          P quantised along the keys with the two-stage rule
"""
import numpy as np

from . import dequantize, gemm, quantize


def scores(q_canonical, k_canonical, scale):
    """(S, T): S = dq(Q) dq(K)^T * scale in fp64 and the tolerance base T = scale * sum |q||k|."""
    S, T = gemm(dequantize(*q_canonical), dequantize(*k_canonical))
    return S * scale, T * abs(scale)


def softmax_rows(S):
    """Row-wise softmax in fp64: exp(s - max) / sum."""
    S = np.asarray(S, np.float64)
    z = np.exp(S - S.max(axis=-1, keepdims=True))
    return z / z.sum(axis=-1, keepdims=True)


def pv(P32, v_canonical, block=32):
    """(O, T, Pq): fp32 probabilities [q, keys] quantised along the keys, times the value operand [d, keys]."""
    pq = quantize(np.ascontiguousarray(P32, np.float32), block=block)
    O, T = gemm(dequantize(*pq), dequantize(*v_canonical))
    return O, T, pq


def attention(q_canonical, k_canonical, v_canonical, scale):
    """The whole chain; returns (O, S, P32)."""
    S, _ = scores(q_canonical, k_canonical, scale)
    P32 = softmax_rows(S).astype(np.float32)
    O, _, _ = pv(P32, v_canonical)
    return O, S, P32
