"""CPU oracle of the KV-cache structure (test infrastructure, like the rest of this package).

The paper's appendix "Quantization Dimension" (Fig. 9b) lays the cache of one KV head out like this:
  * keys are quantised sub-token-wise (blocks of 32 along head_dim), so a new key vector is quantised once,
    before its product, and appended;
  * values are quantised sub-channel-wise (blocks along the token axis, their multiplication dimension in
    score x V), which a single new token cannot extend.  Values are therefore stored in 4-bit chunks of
    `block` tokens, and only the most recent chunk, of N mod block tokens, is kept in high precision; when it
    reaches `block` tokens it is quantised once and stored in 4-bit form.  Nothing is ever requantised.
Written with the package's plain quantizer, dequantizer and fp64 product; lists and numpy only.
"""
import numpy as np

from . import BF16, F16, F32, dequantize, gemm, quantize

_NP_OF = {F32: np.float32, BF16: np.uint16, F16: np.uint16}


def _to_f64(rows, dtype):
    """Exact values of source rows given as fp32 or as 16-bit patterns."""
    rows = np.asarray(rows)
    if dtype == F32:
        return rows.astype(np.float64)
    if dtype == BF16:
        return (rows.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    return rows.view(np.float16).astype(np.float64)


class KVCache:
    def __init__(self, head_dim, dtype=BF16, block=32):
        self.d, self.dtype, self.block = head_dim, dtype, block
        self.key_codes, self.key_ids, self.key_scales = [], [], []     # one entry per token
        self.chunks = []                                                # per full chunk: canonical (codes, ids, scales) of [d, block]
        self.recent = []                                                # source rows of the newest N mod block tokens

    @property
    def length(self):
        return len(self.key_codes)

    def append(self, k_rows, v_rows):
        """k_rows, v_rows: [t, head_dim] in the cache's source type (fp32, or uint16 patterns)."""
        k_rows, v_rows = np.asarray(k_rows), np.asarray(v_rows)
        for t in range(k_rows.shape[0]):
            c, i, s = quantize(k_rows[t:t + 1], dtype=self.dtype)       # the key vector: blocks of 32 along head_dim
            self.key_codes.append(c[0]); self.key_ids.append(i[0]); self.key_scales.append(s[0])
            self.recent.append(v_rows[t].copy())
            if len(self.recent) == self.block:                          # the newest chunk is full: 4-bit form, once
                chunk = np.ascontiguousarray(np.stack(self.recent).T)   # [d, block]: a block = `block` tokens of a channel
                self.chunks.append(quantize(chunk, dtype=self.dtype, block=self.block))
                self.recent = []

    def keys(self):
        """Canonical (codes, ids, scales) of the key operand [length, head_dim]."""
        return np.stack(self.key_codes), np.stack(self.key_ids), np.stack(self.key_scales)

    def values_quantised(self):
        """Canonical (codes, ids, scales) of the stored value operand [head_dim, n_q], n_q = tokens in full chunks."""
        if not self.chunks:
            return (np.zeros((self.d, 0), np.uint8),) * 3
        return tuple(np.concatenate([ch[j] for ch in self.chunks], axis=1) for j in range(3))

    def values_recent(self):
        """The high-precision rows [N mod block, head_dim] as exact fp64 values."""
        if not self.recent:
            return np.zeros((0, self.d), np.float64)
        return _to_f64(np.stack(self.recent), self.dtype)

    def scores(self, q_canonical):
        """S = dq(Q) dq(K)^T for a quantised query operand [q, head_dim]; returns (S, T)."""
        return gemm(dequantize(*q_canonical), dequantize(*self.keys()))

    def attention(self, q_canonical, scale):
        """One decode step (Sec. 4.1 scope "all", Sec. 3.3): S = dq(Q) dq(K)^T, P = softmax(scale * S) in fp64 stored as
        fp32, O = P V as in pv().  Returns (O, T, P32)."""
        S, _ = self.scores(q_canonical)
        z = np.exp(scale * S - (scale * S).max(axis=-1, keepdims=True))
        P32 = (z / z.sum(axis=-1, keepdims=True)).astype(np.float32)
        O, T = self.pv(P32)
        return O, T, P32

    def pv(self, P):
        """O = P V with P [q, length] fp32: the part over full chunks is quantised along the keys (two-stage rule)
        and multiplied with the 4-bit values; the part over the recent tokens stays in high precision (fp64 here).
        Returns (O, T) with T = sum |p| |v| over both parts."""
        P = np.ascontiguousarray(P, np.float32)
        nq = len(self.chunks) * self.block
        O = np.zeros((P.shape[0], self.d), np.float64)
        T = np.zeros_like(O)
        if nq:
            pq = quantize(np.ascontiguousarray(P[:, :nq]), block=self.block)
            o, t = gemm(dequantize(*pq), dequantize(*self.values_quantised()))
            O += o
            T += t
        if self.recent:
            pr, vr = P[:, nq:].astype(np.float64), self.values_recent()
            O += pr @ vr
            T += np.abs(pr) @ np.abs(vr)
        return O, T
