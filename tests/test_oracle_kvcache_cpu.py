"""Pins of the KV-cache oracle (appendix "Quantization Dimension", Fig. 9b): what the structure must satisfy
whatever the implementation, checked with exact rationals and with the (separately pinned) block quantizer."""
from fractions import Fraction

import numpy as np

import oracle
from oracle.kvcache import KVCache
from paper_2501_01144_b200 import inputs

FB = oracle.formatbook()


def _dq_entry(code_nibble, dialect, scale):
    v = Fraction(int(FB[dialect][code_nibble & 7]), 2) * Fraction(2) ** (int(scale) - 127)
    return -v if code_nibble & 8 else v


def _data(n, d, seed):
    rng = np.random.default_rng(seed)
    k = inputs.to_bf16_bits(rng.standard_normal((n, d)).astype(np.float32))
    v = inputs.to_bf16_bits((rng.standard_normal((n, d)) * np.exp2(rng.integers(-3, 4, (1, d)))).astype(np.float32))
    return k, v


def test_chunks_of_block_tokens_and_a_high_precision_remainder():
    k, v = _data(77, 64, 1)
    c = KVCache(64)
    c.append(k, v)
    assert c.length == 77 and len(c.chunks) == 77 // 32 and len(c.recent) == 77 % 32      # N mod block_size stays in high precision
    # the stored values are the sub-channel-wise quantisation of the full chunks: blocks of 32 TOKENS per channel
    ref = oracle.quantize(np.ascontiguousarray(v[:64].T), dtype=oracle.BF16)
    got = c.values_quantised()
    assert all(np.array_equal(g, r) for g, r in zip(got, ref))
    # keys: one sub-token-wise quantisation per token
    assert all(np.array_equal(g, r) for g, r in zip(c.keys(), oracle.quantize(k, dtype=oracle.BF16)))
    # the remainder is the source, bit for bit
    assert np.array_equal(c.values_recent(), inputs.bf16_bits_to_f32(v[64:]).astype(np.float64))


def test_token_by_token_equals_bulk_append_and_nothing_is_requantised():
    k, v = _data(70, 32, 2)
    bulk, step = KVCache(32), KVCache(32)
    bulk.append(k, v)
    snapshots = []
    for t in range(70):
        step.append(k[t:t + 1], v[t:t + 1])
        snapshots.append([ch[0].copy() for ch in step.chunks])
    assert all(np.array_equal(a, b) for a, b in zip(bulk.values_quantised(), step.values_quantised()))
    assert np.array_equal(bulk.values_recent(), step.values_recent())
    # a chunk, once stored, never changes when later tokens arrive
    assert all(np.array_equal(snapshots[40][0], s[0]) for s in snapshots[40:])


def test_pv_against_rational_arithmetic():
    k, v = _data(40, 32, 3)            # one full chunk + 8 recent tokens
    c = KVCache(32)
    c.append(k, v)
    rng = np.random.default_rng(4)
    P = rng.dirichlet(np.full(40, 0.3), 3).astype(np.float32)
    O, T = c.pv(P)
    pq = oracle.quantize(np.ascontiguousarray(P[:, :32]))
    vc, vi, vs = c.values_quantised()
    vr = inputs.bf16_bits_to_f32(v[32:])
    for q in range(3):
        for ch in (0, 7, 31):
            exact = Fraction(0)
            for n in range(32):
                pn = (int(pq[0][q, n // 2]) >> (4 * (n % 2))) & 15
                vn = (int(vc[ch, n // 2]) >> (4 * (n % 2))) & 15
                exact += _dq_entry(pn, pq[1][q, 0], pq[2][q, 0]) * _dq_entry(vn, vi[ch, 0], vs[ch, 0])
            for n in range(8):          # the recent tokens: full-precision P times the stored source values
                exact += Fraction(float(P[q, 32 + n])) * Fraction(float(vr[n, ch]))
            assert abs(Fraction(float(O[q, ch])) - exact) <= Fraction(float(T[q, ch])) * Fraction(1, 10 ** 13)


def test_fewer_tokens_than_a_block_is_the_exact_product():
    k, v = _data(19, 32, 5)
    c = KVCache(32)
    c.append(k, v)
    P = np.random.default_rng(6).random((2, 19)).astype(np.float32)
    O, _ = c.pv(P)
    assert np.allclose(O, P.astype(np.float64) @ inputs.bf16_bits_to_f32(v).astype(np.float64), rtol=1e-14, atol=0)
    assert len(c.chunks) == 0


def test_attention_special_cases():
    # one cached token: its probability is 1 and it is still in high precision, so the result is that value row itself
    d = 64
    rng = np.random.default_rng(3)
    k, v = rng.standard_normal((40, d)).astype(np.float32), rng.standard_normal((40, d)).astype(np.float32)
    q = oracle.quantize(rng.standard_normal((3, d)).astype(np.float32))
    c = KVCache(d, dtype=oracle.F32)
    c.append(k[:1], v[:1])
    O, _, P = c.attention(q, 0.3)
    assert np.array_equal(P, np.ones((3, 1), np.float32)) and np.array_equal(O, np.repeat(v[:1].astype(np.float64), 3, 0))
    # a query that is a large multiple of one key: the softmax is one-hot up to rounding, the result is that token's
    # stored value (a full chunk, so the dequantised 4-bit row) and the rows of P are distributions
    c = KVCache(d, dtype=oracle.F32)
    c.append(k[:32], v[:32])
    j = 7
    q = oracle.quantize((64.0 * k[j:j + 1]).astype(np.float32))
    O, _, P = c.attention(q, 1.0)
    assert P.argmax() == j and P[0, j] > 1.0 - 1e-6 and abs(P.sum() - 1.0) < 1e-6
    vq = oracle.dequantize(*c.values_quantised())                 # [d, 32]
    assert np.allclose(O[0], vq[:, j], rtol=0, atol=1e-5 * np.abs(vq).max())
    # scale 0: uniform probabilities over 40 tokens = the plain pv of a constant row
    c.append(k[32:], v[32:])
    O, _, P = c.attention(q, 0.0)
    assert np.array_equal(P, np.full((1, 40), np.float32(1.0 / 40)))
    O2, _ = c.pv(np.full((1, 40), 1.0 / 40, np.float32))
    assert np.array_equal(O, O2)
