"""Pins of the attention oracle: properties the chain must have whatever its implementation."""
from fractions import Fraction

import numpy as np

import oracle
from oracle import attention as oa
from paper_2501_01144_b200 import inputs


def _case(sq, sk, d, seed):
    rng = np.random.default_rng(seed)
    q = inputs.to_bf16_bits(rng.standard_normal((sq, d)).astype(np.float32))
    k = inputs.to_bf16_bits(rng.standard_normal((sk, d)).astype(np.float32))
    v = inputs.to_bf16_bits(rng.standard_normal((sk, d)).astype(np.float32))
    return (oracle.quantize(q, dtype=oracle.BF16), oracle.quantize(k, dtype=oracle.BF16),
            oracle.quantize(np.ascontiguousarray(v.T), dtype=oracle.BF16))


def test_softmax_rows_are_distributions_and_shift_invariant():
    rng = np.random.default_rng(1)
    S = rng.standard_normal((5, 64)) * 7
    P = oa.softmax_rows(S)
    assert np.allclose(P.sum(-1), 1.0, rtol=0, atol=1e-15) and (P >= 0).all()
    assert np.allclose(oa.softmax_rows(S + 123.25), P, rtol=1e-12, atol=0)      # softmax ignores a common shift
    assert (P.argmax(-1) == S.argmax(-1)).all()
    # against the defining formula in rationals of floats (tiny row)
    row = [Fraction(float(np.exp(v - S[0].max()))) for v in S[0, :8]]
    ref = [float(r / sum(row)) for r in row]
    assert np.allclose(oa.softmax_rows(S[:1, :8])[0], ref, rtol=1e-14, atol=0)


def test_equal_scores_give_uniform_probabilities_and_the_mean_of_v():
    qz, kq, vq = _case(4, 64, 32, 2)
    qz = tuple(np.zeros_like(t) for t in qz)                         # all-zero queries: every score is 0
    O, S, P = oa.attention(qz, kq, vq, 0.5)
    assert not S.any() and np.array_equal(P, np.full((4, 64), np.float32(1 / 64)))
    # 1/64 is a power of two: its quantisation is exact, so O is the plain mean of the dequantised values
    assert np.allclose(O, oracle.dequantize(*vq).mean(axis=1)[None, :].repeat(4, 0), rtol=1e-13, atol=0)


def test_a_dominant_key_selects_its_value_row():
    q, k, v = _case(2, 32, 32, 3)
    S, _ = oa.scores(q, k, 1.0)
    S[:, 5] += 200.0                                                 # one key far ahead: P is one-hot up to fp32
    P = oa.softmax_rows(S).astype(np.float32)
    assert np.array_equal(P[:, 5], np.ones(2, np.float32)) and not np.delete(P, 5, axis=1).any()
    O, T, pq = oa.pv(P, v)
    assert np.array_equal(O, oracle.dequantize(*v)[:, 5][None, :].repeat(2, 0))


def test_scale_multiplies_the_scores_and_tolerance_base():
    q, k, _ = _case(3, 96, 64, 4)
    S1, T1 = oa.scores(q, k, 1.0)
    S2, T2 = oa.scores(q, k, 0.125)
    assert np.array_equal(S2, S1 * 0.125) and np.array_equal(T2, T1 * 0.125)
