"""Fused full-path attention against its oracle.  The kernel never writes S or P on its own; for checking it can dump
them, and the comparison then goes link by link: the scores against the oracle's fp64 product, the probabilities
against the fp64 softmax of the library's own scores, the codes, ids and scales of the quantised probabilities bit for
bit against the oracle's two-stage rule on the library's own fp32 probabilities, and the result against the oracle's
product of those codes with the value operand."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from oracle import attention as oa
from paper_2501_01144_b200 import inputs
from util import gemm_tolerance_ok, oracle_quantize, to_device

pytestmark = pytest.mark.gpu


def _operands(Q, K, V):
    Qs = [bd.quantize_act(to_device(q, torch.bfloat16)) for q in Q]
    Ks = [bd.quantize_act(to_device(k, torch.bfloat16)) for k in K]
    Vs = [bd.quantize_act(to_device(v, torch.bfloat16), axis=bd.AXIS_STRIDED) for v in V]
    return Qs, Ks, Vs


def _check_head(h, group, Q, K, V, scale, O, dump, rows):
    qq = oracle_quantize(Q[h][rows], torch.bfloat16)
    kq = oracle_quantize(K[h // group], torch.bfloat16)
    vq = oracle_quantize(np.ascontiguousarray(V[h // group].T), torch.bfloat16)
    # scores
    S_ref, T = oa.scores(qq, kq, scale)
    S = dump["S"][h].cpu().numpy()[rows]
    ok, ratio = gemm_tolerance_ok(S, S_ref, T)
    assert ok, f"head {h} scores: max err / bound = {ratio}"
    # probabilities: the fp64 softmax of the library's own scores (fp32 exponentials and sums on the device)
    P = dump["P"][h].cpu().numpy()[rows]
    P_ref = oa.softmax_rows(S)
    assert np.abs(P - P_ref).max() <= 3e-6 * P_ref.max(-1).max() and np.allclose(P, P_ref, rtol=2e-5, atol=1e-30), f"head {h} probabilities"
    assert np.allclose(P.sum(-1, dtype=np.float64), 1.0, atol=1e-5)
    # the quantised probabilities: bit for bit the two-stage rule on the library's own fp32 probabilities
    pq_ref = oracle.quantize(P)
    for name, j in (("scales", 2), ("ids", 1), ("codes", 0)):
        got = dump[name][h].cpu().numpy()[rows]
        bad = np.argwhere(got != pq_ref[j])
        assert bad.size == 0, f"head {h} quantised P: {len(bad)} {name} mismatches, first at {bad[0]}"
    # result: the oracle's product of those operands
    O_ref, To = oracle.gemm(oracle.dequantize(*pq_ref), oracle.dequantize(*vq))
    ok, ratio = gemm_tolerance_ok(O[h].float().cpu().numpy()[rows], O_ref, To)
    assert ok, f"head {h} result: max err / bound = {ratio}"


@pytest.mark.parametrize("heads,kv,sq,sk,d", [(2, 1, 64, 64, 128), (4, 2, 130, 96, 128), (3, 3, 200, 352, 64), (8, 2, 256, 1024, 128)])
def test_fused_attention_link_by_link(heads, kv, sq, sk, d):
    rng = np.random.default_rng(heads + sq + sk)
    Q = inputs.to_bf16_bits(rng.standard_normal((heads, sq, d)).astype(np.float32))
    K = inputs.to_bf16_bits(rng.standard_normal((kv, sk, d)).astype(np.float32))
    V = inputs.to_bf16_bits((rng.standard_normal((kv, sk, d)) * np.exp2(rng.integers(-2, 3, (kv, 1, d)))).astype(np.float32))
    K[:, :, 3] = inputs.to_bf16_bits((inputs.bf16_bits_to_f32(K[:, :, 3]) * 6).astype(np.float32))      # an outlier channel
    Qs, Ks, Vs = _operands(Q, K, V)
    scale = d ** -0.5
    O, dump = bd.attention(Qs, Ks, Vs, group=heads // kv, scale=scale, dtype=torch.float32, dump=True)
    rows = np.arange(sq)
    for h in range(heads):
        _check_head(h, heads // kv, Q, K, V, scale, O, dump, rows)
    # without the dump and with bf16 output: the same result, rounded
    O16 = bd.attention(Qs, Ks, Vs, group=heads // kv, scale=scale, dtype=torch.bfloat16)
    assert torch.equal(O16, O.to(torch.bfloat16))
    # without the scratch for the expanded K and V the kernel expands its key tiles itself: the same bits
    O_plain, dump_plain = bd.attention(Qs, Ks, Vs, group=heads // kv, scale=scale, dtype=torch.float32, dump=True, workspace=None)
    assert torch.equal(O_plain, O) and all(torch.equal(dump_plain[k], dump[k]) for k in dump)
    # a caller's scratch with guard bands
    need = bd.attention_workspace_size(heads, heads // kv, sk, d)
    raw = torch.full((need + 8192,), 0xA5, dtype=torch.uint8, device="cuda")
    O_ws = bd.attention(Qs, Ks, Vs, group=heads // kv, scale=scale, dtype=torch.float32, workspace=raw[4096:4096 + need])
    assert torch.equal(O_ws, O) and bool((raw[:4096] == 0xA5).all()) and bool((raw[4096 + need:] == 0xA5).all())
    bd.poll_status()


def test_fused_attention_matches_the_materialised_route():
    """The unfused chain through bd_gemm_batched, a host softmax and bd_linear quantises (nearly) the same
    probabilities, so on smooth score distributions the two routes agree up to a few codes that sit within fp32
    rounding of a boundary.  (Nearly one-hot rows are left out here on purpose: a top probability of 1.0 or of
    1 - 2^-24 falls on the two sides of a power of two and quantises to 1.0 or to 0.9375.)"""
    heads, kv, s, d = 4, 1, 256, 128
    rng = np.random.default_rng(5)
    Q = inputs.to_bf16_bits(rng.standard_normal((heads, s, d)).astype(np.float32))
    Kt = inputs.to_bf16_bits(rng.standard_normal((kv, s, d)).astype(np.float32))
    V = inputs.to_bf16_bits(rng.standard_normal((kv, s, d)).astype(np.float32))
    Qs, Ks, Vs = _operands(Q, Kt, V)
    O = bd.attention(Qs, Ks, Vs, group=heads // kv, dtype=torch.float32)
    S = bd.gemm_batched(Qs, Ks, b_group=heads // kv)
    P = torch.softmax(S.double() * d ** -0.5, -1).float()
    O2 = torch.stack([bd.linear(P[h].contiguous(), Vs[0], dtype=torch.float32) for h in range(heads)])
    diff = (O - O2).abs()
    assert float((diff > 1e-2 * float(O2.abs().max())).float().mean()) <= 2e-3
    assert float(diff.mean()) <= 1e-3 * float(O2.abs().mean())
    bd.poll_status()
