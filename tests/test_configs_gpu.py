"""Parity at the benchmark's full sizes (the launch configuration bench.py times), on
sampled outputs the oracle can compute one by one: whole rows, whole columns and tile
boundaries of the LLaMA-shaped linear layers, the decode-to-prefill M sweep, and the
Mistral-shaped attention products with both operands quantised online."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import assert_bit_exact, gemm_tolerance_ok, oracle_quantize, to_device

pytestmark = pytest.mark.gpu


def _check_rows_cols(Y, xb, wb, rows, cols, what):
    """Y [M,N] from the library; xb/wb bf16 bit patterns.  Compares Y[rows, :] and Y[:, cols]."""
    qa_all = None
    qb = oracle.quantize(wb, dtype=oracle.BF16)
    wdq = oracle.dequantize(*qb)
    qa = oracle.quantize(xb[rows], dtype=oracle.BF16)
    Yref, T = oracle.gemm(oracle.dequantize(*qa), wdq)
    ok, ratio = gemm_tolerance_ok(Y[rows], Yref, T)
    assert ok, f"{what} rows: max err / bound = {ratio}"
    if len(cols):
        qa_all = oracle.quantize(xb, dtype=oracle.BF16)
        Yref, T = oracle.gemm(oracle.dequantize(*qa_all), wdq[cols])
        ok, ratio = gemm_tolerance_ok(Y[:, cols], Yref, T)
        assert ok, f"{what} cols: max err / bound = {ratio}"


@pytest.mark.parametrize("K,N", [(4096, 4096), (4096, 1024), (4096, 14336), (14336, 4096)])
def test_llama3_linear_layers_m2048(K, N):
    M = 2048
    xb = inputs.act_student_t(M, K, seed=2)
    wb = inputs.weights_normal(N, K, seed=2)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    Y = bd.linear(to_device(xb, torch.bfloat16), Wq, dtype=torch.float32).cpu().numpy()
    rng = np.random.default_rng(K + N)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 1], rng.choice(M, 4, replace=False)]))
    cols = np.unique(np.concatenate([[0, 255, 256, N - 1], rng.choice(N, 4, replace=False)]))
    _check_rows_cols(Y, xb, wb, rows, cols, f"K={K} N={N}")
    # bf16 output (what the benchmark times) is the rounded fp32 result
    Y16 = bd.linear(to_device(xb, torch.bfloat16), Wq, dtype=torch.bfloat16)
    assert torch.equal(Y16.cpu(), torch.from_numpy(Y).to(torch.bfloat16))
    # every element against the library's CUDA-core product (exact block sums, fp64 across blocks), which
    # shares no code with the tensor-core kernel after the quantizer
    xd = to_device(xb, torch.bfloat16)
    bd.set_gemm_impl(bd.GEMM_SIMT)
    Yexact = bd.linear(xd, Wq, dtype=torch.float32)
    bd.set_gemm_impl(bd.GEMM_AUTO)
    bound = 2e-6 * (bd.dequantize(bd.quantize_act(xd)).abs() @ bd.dequantize(Wq).abs().T) + 2.0 ** -120
    assert bool(((torch.from_numpy(Y).cuda() - Yexact).abs() <= bound).all())
    bd.poll_status()


def test_llama3_weights_exact_mse_rule_on_kv_shape():
    wb = inputs.weights_normal(1024, 4096, seed=2)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_MSE)
    assert_bit_exact(Wq, oracle_quantize(wb, torch.bfloat16, oracle.SELECT_MSE), "kv weights, MSE rule")


@pytest.mark.parametrize("K,N", [(4096, 11008), (11008, 4096)])
@pytest.mark.parametrize("M", [1, 16, 128, 1024, 8192])
def test_llama2_mlp_m_sweep(K, N, M):
    xb = inputs.act_post_silu(M, K, seed=3)
    wb = inputs.weights_normal(N, K, seed=3)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    xd = to_device(xb, torch.bfloat16)
    Yd = bd.linear(xd, Wq, dtype=torch.float32)
    Y = Yd.cpu().numpy()
    rng = np.random.default_rng(M)
    # rows and columns at the tile boundaries of the tensor-core kernel (256 tokens x 256 weight rows, items of
    # 128 tokens) plus random ones: eight or more whole rows and eight or more whole columns at every M
    edge_rows = [r for r in (0, 127, 128, 255, 256, M - 129, M - 128, M - 1) if 0 <= r < M]
    rows = np.unique(np.concatenate([edge_rows, rng.choice(M, min(M, 8), replace=False)]))
    cols = np.unique(np.concatenate([[0, 127, 128, 255, 256, N - 257, N - 256, N - 1], rng.choice(N, 8, replace=False)]))
    _check_rows_cols(Y, xb, wb, rows, cols, f"M={M} K={K} N={N}")
    if M >= 1024:
        # 4096 further entries: a random 64 x 64 sub-grid of the result
        r64, c64 = rng.choice(M, 64, replace=False), rng.choice(N, 64, replace=False)
        qa = oracle.quantize(xb[r64], dtype=oracle.BF16)
        qb = oracle.quantize(wb[c64], dtype=oracle.BF16)
        Yref, T = oracle.gemm(oracle.dequantize(*qa), oracle.dequantize(*qb))
        ok, ratio = gemm_tolerance_ok(Y[np.ix_(r64, c64)], Yref, T)
        assert ok, f"M={M} K={K} N={N} sub-grid: max err / bound = {ratio}"
    # every element against the library's CUDA-core product (exact block sums, fp64 across blocks), which shares
    # no code with the tensor-core kernel after the quantizer
    bd.set_gemm_impl(bd.GEMM_SIMT)
    Yexact = bd.linear(xd, Wq, dtype=torch.float32)
    bd.set_gemm_impl(bd.GEMM_AUTO)
    wabs = bd.dequantize(Wq).abs()
    xabs = bd.dequantize(bd.quantize_act(xd)).abs()
    for r0 in range(0, M, 2048):                              # the bound in slabs of 2048 tokens
        bound = 2e-6 * (xabs[r0:r0 + 2048] @ wabs.T) + 2.0 ** -120
        assert bool(((Yd[r0:r0 + 2048] - Yexact[r0:r0 + 2048]).abs() <= bound).all()), f"tokens from {r0}"
    bd.poll_status()


def test_attention_products_both_operands_online():
    heads, kv, S, d = 32, 8, 4096, 128
    n_p = 2                                                   # heads of P generated (each is 64 MiB of fp32)
    Q, Kt, P, V = inputs.attention_case(heads, kv, S, d, seed=4, p_heads=n_p)
    group = heads // kv
    # ---- QK^T: both along head_dim (K = 128), grouped-query batching over all 32 heads ----
    Aq = [bd.quantize_act(to_device(Q[h], torch.bfloat16)) for h in range(heads)]
    Bk = [bd.quantize_act(to_device(Kt[g], torch.bfloat16)) for g in range(kv)]
    for h in (0, 5, 31):
        assert_bit_exact(Aq[h], oracle_quantize(Q[h], torch.bfloat16), f"Q head {h}")
    assert_bit_exact(Bk[7], oracle_quantize(Kt[7], torch.bfloat16), "K head 7")
    out = torch.empty(4, S, S, dtype=torch.float32, device="cuda")
    check_heads = [0, 13, 30, 31]
    Ssc = bd.gemm_batched([Aq[h] for h in check_heads], [Bk[h // group] for h in check_heads], b_group=1, out=out)
    rows = np.array([0, 127, 128, 2049, S - 1])
    for i, h in enumerate(check_heads):
        qa = oracle_quantize(Q[h][rows], torch.bfloat16)
        qb = oracle_quantize(Kt[h // group], torch.bfloat16)
        Yref, T = oracle.gemm(oracle.dequantize(*qa), oracle.dequantize(*qb))
        ok, ratio = gemm_tolerance_ok(Ssc[i].cpu().numpy()[rows], Yref, T)
        assert ok, f"QK^T head {h}: max err / bound = {ratio}"
    # grouped batching: heads 0..3 share KV head 0
    out4 = bd.gemm_batched(Aq[:4], Bk[:1], b_group=4, out=torch.empty(4, S, S, dtype=torch.float32, device="cuda"))
    assert torch.equal(out4[0], Ssc[0])
    del out, out4, Ssc
    # ---- PV: P along keys (K = 4096, fp32 source), V along tokens (strided axis) ----
    Bv = [bd.quantize_act(to_device(V[g], torch.bfloat16), axis=bd.AXIS_STRIDED) for g in range(kv)]
    assert_bit_exact(Bv[0], oracle_quantize(np.ascontiguousarray(V[0].T), torch.bfloat16), "V head 0 (token axis)")
    for h in range(n_p):
        Ap = bd.quantize_act(to_device(P[h], torch.float32))
        assert_bit_exact(Ap, oracle.quantize(P[h]), f"P head {h}")
        O = bd.gemm(Ap, Bv[h // group]).cpu().numpy()
        qa = oracle.quantize(P[h][rows])
        qb = oracle_quantize(np.ascontiguousarray(V[h // group].T), torch.bfloat16)
        Yref, T = oracle.gemm(oracle.dequantize(*qa), oracle.dequantize(*qb))
        ok, ratio = gemm_tolerance_ok(O[rows], Yref, T)
        assert ok, f"PV head {h}: max err / bound = {ratio}"
    bd.poll_status()


def test_attention_fused_path_at_the_benchmark_size():
    """Config 5 through the fused kernel: 32 query heads, 8 KV heads, 4096 tokens, head_dim 128, no S or P in
    memory.  Three heads are run again with the kernel's checking dumps and compared link by link with the oracle on
    sampled rows; their results must equal the full call's bit for bit."""
    from oracle import attention as oa
    heads, kv, S, d = 32, 8, 4096, 128
    group = heads // kv
    Q, Kt, _, V = inputs.attention_case(heads, kv, S, d, seed=4, p_heads=0)
    Qs = [bd.quantize_act(to_device(Q[h], torch.bfloat16)) for h in range(heads)]
    Ks = [bd.quantize_act(to_device(Kt[g], torch.bfloat16)) for g in range(kv)]
    Vs = [bd.quantize_act(to_device(V[g], torch.bfloat16), axis=bd.AXIS_STRIDED) for g in range(kv)]
    scale = d ** -0.5
    O = bd.attention(Qs, Ks, Vs, group=group, scale=scale, dtype=torch.float32)
    rows = np.array([0, 63, 64, 1000, 2049, S - 1])
    for h in (0, 13, 31):
        Oh, dump = bd.attention([Qs[h]], [Ks[h // group]], [Vs[h // group]], group=1, scale=scale, dtype=torch.float32, dump=True)
        assert torch.equal(Oh[0], O[h]), f"head {h}: the result depends on the launch it was part of"
        qq = oracle_quantize(Q[h][rows], torch.bfloat16)
        kq = oracle_quantize(Kt[h // group], torch.bfloat16)
        vq = oracle_quantize(np.ascontiguousarray(V[h // group].T), torch.bfloat16)
        S_ref, T = oa.scores(qq, kq, scale)
        S_lib = dump["S"][0].cpu().numpy()[rows]
        ok, ratio = gemm_tolerance_ok(S_lib, S_ref, T)
        assert ok, f"head {h} scores: max err / bound = {ratio}"
        P_lib = dump["P"][0].cpu().numpy()[rows]
        P_ref = oa.softmax_rows(S_lib)
        # the scores of this case reach the thousands (outlier channels), so the fp32 exponent carries their rounding
        assert np.abs(P_lib - P_ref).max() <= 2e-3, f"head {h} probabilities"
        pq_ref = oracle.quantize(P_lib)
        for name, j in (("scales", 2), ("ids", 1), ("codes", 0)):
            assert np.array_equal(dump[name][0].cpu().numpy()[rows], pq_ref[j]), f"head {h}: {name} of the quantised probabilities"
        O_ref, To = oracle.gemm(oracle.dequantize(*pq_ref), oracle.dequantize(*vq))
        ok, ratio = gemm_tolerance_ok(O[h].cpu().numpy()[rows], O_ref, To)
        assert ok, f"head {h} result: max err / bound = {ratio}"
    bd.poll_status()
