"""The requantising epilogue (Sec. 3.3, last paragraph): a product whose result is written as the next product's
DialectFP4 operand.  The product itself is only equal to the oracle's within the tolerance, so the emitted codes,
dialect ids and scales are compared bit for bit with the oracle's two-stage quantisation of the library's own fp32
result of the same call; the chain of two layers is then compared with the oracle's product of those operands."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import assert_bit_exact, gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu

GUARD = 4096


@pytest.fixture(autouse=True)
def _reset_impl():
    yield
    bd.set_gemm_impl(bd.GEMM_AUTO)


def _guarded_qtensor(rows, K):
    q = bd.QTensor(rows, K)
    raws = {}
    for name in ("codes", "ids", "scales"):
        n = getattr(q, name).numel()
        raw = torch.full((n + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        raws[name] = (raw, n)
        setattr(q, name, raw[GUARD:GUARD + n])
    return q, raws


def _guards_intact(raws):
    return all(bool((raw[:GUARD] == 0xA5).all()) and bool((raw[GUARD + n:] == 0xA5).all()) for raw, n in raws.values())


def _layer(M, N, K, seed):
    xb = inputs.act_student_t(M, K, seed=seed)
    wb = inputs.weights_normal(N, K, seed=seed)
    return xb, wb, to_device(xb, torch.bfloat16), bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)


@pytest.mark.parametrize("K,N", [(4096, 4096), (4096, 1024), (4096, 14336), (14336, 4096)])
def test_llama3_layers_requantised_in_the_epilogue(K, N):
    M = 2048
    xb, wb, xd, Wq = _layer(M, N, K, seed=2)
    Yq, raws = _guarded_qtensor(M, N)
    before = bd.launch_count()
    bd.linear_requant(xd, Wq, out=Yq)
    assert bd.launch_count() - before == 2, "quantizer of X and the product with its requantising epilogue"
    Y32 = bd.linear(xd, Wq, dtype=torch.float32).cpu().numpy()
    assert_bit_exact(Yq, oracle.requantize(Y32), f"K={K} N={N}")
    assert _guards_intact(raws), "write outside the quantised result"
    # the same operand from the standalone quantizer on the fp32 result
    assert_bit_exact(bd.quantize_act(torch.from_numpy(Y32).cuda()), oracle.requantize(Y32), "standalone")
    bd.poll_status()


@pytest.mark.parametrize("M,N,K", [(129, 32, 32), (130, 288, 352), (300, 544, 2144), (257, 1056, 1056), (448, 512, 256),
                                   (640, 320, 160), (1280, 3840, 256), (700, 96, 512),
                                   # at most 128 tokens: the fp32 result is parked in scratch and the quantizer follows
                                   (1, 256, 8192), (16, 512, 4128), (100, 544, 224), (128, 1024, 4096)])
@pytest.mark.parametrize("impl", [bd.GEMM_AUTO, bd.GEMM_TCGEN05, bd.GEMM_SIMT])
def test_requantised_results_of_ragged_shapes(M, N, K, impl):
    rng = np.random.default_rng(M + 31 * N + 977 * K)
    xb = inputs.to_bf16_bits((rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-4, 5, (M, 1)))).astype(np.float32))
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    xd = to_device(xb, torch.bfloat16)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(impl)
    Yq, raws = _guarded_qtensor(M, N)
    ws_bytes = bd.linear_requant_workspace_size(M, N, K)
    raw_ws = torch.full((ws_bytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    bd.linear_requant(xd, Wq, out=Yq, workspace=raw_ws[GUARD:GUARD + ws_bytes])
    Y32 = bd.linear(xd, Wq, dtype=torch.float32).cpu().numpy()
    torch.cuda.synchronize()
    assert_bit_exact(Yq, oracle.requantize(Y32), f"{M}x{N}x{K} impl {impl}")
    assert _guards_intact(raws), "write outside the quantised result"
    assert bool((raw_ws[:GUARD] == 0xA5).all()) and bool((raw_ws[GUARD + ws_bytes:] == 0xA5).all()), "write outside the workspace"
    # the result against the oracle's product (fp32 route of the same call)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)),
                          oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    ok, ratio = gemm_tolerance_ok(Y32, Yref, T)
    assert ok, f"max err / bound = {ratio}"
    bd.poll_status()


@pytest.mark.parametrize("M,d0,d1,d2", [(512, 1024, 2048, 768), (2048, 4096, 4096, 1024), (100, 512, 1024, 256)])
def test_two_chained_layers_without_a_high_precision_result_between_them(M, d0, d1, d2):
    # layer 1: X [M, d0] x W1 [d1, d0] -> requantised operand [M, d1]; layer 2: that operand x W2 [d2, d1] -> fp32
    xb, w1b, xd, W1q = _layer(M, d1, d0, seed=21)
    w2b = inputs.weights_normal(d2, d1, seed=22)
    W2q = bd.quantize_weights(to_device(w2b, torch.bfloat16), bd.SELECT_TWO_STAGE)
    H = bd.linear_requant(xd, W1q)
    Y = bd.gemm(H, W2q, dtype=torch.float32).cpu().numpy()
    # the chain with the high-precision result in between gives the same bits
    H32 = bd.linear(xd, W1q, dtype=torch.float32)
    Y_two_step = bd.linear(H32, W2q, dtype=torch.float32).cpu().numpy()
    assert np.array_equal(Y, Y_two_step)
    # against the oracle: its quantisation of the library's fp32 layer-1 result, then its fp64 product
    h_ref = oracle.requantize(H32.cpu().numpy())
    assert_bit_exact(H, h_ref, "layer-1 operand")
    Yref, T = oracle.gemm(oracle.dequantize(*h_ref), oracle.dequantize(*oracle.quantize(w2b, dtype=oracle.BF16)))
    ok, ratio = gemm_tolerance_ok(Y, Yref, T)
    assert ok, f"layer 2: max err / bound = {ratio}"
    # the oracle's own chain (its fp64 layer-1 result rounded to fp32) picks the same codes except where a value
    # sits within the product tolerance of a rounding boundary
    Y1ref, _ = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)),
                           oracle.dequantize(*oracle.quantize(w1b, dtype=oracle.BF16)))
    pure = oracle.requantize(Y1ref.astype(np.float32))
    differing = float((pure[0] != h_ref[0]).mean())
    assert differing <= 1e-4, f"{differing} of the code bytes differ from the oracle's own chain"
    # a third layer through the product that takes and gives quantised operands
    w3b = inputs.weights_normal(d1, d2, seed=23)
    W3q = bd.quantize_weights(to_device(w3b, torch.bfloat16), bd.SELECT_TWO_STAGE)
    H2 = bd.gemm_requant(H, W2q)
    assert_bit_exact(H2, oracle.requantize(Y), "layer-2 operand")
    Y3 = bd.gemm(H2, W3q, dtype=torch.float32).cpu().numpy()
    Yref3, T3 = oracle.gemm(oracle.dequantize(*oracle.requantize(Y)), oracle.dequantize(*oracle.quantize(w3b, dtype=oracle.BF16)))
    ok, ratio = gemm_tolerance_ok(Y3, Yref3, T3)
    assert ok, f"layer 3: max err / bound = {ratio}"
    bd.poll_status()
