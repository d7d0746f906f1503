"""bd_set_formatbook on the GPU: with another table loaded on both sides (the CUDA library and the
oracle each rebuild their own tables from it), quantisation stays bit-exact and the products stay
inside the tolerance; restoring the built-in table gives the original results back."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import assert_bit_exact, gemm_tolerance_ok, oracle_quantize, to_device

pytestmark = pytest.mark.gpu


def _alternative(default):
    alt = default.copy()
    alt[0, 6], alt[1, 6] = 13, 11                       # other slot-6 values
    alt[2, 6], alt[3, 6] = 12, 10
    alt[6] = [0, 1, 2, 3, 5, 7, 10, 12]                 # another common set for pair 3
    alt[7] = [0, 1, 2, 3, 5, 7, 8, 12]
    alt[10, 6], alt[11, 6] = 9, 8
    return alt


def test_alternative_formatbook_end_to_end():
    default = oracle.formatbook()
    assert (bd.get_formatbook().numpy() == default).all()
    alt = _alternative(default)
    M, K, N = 300, 1024, 260
    xb = inputs.act_student_t(M, K, seed=11)
    wb = inputs.weights_normal(N, K, seed=12)
    x, w = to_device(xb, torch.bfloat16), to_device(wb, torch.bfloat16)
    before = [t.clone() for t in bd.export_canonical(bd.quantize_act(x))]
    try:
        bd.set_formatbook(alt)
        oracle.set_formatbook(alt)
        assert (bd.get_formatbook().numpy() == alt).all()
        qx = bd.quantize_act(x)
        ref_x = oracle_quantize(xb, torch.bfloat16)
        assert_bit_exact(qx, ref_x, "activations, alternative table")
        assert not all(torch.equal(a, b) for a, b in zip(before, bd.export_canonical(qx))), "the table had no effect"
        qw = bd.quantize_weights(w, bd.SELECT_MSE)
        ref_w = oracle_quantize(wb, torch.bfloat16, oracle.SELECT_MSE)
        assert_bit_exact(qw, ref_w, "weights (MSE rule), alternative table")
        Yref, T = oracle.gemm(oracle.dequantize(*ref_x), oracle.dequantize(*ref_w))
        for impl in (bd.GEMM_SIMT, bd.GEMM_TCGEN05):
            bd.set_gemm_impl(impl)
            ok, ratio = gemm_tolerance_ok(bd.gemm(qx, qw).cpu().numpy(), Yref, T)
            assert ok, f"impl {impl}: max err / bound = {ratio}"
        # the warp-level kernel reads the table of half-unit integers: a few rows of A through both of its front ends
        bd.set_gemm_impl(bd.GEMM_WARP)
        qx11 = bd.quantize_act(x[:11])
        Yref11, T11 = oracle.gemm(oracle.dequantize(*oracle_quantize(xb[:11], torch.bfloat16)), oracle.dequantize(*ref_w))
        ok, ratio = gemm_tolerance_ok(bd.gemm(qx11, qw).cpu().numpy(), Yref11, T11)
        assert ok, f"warp-level kernel, bd_gemm: max err / bound = {ratio}"
        ok, ratio = gemm_tolerance_ok(bd.linear(x[:11], qw, dtype=torch.float32).cpu().numpy(), Yref11, T11)
        assert ok, f"warp-level kernel, bd_linear: max err / bound = {ratio}"
        bd.set_gemm_impl(bd.GEMM_AUTO)
        Y = bd.linear(x, bd.quantize_weights(w, bd.SELECT_TWO_STAGE), dtype=torch.float32).cpu().numpy()
        ref_w2 = oracle_quantize(wb, torch.bfloat16)
        Yref2, T2 = oracle.gemm(oracle.dequantize(*ref_x), oracle.dequantize(*ref_w2))
        ok, ratio = gemm_tolerance_ok(Y, Yref2, T2)
        assert ok, f"bd_linear: max err / bound = {ratio}"
        deq = bd.dequantize(qx).cpu().numpy()
        assert np.array_equal(deq, oracle.dequantize(*ref_x).astype(np.float32))
    finally:
        bd.set_gemm_impl(bd.GEMM_AUTO)
        bd.set_formatbook(None)
        oracle.set_formatbook(None)
    assert (bd.get_formatbook().numpy() == default).all()
    after = bd.export_canonical(bd.quantize_act(x))
    assert all(torch.equal(a, b) for a, b in zip(before, after))
    bd.poll_status()


def _random_book(rng):
    """A table with the pair structure the library asks for: pair p has maximum 15 - p, its two rows share the
    six smallest values and differ in the seventh (the even row's is the larger)."""
    book = np.zeros((16, 8), np.uint8)
    for p in range(8):
        mx = 15 - p
        while True:
            picks = np.sort(rng.choice(np.arange(1, mx), 7, replace=False))
            common, d_odd, d_even = picks[:5], picks[5], picks[6]
            if d_even < mx:
                break
        book[2 * p] = [0, *common, d_even, mx]
        book[2 * p + 1] = [0, *common, d_odd, mx]
    return book


@pytest.mark.parametrize("seed", range(6))
def test_random_formatbooks(seed):
    # tables drawn at random within the structure the kernels assume (those the library's own check refuses are
    # drawn again): quantizer in both output forms, MSE rule and both product kernels against the oracle with
    # the same table
    rng = np.random.default_rng(500 + seed)
    M, K, N = 130, 512, 200
    xb = inputs.to_bf16_bits((rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-3, 4, (M, 1)))).astype(np.float32))
    xf = (rng.standard_normal((M, K)) * 3).astype(np.float32)
    wb = inputs.to_bf16_bits((0.05 * rng.standard_normal((N, K))).astype(np.float32))
    try:
        for _ in range(200):
            book = _random_book(rng)
            try:
                bd.set_formatbook(book)
                break
            except bd.BdError:
                continue
        else:
            pytest.skip("no acceptable table drawn")
        oracle.set_formatbook(book)
        x, w = to_device(xb, torch.bfloat16), to_device(wb, torch.bfloat16)
        ref_x = oracle_quantize(xb, torch.bfloat16)
        assert_bit_exact(bd.quantize_act(x), ref_x, "bf16 activations")
        assert_bit_exact(bd.quantize_act(to_device(xf, torch.float32)), oracle_quantize(xf, torch.float32), "fp32 activations")
        assert_bit_exact(bd.quantize_weights(w, bd.SELECT_MSE), oracle_quantize(wb, torch.bfloat16, oracle.SELECT_MSE), "MSE")
        ref_w = oracle_quantize(wb, torch.bfloat16)
        Wq = bd.quantize_weights(w, bd.SELECT_TWO_STAGE)
        assert_bit_exact(Wq, ref_w, "weights")
        Yref, T = oracle.gemm(oracle.dequantize(*ref_x), oracle.dequantize(*ref_w))
        for impl in (bd.GEMM_SIMT, bd.GEMM_TCGEN05):
            bd.set_gemm_impl(impl)
            ok, ratio = gemm_tolerance_ok(bd.linear(x, Wq, dtype=torch.float32).cpu().numpy(), Yref, T)
            assert ok, f"impl {impl}: max err / bound = {ratio}"
        bd.set_gemm_impl(bd.GEMM_WARP)
        ok, ratio = gemm_tolerance_ok(bd.linear(x[:7], Wq, dtype=torch.float32).cpu().numpy(), Yref[:7], T[:7])
        assert ok, f"warp-level kernel: max err / bound = {ratio}"
    finally:
        bd.set_gemm_impl(bd.GEMM_AUTO)
        bd.set_formatbook(None)
        oracle.set_formatbook(None)
    bd.poll_status()
