"""Block sizes 16 and 64 (the block-size study of Sec. 4.2, Table 3): codes, dialect ids and scales bit for bit against
the oracle run with the same block size, for both selection rules and every source type, and the product of two such
operands against the oracle's fp64 product within the tolerance."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import ORACLE_DTYPE, gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu

GUARD = 4096


@pytest.fixture(autouse=True)
def _reset_impl():
    yield
    bd.set_gemm_impl(bd.GEMM_AUTO)


def _host(x, kind):
    if kind == torch.float32:
        return x
    if kind == torch.bfloat16:
        return inputs.to_bf16_bits(x)
    return inputs.to_f16_bits(np.clip(x, -6e4, 6e4))


def _assert_canonical_equal(q, block, ref, what):
    got = [t.cpu().numpy() for t in bd.export_canonical_bs(q, block)]
    for name, g, r in zip(("scales", "ids", "codes"), (got[2], got[1], got[0]), (ref[2], ref[1], ref[0])):
        assert g.shape == r.shape, f"{what}: {name} shape {g.shape} vs {r.shape}"
        bad = np.argwhere(g != r)
        assert bad.size == 0, f"{what}: {len(bad)} {name} mismatches, first at {bad[0]}"


@pytest.mark.parametrize("block", [16, 32, 64])
@pytest.mark.parametrize("rows,K,kind,mse", [(1, 64, torch.float32, 0), (33, 192, torch.bfloat16, 0), (130, 448, torch.float16, 0),
                                             (200, 1024, torch.bfloat16, 1), (64, 320, torch.float32, 1), (517, 4096, torch.bfloat16, 0)])
def test_quantizer_block_sizes_bit_exact(block, rows, K, kind, mse):
    rng = np.random.default_rng(rows * 7 + K + block)
    x = (rng.standard_t(4, (rows, K)) * np.exp2(rng.integers(-10, 11, (rows, 1)))).astype(np.float32)
    x[:, rng.integers(0, K)] *= 40
    x[0, :block] = 0.0                                           # an all-zero block
    host = _host(x, kind)
    select = oracle.SELECT_MSE if mse else oracle.SELECT_TWO_STAGE
    q = bd.QTensor(rows, bd.physical_k(K, block))
    raws = {}
    for name in ("codes", "ids", "scales"):
        n = getattr(q, name).numel()
        raw = torch.full((n + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        raws[name] = (raw, n)
        setattr(q, name, raw[GUARD:GUARD + n])
    wide = torch.zeros(rows, K + 32, dtype=kind, device="cuda")
    wide[:, :K] = to_device(host, kind)
    bd.quantize_bs(wide[:, :K], block, select=select, out=q)
    _assert_canonical_equal(q, block, oracle.quantize(host, select, dtype=ORACLE_DTYPE[kind], block=block), f"{rows}x{K} block {block}")
    for raw, n in raws.values():
        assert bool((raw[:GUARD] == 0xA5).all()) and bool((raw[GUARD + n:] == 0xA5).all()), "write outside a buffer"
    # the stored operand dequantises to the oracle's values (block 16: real elements interleaved with zero halves)
    dq = bd.dequantize(q).cpu().numpy().astype(np.float64)
    ref = oracle.dequantize(*oracle.quantize(host, select, dtype=ORACLE_DTYPE[kind], block=block))
    if block == 16:
        dq = dq.reshape(rows, K // 16, 32)
        assert not dq[:, :, 16:].any()
        dq = dq[:, :, :16].reshape(rows, K)
    assert np.array_equal(dq, ref)
    bd.poll_status()


@pytest.mark.parametrize("block", [16, 64])
@pytest.mark.parametrize("M,N,K", [(5, 300, 128), (37, 264, 448), (300, 520, 1088), (128, 1024, 4096), (2048, 1024, 4096)])
@pytest.mark.parametrize("impl", [bd.GEMM_AUTO, bd.GEMM_SIMT])
def test_linear_with_other_block_sizes(block, M, N, K, impl):
    if impl == bd.GEMM_SIMT and M * N * K > 1 << 28:
        pytest.skip("the CUDA-core route is the cross-check for the small shapes")
    rng = np.random.default_rng(M + N + K + block)
    xb = inputs.to_bf16_bits((rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-4, 5, (M, 1)))).astype(np.float32))
    xb_f = inputs.bf16_bits_to_f32(xb)
    wb = inputs.weights_normal(N, K, seed=K + block)
    Wq = bd.quantize_bs(to_device(wb, torch.bfloat16), block, select=bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(impl)
    ws_bytes = bd.linear_bs_workspace_size(M, N, K, block)
    raw_ws = torch.full((ws_bytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    Y = bd.linear_bs(to_device(xb, torch.bfloat16), Wq, block, dtype=torch.float32, workspace=raw_ws[GUARD:GUARD + ws_bytes])
    torch.cuda.synchronize()
    assert bool((raw_ws[:GUARD] == 0xA5).all()) and bool((raw_ws[GUARD + ws_bytes:] == 0xA5).all()), "write outside the workspace"
    rows = np.unique(np.concatenate([[0, M - 1], rng.choice(M, min(M, 12), replace=False)]))
    qa = oracle.quantize(xb[rows], dtype=oracle.BF16, block=block)
    qb = oracle.quantize(wb, dtype=oracle.BF16, block=block)
    Yref, T = oracle.gemm(oracle.dequantize(*qa), oracle.dequantize(*qb))
    ok, ratio = gemm_tolerance_ok(Y.cpu().numpy()[rows], Yref, T)
    assert ok, f"block {block} {M}x{N}x{K}: max err / bound = {ratio}"
    # the paper's block MAC at this block size (integer sums, one rescale per block) gives the same product
    if M * N * K <= 1 << 24:
        assert np.abs(oracle.gemm_blockmac(qa, qb) - Yref).max() <= 1e-12 * T.max()
    # finer blocks follow the data more closely: mean squared quantisation error of X does not grow as blocks shrink
    del xb_f
    bd.poll_status()


def test_quantisation_error_shrinks_with_the_block_size():
    # the trend of Table 3 on synthetic activations with outlier channels: 16 <= 32 <= 64 in mean squared error
    xb = inputs.act_normal_outliers(256, 4096, seed=1)
    x = inputs.bf16_bits_to_f32(xb).astype(np.float64)
    xd = to_device(xb, torch.bfloat16)
    errs = []
    for block in (16, 32, 64):
        dq = bd.dequantize(bd.quantize_bs(xd, block)).cpu().numpy().astype(np.float64)
        if block == 16:
            dq = dq.reshape(256, 256, 32)[:, :, :16].reshape(256, 4096)
        errs.append(float(((dq - x) ** 2).mean()))
    assert errs[0] <= errs[1] <= errs[2], errs
