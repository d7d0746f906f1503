"""The warp-level linear layer for calls of at most 16 tokens (BD_GEMM_WARP) against the CPU oracle: every element,
guard bands around result and workspace, the shapes the decode phase has and ragged small ones."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu

GUARD = 4096


@pytest.fixture(autouse=True)
def _reset_impl():
    yield
    bd.set_gemm_impl(bd.GEMM_AUTO)


def _guarded(n_bytes):
    raw = torch.full((n_bytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
    return raw, raw[GUARD:GUARD + n_bytes]


def _intact(raw, n_bytes):
    return bool((raw[:GUARD] == 0xA5).all()) and bool((raw[GUARD + n_bytes:] == 0xA5).all())


def _host(x, kind):
    if kind == torch.float32:
        return x, oracle.F32
    if kind == torch.bfloat16:
        return inputs.to_bf16_bits(x), oracle.BF16
    return inputs.to_f16_bits(np.clip(x, -6e4, 6e4)), oracle.F16


CASES = [(1, 16, 128, torch.bfloat16), (2, 48, 256, torch.float32), (7, 144, 384, torch.float16), (8, 272, 1152, torch.bfloat16),
         (9, 16, 128, torch.bfloat16), (13, 4112, 640, torch.float32), (16, 1040, 2176, torch.bfloat16),
         (1, 4096, 4096, torch.bfloat16), (16, 4096, 4096, torch.bfloat16), (5, 11008, 4096, torch.float16),
         (16, 4096, 11008, torch.bfloat16), (1, 1024, 14336, torch.float32),
         # rows that do not fill the last tile of 16, K that does not fill the last unit of 128
         (4, 40, 256, torch.bfloat16), (4, 64, 96, torch.float32), (3, 4113, 128, torch.bfloat16), (8, 17, 32, torch.float16),
         (5, 130, 160, torch.bfloat16), (12, 1, 2080, torch.float32), (2, 2063, 4064, torch.bfloat16)]


@pytest.mark.parametrize("M,N,K,kind", CASES)
@pytest.mark.parametrize("impl", [bd.GEMM_WARP, bd.GEMM_AUTO])
def test_every_element_against_the_oracle(M, N, K, kind, impl):
    rng = np.random.default_rng(M + 31 * N + 977 * K)
    x = (rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-4, 5, (M, 1)))).astype(np.float32)
    host, odt = _host(x, kind)
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K)) * np.exp2(rng.integers(-3, 4, (N, 1)))).astype(np.float32))
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(host, dtype=odt)), oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    bd.set_gemm_impl(impl)
    xd = to_device(host, kind)
    ws_bytes = bd.linear_workspace_size(M, N, K)
    for ydt in (torch.float32, torch.bfloat16):
        esz = 4 if ydt == torch.float32 else 2
        ldy = N + 8
        raw_y, ybytes = _guarded(M * ldy * esz)
        y = ybytes.view(ydt).view(M, ldy)
        y.fill_(-7.0)
        raw_ws, ws = _guarded(ws_bytes)
        before = bd.launch_count()
        bd.linear(xd, Wq, out=y[:, :N], workspace=ws)
        torch.cuda.synchronize()
        if impl == bd.GEMM_WARP or (N * K >= 1 << 18 and (M <= 8 or N * K <= 1 << 25)):   # the library's own choice: see bd.h
            assert bd.launch_count() - before == 2, "expected the record quantizer and the product"
        assert _intact(raw_y, M * ldy * esz) and _intact(raw_ws, ws_bytes), "write outside a buffer"
        assert (y[:, N:] == -7.0).all(), "write into the padding columns"
        got = y[:, :N].float().cpu().numpy().astype(np.float64)
        bound = 1e-6 * T + (2.0 ** -8 * np.abs(Yref) if ydt == torch.bfloat16 else 0.0) + 2.0 ** -120
        err = np.abs(got - Yref)
        assert (err <= bound).all(), f"{M}x{N}x{K} {kind} -> {ydt}: max err / bound = {float((err / bound).max())}"
    bd.poll_status()


def test_a_single_nonzero_block_is_exact():
    # one block of K carries data, the rest is zero: the result is one in-block sum times two powers of two, which
    # fp32 holds exactly, so the kernel must return the oracle's value bit for bit (Sec. 3.3: integer in-block sums)
    rng = np.random.default_rng(5)
    M, N, K = 8, 64, 512
    for blk in (0, 5, 15):
        x = np.zeros((M, K), np.float32)
        w = np.zeros((N, K), np.float32)
        x[:, 32 * blk:32 * blk + 32] = rng.standard_t(3, (M, 32)) * np.exp2(rng.integers(-6, 7, (M, 1)))
        w[:, 32 * blk:32 * blk + 32] = rng.standard_normal((N, 32)) * np.exp2(rng.integers(-9, 2, (N, 1)))
        wb = inputs.to_bf16_bits(w)
        Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
        Yref, _ = oracle.gemm(oracle.dequantize(*oracle.quantize(x)), oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
        bd.set_gemm_impl(bd.GEMM_WARP)
        Y = bd.linear(to_device(x, torch.float32), Wq, dtype=torch.float32).cpu().numpy()
        assert np.array_equal(Y.astype(np.float64), Yref), f"block {blk}: {np.abs(Y - Yref).max()}"
    bd.poll_status()


def test_zero_rows_and_zero_blocks_give_zeros_not_nans():
    # an all-zero weight row stores scale byte 0; activations with a block maximum in [2, 4) store 126: the two
    # exponent fields must not meet in a way that makes 0 * inf
    M, N, K = 4, 32, 256
    x = np.full((M, K), 3.0, np.float32)
    x[1] = 0.0
    w = np.zeros((N, K), np.float32)
    w[3] = 1.0
    wb = inputs.to_bf16_bits(w)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(bd.GEMM_WARP)
    Y = bd.linear(to_device(x, torch.float32), Wq, dtype=torch.float32).cpu().numpy()
    Yref, _ = oracle.gemm(oracle.dequantize(*oracle.quantize(x)), oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    assert np.isfinite(Y).all()
    assert np.array_equal(Y.astype(np.float64), Yref)
    bd.poll_status()


def test_block_scales_far_apart():
    # token rows and weight rows whose magnitudes span 2^-30 .. 2^30: the fp32 factors of the two operands are
    # applied one after the other, so no single factor leaves the fp32 range
    rng = np.random.default_rng(9)
    M, N, K = 16, 128, 1024
    x = (rng.standard_normal((M, K)) * np.exp2(rng.integers(-30, 31, (M, 1)))).astype(np.float32)
    w = (rng.standard_normal((N, K)) * np.exp2(rng.integers(-30, 31, (N, 1)))).astype(np.float32)
    wb = inputs.to_bf16_bits(w)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(x)), oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    bd.set_gemm_impl(bd.GEMM_WARP)
    Y = bd.linear(to_device(x, torch.float32), Wq, dtype=torch.float32).cpu().numpy()
    ok, ratio = gemm_tolerance_ok(Y, Yref, T)
    assert ok, f"max err / bound = {ratio}"
    bd.poll_status()


def test_more_than_16_tokens_are_refused_when_forced():
    M, N, K = 17, 64, 256
    x = torch.randn(M, K, device="cuda", dtype=torch.bfloat16)
    Wq = bd.quantize_weights(torch.randn(N, K, device="cuda", dtype=torch.bfloat16), bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(bd.GEMM_WARP)
    with pytest.raises(bd.BdError):
        bd.linear(x, Wq)
    bd.set_gemm_impl(bd.GEMM_AUTO)
    bd.linear(x, Wq)                                              # the library's own choice serves them
    torch.cuda.synchronize()
    bd.poll_status()


@pytest.mark.parametrize("M,N,K", [(1, 16, 128), (4, 4113, 128), (4, 128, 4096), (8, 130, 160), (11, 257, 1056), (16, 48, 32)])
@pytest.mark.parametrize("ydt", [torch.float32, torch.bfloat16])
def test_product_of_two_quantised_operands(M, N, K, ydt):
    # bd_gemm with a few rows of A: the records come from A's codes, not from a quantizer; every element against the
    # oracle's product of the same two quantised operands, guard bands around the result and the workspace
    rng = np.random.default_rng(M + 31 * N + 977 * K)
    a = inputs.to_bf16_bits((rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-4, 5, (M, 1)))).astype(np.float32))
    b = inputs.to_bf16_bits((rng.standard_normal((N, K)) * np.exp2(rng.integers(-3, 4, (N, 1)))).astype(np.float32))
    qa, qb = bd.quantize_act(to_device(a, torch.bfloat16)), bd.quantize_act(to_device(b, torch.bfloat16))
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(a, dtype=oracle.BF16)), oracle.dequantize(*oracle.quantize(b, dtype=oracle.BF16)))
    bd.set_gemm_impl(bd.GEMM_WARP)
    esz = 4 if ydt == torch.float32 else 2
    ldy = N + 8
    raw_y, ybytes = _guarded(M * ldy * esz)
    y = ybytes.view(ydt).view(M, ldy)
    y.fill_(-7.0)
    ws_bytes = bd.gemm_workspace_size(M, N, K)
    raw_ws, ws = _guarded(ws_bytes)
    before = bd.launch_count()
    bd.gemm(qa, qb, out=y[:, :N], workspace=ws)
    torch.cuda.synchronize()
    assert bd.launch_count() - before == 2
    assert _intact(raw_y, M * ldy * esz) and _intact(raw_ws, ws_bytes), "write outside a buffer"
    assert (y[:, N:] == -7.0).all(), "write into the padding columns"
    err = np.abs(y[:, :N].float().cpu().numpy().astype(np.float64) - Yref)
    bound = 1e-6 * T + (2.0 ** -8 * np.abs(Yref) if ydt == torch.bfloat16 else 0.0) + 2.0 ** -120
    assert (err <= bound).all(), f"max err / bound = {float((err / bound).max())}"
    bd.poll_status()


def test_graph_replay_and_back_to_back_calls():
    # the two launches are linked by programmatic dependent launch and share the record area of the workspace:
    # calls with different activations behind one another, eagerly and replayed from a CUDA graph, must each see their own
    rng = np.random.default_rng(11)
    M, N, K = 4, 2048, 2048
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    wdq = oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16))
    xs = [inputs.to_bf16_bits(rng.standard_t(4, (M, K)).astype(np.float32)) for _ in range(4)]
    refs = [oracle.gemm(oracle.dequantize(*oracle.quantize(x, dtype=oracle.BF16)), wdq) for x in xs]
    xd = [to_device(x, torch.bfloat16) for x in xs]
    ws = torch.empty(bd.linear_workspace_size(M, N, K), dtype=torch.uint8, device="cuda")
    ys = [torch.empty(M, N, dtype=torch.float32, device="cuda") for _ in xs]
    for _ in range(3):
        for x, y in zip(xd, ys):
            bd.linear(x, Wq, out=y, workspace=ws)
    torch.cuda.synchronize()
    for y, (Yref, T) in zip(ys, refs):
        ok, ratio = gemm_tolerance_ok(y.cpu().numpy(), Yref, T)
        assert ok, ratio
    st = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    for y in ys:
        y.zero_()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for x, y in zip(xd, ys):
                bd.linear(x, Wq, out=y, workspace=ws)
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for y, (Yref, T) in zip(ys, refs):
        ok, ratio = gemm_tolerance_ok(y.cpu().numpy(), Yref, T)
        assert ok, ratio
    bd.poll_status()


def _fuzz_cases():
    rng = np.random.default_rng(77)
    return [(int(rng.integers(1, 17)), int(rng.integers(1, 700)), 32 * int(rng.integers(1, 81)), [torch.bfloat16, torch.float32, torch.float16][i % 3])
            for i in range(24)]


@pytest.mark.parametrize("M,N,K,kind", _fuzz_cases())
def test_random_shapes_against_the_exact_cuda_core_kernel(M, N, K, kind):
    # every element against the library's CUDA-core product (exact integer block sums, fp64 across blocks), which
    # shares nothing with this kernel after the weights' codes; guard bands as above
    rng = np.random.default_rng(M + 31 * N + K)
    x = (rng.standard_t(3, (M, K)) * np.exp2(rng.integers(-6, 7, (M, 1)))).astype(np.float32)
    w = (rng.standard_normal((N, K)) * np.exp2(rng.integers(-8, 3, (N, 1)))).astype(np.float32)
    host, _ = _host(x, kind)
    xd = to_device(host, kind)
    Wq = bd.quantize_weights(to_device(inputs.to_bf16_bits(w), torch.bfloat16), bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(bd.GEMM_SIMT)
    Yexact = bd.linear(xd, Wq, dtype=torch.float32)
    bound = 2e-6 * (bd.dequantize(bd.quantize_act(xd)).abs() @ bd.dequantize(Wq).abs().T) + 2.0 ** -120
    bd.set_gemm_impl(bd.GEMM_WARP)
    ws_bytes = bd.linear_workspace_size(M, N, K)
    raw_ws, ws = _guarded(ws_bytes)
    raw_y, ybytes = _guarded(M * N * 4)
    y = ybytes.view(torch.float32).view(M, N)
    bd.linear(xd, Wq, out=y, workspace=ws)
    torch.cuda.synchronize()
    assert _intact(raw_y, M * N * 4) and _intact(raw_ws, ws_bytes), "write outside a buffer"
    assert bool(((y - Yexact).abs() <= bound).all()), f"{M}x{N}x{K}: max err / bound = {float(((y - Yexact).abs() / bound).max())}"
    bd.poll_status()


@pytest.mark.parametrize("heads,group,M,N,K", [(8, 4, 4, 4113, 128), (6, 1, 1, 130, 160), (70, 2, 9, 48, 64), (4, 2, 16, 257, 1056)])
@pytest.mark.parametrize("ydt", [torch.float32, torch.bfloat16])
def test_batched_products_with_a_few_rows_share_a_launch(heads, group, M, N, K, ydt):
    # bd_gemm_batched with at most 16 rows of A per product: all products (64 per launch) through grid.y of the
    # warp-level kernel, which expands the A operands' code words itself; every head against the oracle
    rng = np.random.default_rng(heads + 31 * M + 977 * N + K)
    a = inputs.to_bf16_bits((rng.standard_t(4, (heads, M, K)) * np.exp2(rng.integers(-3, 4, (heads, M, 1)))).astype(np.float32))
    b = inputs.to_bf16_bits(rng.standard_normal((heads // group, N, K)).astype(np.float32))
    As = [bd.quantize_act(to_device(a[h], torch.bfloat16)) for h in range(heads)]
    Bs = [bd.quantize_act(to_device(b[g], torch.bfloat16)) for g in range(heads // group)]
    esz = 4 if ydt == torch.float32 else 2
    raw_y, ybytes = _guarded(heads * M * N * esz)
    out = ybytes.view(ydt).view(heads, M, N)
    ws_bytes = bd.gemm_batched_workspace_size(M, N, K, group)
    raw_ws, ws = _guarded(max(ws_bytes, 256))
    bd.set_gemm_impl(bd.GEMM_WARP)                                # (the library's own choice leaves tiny products to the CUDA-core kernel)
    before = bd.launch_count()
    bd.gemm_batched(As, Bs, b_group=group, out=out, workspace=ws)
    torch.cuda.synchronize()
    assert bd.launch_count() - before == (heads + 63) // 64
    assert _intact(raw_y, heads * M * N * esz) and _intact(raw_ws, max(ws_bytes, 256)), "write outside a buffer"
    for h in range(heads):
        Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(a[h], dtype=oracle.BF16)), oracle.dequantize(*oracle.quantize(b[h // group], dtype=oracle.BF16)))
        err = np.abs(out[h].float().cpu().numpy().astype(np.float64) - Yref)
        bound = 1e-6 * T + (2.0 ** -8 * np.abs(Yref) if ydt == torch.bfloat16 else 0.0) + 2.0 ** -120
        assert (err <= bound).all(), f"head {h}: max err / bound = {float((err / bound).max())}"
    bd.poll_status()


def test_weights_quantised_right_before_the_call():
    # the weights are rewritten by bd_quantize_weights and used by the next call on the stream with nothing in between,
    # twelve times over the same buffers: the product kernel's early copies of the weights must not overtake the kernel
    # that writes them (the record kernel in front waits for it before it lets the product kernel start)
    rng = np.random.default_rng(21)
    M, N, K, reps = 4, 512, 1024, 12
    xb = inputs.to_bf16_bits(rng.standard_t(4, (M, K)).astype(np.float32))
    xd = to_device(xb, torch.bfloat16)
    ws_host = [inputs.to_bf16_bits((rng.standard_normal((N, K)) * np.exp2(rng.integers(-6, 1, (N, 1)))).astype(np.float32)) for _ in range(reps)]
    ws_dev = [to_device(w, torch.bfloat16) for w in ws_host]
    Wq = bd.QTensor(N, K)
    ws = torch.empty(bd.linear_workspace_size(M, N, K), dtype=torch.uint8, device="cuda")
    ys = [torch.empty(M, N, dtype=torch.float32, device="cuda") for _ in range(reps)]
    bd.set_gemm_impl(bd.GEMM_WARP)
    torch.cuda.synchronize()
    for i in range(reps):
        bd.quantize_weights(ws_dev[i], bd.SELECT_TWO_STAGE, out=Wq)
        bd.linear(xd, Wq, out=ys[i], workspace=ws)
    torch.cuda.synchronize()
    xq = oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16))
    for i in range(reps):
        Yref, T = oracle.gemm(xq, oracle.dequantize(*oracle.quantize(ws_host[i], dtype=oracle.BF16)))
        ok, ratio = gemm_tolerance_ok(ys[i].cpu().numpy(), Yref, T)
        assert ok, f"call {i}: max err / bound = {ratio}"
    bd.poll_status()
