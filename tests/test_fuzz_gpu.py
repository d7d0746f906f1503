"""Seeded sweeps of shapes through the quantizers and the linear layer against the CPU oracle.  Every output
and the workspace sit between pattern-filled guard bands, so a store outside a buffer shows as a changed guard
byte even where it would not change a result."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import assert_bit_exact, gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu

GUARD = 4096
EDGES = [1, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 320, 384, 448, 512]


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


def _quantizer_cases():
    rng = np.random.default_rng(101)
    kinds = [torch.bfloat16, torch.float32, torch.float16]
    cases = []
    for i in range(36):
        rows = int(rng.choice(EDGES)) if i % 3 else int(rng.integers(1, 520))
        K = 32 * int(rng.choice([1, 2, 3, 4, 5, 8, 12, 16, 17, 32]) if i % 2 else rng.integers(1, 48))
        cases.append((rows, K, kinds[i % 3], int(rng.choice([0, 32, 64])), int(i % 5 == 4)))
    return cases


@pytest.mark.parametrize("rows,K,kind,ld_extra,mse", _quantizer_cases())
def test_quantizer_shapes_with_guard_bands(rows, K, kind, ld_extra, mse):
    rng = np.random.default_rng(rows * 131 + K)
    x = (rng.standard_t(4, (rows, K)) * np.exp2(rng.integers(-8, 9, (rows, 1)))).astype(np.float32)
    host, odt = _host(x, kind)
    wide = torch.zeros(rows, K + ld_extra, dtype=kind, device="cuda")
    wide[:, :K] = to_device(host, kind)
    q = bd.QTensor(rows, K)
    raws = {}
    for name in ("codes", "ids", "scales"):
        n = getattr(q, name).numel()
        raws[name], view = _guarded(n)
        setattr(q, name, view)
    if mse:
        bd.quantize_weights(wide[:, :K], bd.SELECT_MSE, out=q)
        ref = oracle.quantize(host, oracle.SELECT_MSE, dtype=odt)
    else:
        bd.quantize_act(wide[:, :K], out=q)
        ref = oracle.quantize(host, dtype=odt)
    assert_bit_exact(q, ref, f"{rows}x{K} {kind} ld+{ld_extra} mse={mse}")
    for name, raw in raws.items():
        assert _intact(raw, raw.numel() - 2 * GUARD), f"{name}: write outside the buffer"
    bd.poll_status()


def _linear_cases():
    rng = np.random.default_rng(202)
    cases = []
    for i in range(30):
        M = int(rng.choice(EDGES)) if i % 2 else int(rng.integers(1, 300))
        N = int(rng.choice([8, 127, 128, 129, 255, 256, 257, 384])) if i % 3 == 0 else int(rng.integers(8, 400))
        K = 32 * int(rng.integers(1, 33))
        cases.append((M, N, K, [torch.bfloat16, torch.float32, torch.float16][i % 3], i % 2))
    return cases


@pytest.mark.parametrize("M,N,K,kind,forced", _linear_cases())
def test_linear_shapes_with_guard_bands(M, N, K, kind, forced):
    rng = np.random.default_rng(M * 7 + N * 131 + K)
    x = (rng.standard_t(4, (M, K)) * np.exp2(rng.integers(-4, 5, (M, 1)))).astype(np.float32)
    host, odt = _host(x, kind)
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(host, dtype=odt)),
                          oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    if forced:
        bd.set_gemm_impl(bd.GEMM_TCGEN05)                         # otherwise the library's own choice by shape
    xd = to_device(host, kind)
    ws_bytes = bd.linear_workspace_size(M, N, K)
    for ydt in (torch.float32, torch.bfloat16):
        esz = 4 if ydt == torch.float32 else 2
        ldy = N + 8
        raw_y, ybytes = _guarded(M * ldy * esz)
        y = ybytes.view(ydt).view(M, ldy)
        y.fill_(-7.0)
        raw_ws, ws = _guarded(ws_bytes)
        bd.linear(xd, Wq, out=y[:, :N], workspace=ws)
        torch.cuda.synchronize()
        assert _intact(raw_y, M * ldy * esz) and _intact(raw_ws, ws_bytes), "write outside a buffer"
        assert (y[:, N:] == -7.0).all(), "write into the padding columns"
        got = y[:, :N].float().cpu().numpy()
        if ydt == torch.float32:
            ok, ratio = gemm_tolerance_ok(got, Yref, T)
        else:
            err = np.abs(got.astype(np.float64) - Yref)
            bound = 1e-6 * T + 2.0 ** -8 * np.abs(Yref) + 2.0 ** -120
            ok, ratio = bool((err <= bound).all()), float((err / bound).max())
        assert ok, f"{M}x{N}x{K} {kind} -> {ydt}: max err / bound = {ratio}"
    bd.poll_status()


@pytest.mark.parametrize("tokens,dim,kind", [(32, 8, torch.bfloat16), (64, 128, torch.float32), (96, 33, torch.float16),
                                             (320, 128, torch.bfloat16), (4096, 128, torch.bfloat16), (160, 257, torch.float32),
                                             (1024, 64, torch.float16), (32, 1, torch.bfloat16)])
def test_token_axis_quantizer_shapes(tokens, dim, kind):
    # V [tokens, dim] with blocks of 32 along the tokens: equals quantising the transpose along its rows
    rng = np.random.default_rng(tokens + 977 * dim)
    v = (rng.standard_normal((tokens, dim)) * np.exp2(rng.integers(-6, 7, (1, dim)))).astype(np.float32)
    host, odt = _host(v, kind)
    pad = (-dim) % 8                                              # a row pitch of whole 16 bytes
    wide = torch.zeros(tokens, dim + pad, dtype=kind, device="cuda")
    wide[:, :dim] = to_device(host, kind)
    q = bd.QTensor(dim, tokens)
    raws = {}
    for name in ("codes", "ids", "scales"):
        n = getattr(q, name).numel()
        raws[name], view = _guarded(n)
        setattr(q, name, view)
    bd.quantize_act(wide[:, :dim], axis=bd.AXIS_STRIDED, out=q)
    assert_bit_exact(q, oracle.quantize(np.ascontiguousarray(host.T), dtype=odt), f"token axis {tokens}x{dim} {kind}")
    for name, raw in raws.items():
        assert _intact(raw, raw.numel() - 2 * GUARD), f"{name}: write outside the buffer"
    bd.poll_status()


@pytest.mark.parametrize("heads,group,S,T_,d", [(4, 2, 128, 96, 64), (6, 3, 256, 200, 160), (8, 4, 384, 130, 32),
                                                (3, 1, 100, 257, 96), (4, 4, 128, 512, 128), (2, 2, 130, 64, 64)])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_batched_grouped_products(heads, group, S, T_, d, dtype):
    # queries [heads][S, d] against keys [heads / group][T_, d]: stacked launches where the rows are whole tiles
    # (S a multiple of 128), one launch per product otherwise; every head against the oracle, guard bands around
    # the result and the workspace
    rng = np.random.default_rng(heads + 31 * S + 977 * d)
    q = inputs.to_bf16_bits(rng.standard_normal((heads, S, d)).astype(np.float32))
    k = inputs.to_bf16_bits(rng.standard_normal((heads // group, T_, d)).astype(np.float32))
    As = [bd.quantize_act(to_device(q[h], torch.bfloat16)) for h in range(heads)]
    Bs = [bd.quantize_act(to_device(k[g], torch.bfloat16)) for g in range(heads // group)]
    bd.set_gemm_impl(bd.GEMM_TCGEN05)
    esz = 4 if dtype == torch.float32 else 2
    raw_y, ybytes = _guarded(heads * S * T_ * esz)
    out = ybytes.view(dtype).view(heads, S, T_)
    ws_bytes = bd.gemm_batched_workspace_size(S, T_, d, group)
    raw_ws, ws = _guarded(ws_bytes)
    bd.gemm_batched(As, Bs, b_group=group, out=out, workspace=ws)
    torch.cuda.synchronize()
    assert _intact(raw_y, heads * S * T_ * esz) and _intact(raw_ws, ws_bytes), "write outside a buffer"
    for h in range(heads):
        Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(q[h], dtype=oracle.BF16)),
                              oracle.dequantize(*oracle.quantize(k[h // group], dtype=oracle.BF16)))
        err = np.abs(out[h].float().cpu().numpy().astype(np.float64) - Yref)
        bound = 1e-6 * T + (2.0 ** -8 * np.abs(Yref) if dtype == torch.bfloat16 else 0.0) + 2.0 ** -120
        assert (err <= bound).all(), f"head {h}: max err / bound = {float((err / bound).max())}"
    bd.poll_status()


@pytest.mark.parametrize("M,N,K", [(1280, 3840, 256),      # 75 tiles: one more than the clusters of a wave
                                   (768, 9472, 128),       # 111 tiles: a last wave half full (128-token items)
                                   (1792, 4096, 160),      # 112 tiles: a last wave just over half full
                                   (1700, 5376, 128),      # 147 tiles, ragged last token tile
                                   (1536, 6400, 96),       # 150 tiles: two items into the third wave
                                   (2304, 1000, 256),      # ragged weight rows, nine token tiles
                                   (640, 19200, 64)])      # many weight-row pairs, few token tiles
def test_schedules_over_several_waves(M, N, K):
    # tile counts near whole and half waves of the persistent kernel (a wave = one tile per cluster); sampled rows and columns (tile edges
    # included) against the oracle, and the bf16 output must be the rounded fp32 one
    rng = np.random.default_rng(M + 31 * N + K)
    xb = inputs.to_bf16_bits((rng.standard_t(4, (M, K))).astype(np.float32))
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    xd = to_device(xb, torch.bfloat16)
    Y32 = bd.linear(xd, Wq, dtype=torch.float32)
    Y = Y32.cpu().numpy()
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M - 129, M - 128, M - 1], rng.choice(M, 6, replace=False)]))
    cols = np.unique(np.concatenate([[0, 127, 128, 255, 256, N - 257, N - 256, N - 1], rng.choice(N, 6, replace=False)]))
    wdq = oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16))
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb[rows], dtype=oracle.BF16)), wdq)
    ok, ratio = gemm_tolerance_ok(Y[rows], Yref, T)
    assert ok, f"rows: max err / bound = {ratio}"
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)), wdq[cols])
    ok, ratio = gemm_tolerance_ok(Y[:, cols], Yref, T)
    assert ok, f"cols: max err / bound = {ratio}"
    assert torch.equal(bd.linear(xd, Wq, dtype=torch.bfloat16), Y32.to(torch.bfloat16))
    # every element, against the library's other product kernel (CUDA cores, exact block sums, fp64 across
    # blocks): the two share no code path after the quantizer, so a tile one of them misses shows here
    bd.set_gemm_impl(bd.GEMM_SIMT)
    Yexact = bd.linear(xd, Wq, dtype=torch.float32)
    Aabs = bd.dequantize(bd.quantize_act(xd)).abs()
    Wabs = bd.dequantize(Wq).abs()
    bound = 2e-6 * (Aabs @ Wabs.T) + 2.0 ** -120
    assert bool(((Y32 - Yexact).abs() <= bound).all())
    bd.poll_status()


@pytest.mark.parametrize("M,N,K", [(1, 256, 8192), (5, 300, 2144), (16, 520, 4128), (100, 520, 4128), (128, 1024, 4096),
                                   (64, 4096, 2048)])
@pytest.mark.parametrize("ydt", [torch.float32, torch.bfloat16])
def test_split_k_calls_with_guard_bands(M, N, K, ydt):
    # short calls against few weight rows: K is cut over several clusters, the partial sums live in the workspace
    # and a second kernel adds them; guard bands around the workspace and the result, every element against the
    # oracle
    rng = np.random.default_rng(M + 31 * N + 977 * K)
    xb = inputs.to_bf16_bits(rng.standard_t(4, (M, K)).astype(np.float32))
    wb = inputs.to_bf16_bits((0.02 * rng.standard_normal((N, K))).astype(np.float32))
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)),
                          oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    bd.set_gemm_impl(bd.GEMM_TCGEN05)
    esz = 4 if ydt == torch.float32 else 2
    ldy = N + 8
    raw_y, ybytes = _guarded(M * ldy * esz)
    y = ybytes.view(ydt).view(M, ldy)
    y.fill_(-7.0)
    ws_bytes = bd.linear_workspace_size(M, N, K)
    raw_ws, ws = _guarded(ws_bytes)
    before = bd.launch_count()
    bd.linear(to_device(xb, torch.bfloat16), Wq, out=y[:, :N], workspace=ws)
    torch.cuda.synchronize()
    assert bd.launch_count() - before == 3, "expected quantizer, product and the kernel that adds the partial sums"
    assert _intact(raw_y, M * ldy * esz) and _intact(raw_ws, ws_bytes), "write outside a buffer"
    assert (y[:, N:] == -7.0).all(), "write into the padding columns"
    err = np.abs(y[:, :N].float().cpu().numpy().astype(np.float64) - Yref)
    bound = 1e-6 * T + (2.0 ** -8 * np.abs(Yref) if ydt == torch.bfloat16 else 0.0) + 2.0 ** -120
    assert (err <= bound).all(), f"max err / bound = {float((err / bound).max())}"
    bd.poll_status()
