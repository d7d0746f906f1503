"""GPU parity of the quantizers against the CPU oracle: codes, dialect ids and
shared exponents must match bit for bit (through the canonical export)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import assert_bit_exact, oracle_quantize, to_device

pytestmark = pytest.mark.gpu


def test_tiny_case_activations_two_stage_and_weights_mse():
    X, W = inputs.tiny_case()
    qx = bd.quantize_act(to_device(X, torch.float32))
    assert_bit_exact(qx, oracle.quantize(X), "X two-stage")
    qw = bd.quantize_weights(to_device(W, torch.float32), bd.SELECT_MSE)
    assert_bit_exact(qw, oracle.quantize(W, oracle.SELECT_MSE), "W mse")
    qw2 = bd.quantize_weights(to_device(W, torch.float32), bd.SELECT_TWO_STAGE)
    assert_bit_exact(qw2, oracle.quantize(W), "W two-stage")
    bd.poll_status()


def test_activation_bandwidth_workload_full_size():
    # the benchmarked configuration: bf16 [8192, 4096] with 1 % outlier channels
    xb = inputs.act_normal_outliers(8192, 4096, seed=1)
    q = bd.quantize_act(to_device(xb, torch.bfloat16))
    assert_bit_exact(q, oracle_quantize(xb, torch.bfloat16), "config 2")
    bd.poll_status()


@pytest.mark.parametrize("rows,K", [(1, 32), (3, 96), (127, 160), (129, 4096), (300, 352), (16, 11008),
                                    # whole chunks of 64 rows that do not fill a 128-row tile
                                    (64, 256), (192, 128), (320, 512)])
@pytest.mark.parametrize("kind", [torch.float32, torch.bfloat16, torch.float16])
def test_ragged_shapes_and_dtypes(rows, K, kind):
    rng = np.random.default_rng(rows * 7919 + K)
    x = rng.standard_normal((rows, K)).astype(np.float32) * np.exp2(rng.integers(-6, 6, (rows, 1))).astype(np.float32)
    x[:, rng.integers(0, K)] *= 30
    if kind == torch.float32:
        host = x
    elif kind == torch.bfloat16:
        host = inputs.to_bf16_bits(x)
    else:
        host = inputs.to_f16_bits(x)
    q = bd.quantize_act(to_device(host, kind))
    assert_bit_exact(q, oracle_quantize(host, kind), f"{rows}x{K} {kind}")
    qm = bd.quantize_weights(to_device(host, kind), bd.SELECT_MSE)
    assert_bit_exact(qm, oracle_quantize(host, kind, oracle.SELECT_MSE), f"mse {rows}x{K} {kind}")


def test_degenerate_blocks():
    x = np.zeros((8, 64), np.float32)
    x[0, 3] = -0.0                                   # all-zero block with a negative zero
    x[1, :32] = 1e-44; x[1, 5] = -3e-45              # fp32 subnormals: exponent clamp
    x[2, :32] = 2.0 ** -125                          # exponent exactly at the clamp
    x[2, 32:] = 2.0 ** -124 * 1.7
    x[3, :32] = 3.0e38; x[3, 7] = -1.0               # near the top of the fp32 range
    x[4, :] = np.linspace(-7.75, 7.75, 64)           # every quarter step: ties on every boundary
    x[5, :32] = 7.99; x[5, 32:] = 7.75               # block maximum rounding up to 8.0 saturates at 7.5
    x[6, :32] = np.float32(6.74999); x[6, 32:] = 6.75
    x[7, ::2] = 5.0; x[7, 1::2] = -4.0; x[7, 0] = 6.5   # equal beneficial-range counts
    q = bd.quantize_act(to_device(x, torch.float32))
    assert_bit_exact(q, oracle.quantize(x), "degenerate")
    x[3] = np.linspace(-60000, 60000, 64)            # keep the fp16 copy finite
    h = (x * 1e-3).astype(np.float16)
    h[3] = x[3].astype(np.float16)                   # top of the fp16 range
    h[0, :8] = np.float16(6e-8) * np.arange(8)       # fp16 subnormals
    hb = h.view(np.uint16)
    q = bd.quantize_act(to_device(hb, torch.float16))
    assert_bit_exact(q, oracle_quantize(hb, torch.float16), "fp16 subnormal")


def _bf16_clamped_rows():
    """bf16 bit patterns whose blocks sit at and below the exponent clamp (block maximum under 2^-123)."""
    rng = np.random.default_rng(17)
    b = np.zeros((8, 128), np.uint16)
    b[0, 3] = 0x8000                                              # all-zero block with a negative zero
    b[1, :32] = np.arange(32)                                     # the smallest subnormals
    b[1, 32:64] = rng.integers(1, 0x80, 32)                       # any subnormal
    b[1, 64:96] = rng.integers(1, 0x80, 32) | 0x8000              # negative subnormals
    b[2, :32] = 0x0100; b[2, 5] = 0x0033                          # maximum 2^-125 (exponent field 2)
    b[2, 32:64] = rng.integers(0, 0x0180, 32)                     # fields 0..2
    b[3, :64] = rng.integers(0, 0x0200, 64)                       # fields 0..3: the last clamped exponent
    b[3, 64:] = rng.integers(0, 0x0280, 64)                       # field 4: the first regular one
    b[4] = rng.integers(0, 0x0300, 128) | (rng.integers(0, 2, 128) << 15)
    b[5, :32] = 0x01ff; b[5, 32:64] = 0x017f; b[5, 64:96] = 0x00ff; b[5, 96:] = 0x007f   # all-ones mantissas
    b[6, ::2] = 0x0150; b[6, 1::2] = 0x8140; b[6, 0] = 0x0168    # equal beneficial-range counts at the clamp
    b[7] = rng.integers(0, 0x0400, 128) | (rng.integers(0, 2, 128) << 15)
    return b


def test_bf16_blocks_at_the_exponent_clamp():
    b = _bf16_clamped_rows()
    q = bd.quantize_act(to_device(b, torch.bfloat16))
    ref = oracle_quantize(b, torch.bfloat16)
    assert_bit_exact(q, ref, "bf16 clamp")
    # the form bd_linear quantises to (operand bytes) through a product with large weights: 2^-125 x 2^100
    # lands in the normal fp32 range, so the 1e-6 bound is not hidden by the underflow floor
    rng = np.random.default_rng(18)
    W = (rng.standard_normal((96, 128)) * 2.0 ** 100).astype(np.float32)
    Wq = bd.quantize_weights(to_device(W, torch.float32), bd.SELECT_TWO_STAGE)
    Y = bd.linear(to_device(b, torch.bfloat16), Wq, dtype=torch.float32).cpu().numpy()
    Yref, T = oracle.gemm(oracle.dequantize(*ref), oracle.dequantize(*oracle.quantize(W)))
    err = np.abs(Y.astype(np.float64) - Yref)
    assert (err <= 1e-6 * T).all(), float((err / np.maximum(1e-6 * T, 1e-300)).max())
    assert np.abs(Yref).max() > 2.0 ** -40                        # the check above is not vacuous
    bd.poll_status()


@pytest.mark.parametrize("kind", [torch.bfloat16, torch.float32, torch.float16])
def test_random_bit_patterns_every_finite_exponent(kind):
    # inputs drawn as bit patterns, so that every exponent (subnormals and the top of the range included) and every
    # mantissa meets the quantizer; row i keeps its exponents within a window that moves with i, so that blocks
    # at the clamp, blocks of one exponent and blocks spanning many all occur.  Inf and NaN are left out.
    rng = np.random.default_rng(23)
    rows, K = 192, 256
    if kind == torch.float32:
        ebits, mbits, word = 8, 23, np.uint32
    elif kind == torch.bfloat16:
        ebits, mbits, word = 8, 7, np.uint16
    else:
        ebits, mbits, word = 5, 10, np.uint16
    top = (1 << ebits) - 1                                        # the exponent field of Inf / NaN
    lo = (np.arange(rows) * (top - 1) // rows)[:, None]           # window start per row
    width = rng.integers(1, 12, (rows, 1))
    lo[:8, 0] = [0, 0, 0, 1, 0, 1, 0, 2]                          # the first rows sit at and below the exponent clamp
    width[:8, 0] = [1, 2, 3, 2, 4, 3, 5, 1]
    exp = np.minimum(lo + rng.integers(0, 1 << 30, (rows, K)) % width, top - 1)
    man = rng.integers(0, 1 << mbits, (rows, K))
    sign = rng.integers(0, 2, (rows, K))
    bits = ((sign << (ebits + mbits)) | (exp << mbits) | man).astype(word)
    host = bits.view(np.float32) if kind == torch.float32 else bits
    q = bd.quantize_act(to_device(host, kind))
    assert_bit_exact(q, oracle_quantize(host, kind), f"bit patterns {kind}")
    bd.poll_status()


def test_leading_dimension_and_output_guard_bands():
    rng = np.random.default_rng(5)
    big = rng.standard_normal((40, 512)).astype(np.float32)
    xd = to_device(inputs.to_bf16_bits(big), torch.bfloat16)
    view = xd[:, 128:128 + 256]                      # ld = 512 > K = 256, 16-byte aligned start
    q = bd.QTensor(40, 256)
    guard = 4096
    bufs = {}
    for name in ("codes", "ids", "scales"):          # place each buffer between pattern-filled guards
        n = getattr(q, name).numel()
        raw = torch.full((n + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
        bufs[name] = raw
        setattr(q, name, raw[guard:guard + n])
    bd.quantize_act(view, out=q)
    ref = oracle_quantize(inputs.to_bf16_bits(big[:, 128:384]), torch.bfloat16)
    assert_bit_exact(q, ref, "strided rows")
    for name, raw in bufs.items():
        n = raw.numel() - 2 * guard
        assert (raw[:guard] == 0xA5).all() and (raw[guard + n:] == 0xA5).all(), f"{name}: write outside the buffer"


@pytest.mark.parametrize("kind", [torch.bfloat16, torch.float32])
def test_strided_axis_quantizes_the_transpose(kind):
    # V [tokens, head_dim] quantised along tokens: result equals quantising V^T along its rows
    rng = np.random.default_rng(9)
    v = rng.standard_normal((320, 128)).astype(np.float32)
    host = v if kind == torch.float32 else inputs.to_bf16_bits(v)
    q = bd.quantize_act(to_device(host, kind), axis=bd.AXIS_STRIDED)
    assert (q.rows, q.K) == (128, 320)
    ref = oracle_quantize(np.ascontiguousarray(host.T), kind)
    assert_bit_exact(q, ref, "strided axis")


def test_nonfinite_input_sets_status():
    x = torch.ones(4, 64, device="cuda")
    x[2, 40] = float("inf")
    bd.quantize_act(x)
    with pytest.raises(bd.BdError) as e:
        bd.poll_status()
    assert e.value.status == 6
    bd.poll_status()                                 # the word is cleared by the read


def test_import_export_roundtrip_and_dequantize():
    X, _ = inputs.tiny_case()
    ref = oracle.quantize(X)
    q = bd.import_canonical(*(torch.from_numpy(t).cuda() for t in ref))
    assert_bit_exact(q, ref, "import")
    dq = bd.dequantize(q).cpu().numpy().astype(np.float64)
    assert (dq == oracle.dequantize(*ref)).all()
    assert (np.signbit(dq) == np.signbit(oracle.dequantize(*ref))).all()
