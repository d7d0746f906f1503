"""The allocation-free entry point bd_linear_noalloc, called through the C ABI.

Some callers cannot call cudaMalloc at the point where they need the layer (their
memory plan is frozen, or they were handed only input and output buffers).  For
them the library carries its own fixed scratch array.  This file checks that the
variant gives the same output as bd_linear, twice in a row with different
problems, so that whatever the first call leaves in the shared array cannot leak
into the second, and that a problem beyond the array's size is refused.

Collected last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import gc

import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu


def _problem(M, N, K, seed):
    x = to_device(inputs.act_student_t(M, K, seed=seed), torch.bfloat16)
    w = to_device(inputs.weights_normal(N, K, seed=seed), torch.bfloat16)
    return x, bd.quantize_weights(w, bd.SELECT_TWO_STAGE)


def test_noalloc_matches_linear_on_two_calls_in_a_row():
    cases = [(384, 640, 2048, 11), (130, 257, 352, 12)]        # second one smaller and ragged
    problems = [_problem(*c) for c in cases]
    expected = [bd.linear(x, wq, dtype=torch.float32) for x, wq in problems]
    outs = [torch.empty_like(e) for e in expected]              # outputs allocated before the calls
    gc.collect()                                                # tensors of earlier tests must not be freed in between
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    for (x, wq), out in zip(problems, outs):                    # back to back on one stream
        bd.linear_noalloc(x, wq, out)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before              # the binding allocated nothing either
    for out, exp in zip(outs, expected):
        # same kernels, same operands: equal bit for bit, hence inside every tolerance the suite uses
        assert torch.equal(out, exp)
    bd.poll_status()


def test_noalloc_decode_sized_calls_keep_their_partial_sums_in_the_builtin_array():
    """Short calls against few weight rows cut K over several clusters and park fp32 partial sums in scratch
    between two kernels; a call of fewer than 16 tokens against a small weight matrix takes the CUDA-core
    route, whose scratch holds a packed copy of the activations.  Both run here right after a large call has
    filled the built-in array with other bytes; results must equal bd_linear's bit for bit and the oracle's
    within the product tolerance, and the driver must see no new device allocation."""
    big = _problem(384, 640, 2048, 13)
    cases = [(16, 4096, 11008, 14, torch.float32), (16, 4096, 11008, 14, torch.bfloat16),
             (100, 520, 4128, 15, torch.float32), (5, 300, 224, 16, torch.float32)]
    problems = [(_problem(M, N, K, seed), dt) for M, N, K, seed, dt in cases]
    expected = [bd.linear(x, wq, dtype=dt) for (x, wq), dt in problems]
    outs = [torch.empty_like(e) for e in expected]
    big_out = torch.empty(384, 640, dtype=torch.float32, device="cuda")
    gc.collect()                                                # tensors of earlier tests must not be freed in between
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    allocated_before = torch.cuda.memory_allocated()
    for ((x, wq), dt), out in zip(problems, outs):
        bd.linear_noalloc(big[0], big[1], big_out)              # leaves its own scratch contents behind
        bd.linear_noalloc(x, wq, out)
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == allocated_before
    assert torch.cuda.mem_get_info()[0] == free_before           # nothing came from the driver either
    for out, exp in zip(outs, expected):
        assert torch.equal(out, exp)
    # the decode-sized fp32 result against the oracle
    M, N, K, seed, _ = cases[0]
    xb, wb = inputs.act_student_t(M, K, seed=seed), inputs.weights_normal(N, K, seed=seed)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)),
                          oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    ok, ratio = gemm_tolerance_ok(outs[0].cpu().numpy(), Yref, T)
    assert ok, f"max err / bound = {ratio}"
    bd.poll_status()


def test_noalloc_refuses_problems_beyond_its_scratch():
    M, N, K = 8192, 4096, 14336
    assert bd.linear_workspace_size(M, N, K) > bd.binding.NOALLOC_SCRATCH_BYTES
    x = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda")
    wq = bd.QTensor(N, K)
    out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bd.BdError) as e:
        bd.linear_noalloc(x, wq, out)
    assert e.value.status == 9
