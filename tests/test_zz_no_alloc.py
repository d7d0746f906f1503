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
import numpy as np
import pytest
import torch

import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import to_device

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


def test_noalloc_refuses_problems_beyond_its_scratch():
    M, N, K = 8192, 4096, 14336
    assert bd.linear_workspace_size(M, N, K) > bd.binding.NOALLOC_SCRATCH_BYTES
    x = torch.zeros(M, K, dtype=torch.bfloat16, device="cuda")
    wq = bd.QTensor(N, K)
    out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bd.BdError) as e:
        bd.linear_noalloc(x, wq, out)
    assert e.value.status == 9
