"""A bounded device-side wait that runs out: the kernel records BD_ERR_TIMEOUT, drains and returns, nothing is
written, and the next call on the same stream is served normally.  The wait is made to run out on the host side of
the kernel's own protocol (one copy is never started, so nothing is in flight into the CTA); no trap, no endless
loop, one launch on a one-cluster problem."""
import numpy as np
import pytest
import torch

import oracle
import paper_2501_01144_b200 as bd
from paper_2501_01144_b200 import inputs
from util import gemm_tolerance_ok, to_device

pytestmark = pytest.mark.gpu


def test_a_wait_that_runs_out_reports_timeout_and_the_library_stays_usable():
    M, N, K = 256, 256, 256                                   # one tile: one cluster of two CTAs, two k-steps
    xb = inputs.act_student_t(M, K, seed=31)
    wb = inputs.weights_normal(N, K, seed=31)
    xd = to_device(xb, torch.bfloat16)
    Wq = bd.quantize_weights(to_device(wb, torch.bfloat16), bd.SELECT_TWO_STAGE)
    bd.set_gemm_impl(bd.GEMM_TCGEN05)
    good = bd.linear(xd, Wq, dtype=torch.float32)
    bd.poll_status()
    try:
        bd.debug_fault(poll_limit=10 * 1024, skip_first_code_stage=True)
        y = torch.full((M, N), -7.0, dtype=torch.float32, device="cuda")
        bd.linear(xd, Wq, out=y)
        with pytest.raises(bd.BdError) as e:
            bd.poll_status()
        assert e.value.status == 7                            # BD_ERR_TIMEOUT
        assert bool((y == -7.0).all()), "an aborted product must not write results"
    finally:
        bd.debug_fault(0, False)
        bd.set_gemm_impl(bd.GEMM_AUTO)
    bd.poll_status()                                          # the status word was cleared by the poll above
    again = bd.linear(xd, Wq, dtype=torch.float32)            # same stream, same context: served normally
    assert torch.equal(again, good)
    Yref, T = oracle.gemm(oracle.dequantize(*oracle.quantize(xb, dtype=oracle.BF16)),
                          oracle.dequantize(*oracle.quantize(wb, dtype=oracle.BF16)))
    ok, ratio = gemm_tolerance_ok(again.cpu().numpy(), Yref, T)
    assert ok, f"max err / bound = {ratio}"
    bd.poll_status()
