"""Helpers shared by the GPU parity tests: moving seeded inputs to the device and
comparing the library's canonical export with the oracle's output."""
import numpy as np
import torch

import oracle
import paper_2501_01144_b200 as bd

ORACLE_DTYPE = {torch.float32: oracle.F32, torch.bfloat16: oracle.BF16, torch.float16: oracle.F16}


def to_device(arr, kind):
    """numpy float32 array or uint16 bit patterns -> CUDA tensor of `kind` holding the same bytes."""
    if kind == torch.float32:
        return torch.from_numpy(np.ascontiguousarray(arr, np.float32)).cuda()
    return torch.from_numpy(np.ascontiguousarray(arr, np.uint16).view(np.int16)).cuda().view(kind)


def oracle_quantize(arr, kind, select=oracle.SELECT_TWO_STAGE):
    return oracle.quantize(arr, select, dtype=ORACLE_DTYPE[kind])


def assert_bit_exact(q, ref, what=""):
    codes, ids, scales = (t.cpu().numpy() for t in bd.export_canonical(q))
    rc, ri, rs = ref
    assert codes.shape == rc.shape and ids.shape == ri.shape and scales.shape == rs.shape
    bad_s = np.argwhere(scales != rs)
    assert bad_s.size == 0, f"{what}: {len(bad_s)} scale mismatches, first at {bad_s[0]}: {scales[tuple(bad_s[0])]} vs {rs[tuple(bad_s[0])]}"
    bad_i = np.argwhere(ids != ri)
    assert bad_i.size == 0, f"{what}: {len(bad_i)} id mismatches, first at {bad_i[0]}: {ids[tuple(bad_i[0])]} vs {ri[tuple(bad_i[0])]}"
    bad_c = np.argwhere(codes != rc)
    assert bad_c.size == 0, f"{what}: {len(bad_c)} code-byte mismatches, first at {bad_c[0]}"


def gemm_tolerance_ok(Y, Yref, T, rel=1e-6, floor=2.0 ** -120):
    """|Y - Yref| <= rel * sum_k |a_k||w_k| elementwise (plus an underflow floor)."""
    err = np.abs(np.asarray(Y, np.float64) - Yref)
    bound = rel * T + floor
    ratio = float((err / bound).max())
    return ratio <= 1.0, ratio
