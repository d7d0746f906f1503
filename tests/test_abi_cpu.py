"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol,
and its host-only entry points behave.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np

import oracle
import paper_2501_01144_b200 as bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "bd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bd_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = bd.load()
    names = _declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), f"{name} declared in include/bd.h but not exported"


def test_version_and_status_strings():
    lib = bd.load()
    assert bd.version() >= 100
    for code in range(10):
        assert lib.bd_status_string(code)
    assert lib.bd_status_string(0) == b"ok"


def test_formatbook_matches_independent_oracle_table():
    # the CUDA library and the oracle each carry their own copy of the table
    assert (bd.get_formatbook().numpy() == oracle.formatbook()).all()


def test_set_formatbook_rejects_tables_without_the_pair_structure():
    # validation is host arithmetic and comes before any device call; accepted tables are a GPU test
    lib = bd.load()
    good = bd.get_formatbook().numpy().copy()

    def rc(table):
        buf = (ctypes.c_uint8 * 128)(*[int(v) for v in table.reshape(-1)])
        return lib.bd_set_formatbook(buf)

    t = good.copy(); t[3, 4] = t[3, 3]                       # a row that is not strictly ascending
    assert rc(t) == 1
    t = good.copy(); t[6, 7] = 13; t[7, 7] = 13              # pair 3 must have maximum 15 - 3
    assert rc(t) == 1
    t = good.copy(); t[2, 6], t[3, 6] = good[3, 6], good[2, 6]   # the even member must hold the larger value
    assert rc(t) == 1
    t = good.copy(); t[8, 2] = 3; t[8, 3] = 4; t[8, 4] = 5   # members of a pair may differ at index 6 only
    assert rc(t) == 1
    t = good.copy(); t[0, 0] = 1                             # every dialect contains zero
    assert rc(t) == 1
    assert (bd.get_formatbook().numpy() == good).all()       # nothing changed


def test_qtensor_sizes_and_argument_errors():
    lib = bd.load()
    c, i, s = (ctypes.c_size_t() for _ in range(3))
    assert lib.bd_qtensor_sizes(8192, 4096, ctypes.byref(c), ctypes.byref(i), ctypes.byref(s)) == 0
    assert c.value == 8192 * 4096 // 2
    assert i.value == 8192 * 4096 // 32 // 2          # 4 bits per block
    assert s.value == 8192 * 4096 // 32               # 8 bits per block
    # ragged shapes are padded to whole 128-row x 4-block atoms
    assert lib.bd_qtensor_sizes(130, 96, ctypes.byref(c), ctypes.byref(i), ctypes.byref(s)) == 0
    assert c.value == 130 * 48 and s.value == 2 * 1 * 512 and i.value == 2 * 1 * 256
    assert lib.bd_qtensor_sizes(16, 100, None, None, None) == 2      # K % 32
    assert lib.bd_qtensor_sizes(0, 64, None, None, None) == 1
    b = ctypes.c_size_t()
    assert lib.bd_linear_workspace_size(16, 128, 100, ctypes.byref(b)) == 2
    assert lib.bd_gemm_workspace_size(16, 128, 256, None) == 1
    assert lib.bd_set_gemm_impl(7) == 1 and lib.bd_set_gemm_impl(0) == 0


def test_workspace_sizes_follow_the_documented_parts():
    """Host arithmetic only: the operand bytes of the activations, their scale atoms, and for short calls
    against few weight rows the fp32 partial sums of a K split."""
    lib = bd.load()
    b = ctypes.c_size_t()

    def linear_ws(M, N, K):
        assert lib.bd_linear_workspace_size(M, N, K, ctypes.byref(b)) == 0
        return b.value

    def gemm_ws(M, N, K):
        assert lib.bd_gemm_workspace_size(M, N, K, ctypes.byref(b)) == 0
        return b.value

    atoms = lambda M, K: ((M + 127) // 128) * ((K // 32 + 3) // 4) * 512
    # at most 16 rows on the activation side: never less than the warp-level kernel's records (K rounded up to 128,
    # two groups of 8 rows, 32 fp16 values and one fp32 factor per row and block)
    records = lambda K: ((K + 127) // 128 * 4) * 2 * (8 * 32 * 2 + 8 * 4)
    # the benchmark's layers: operand bytes + scale atoms, nothing else
    assert gemm_ws(2048, 14336, 4096) == 2048 * 4096
    assert linear_ws(2048, 14336, 4096) == atoms(2048, 4096) + 2048 * 4096
    # up to 128 tokens against at most 37 pairs of 128 weight rows (half of the clusters): room for four splits of
    # [tokens rounded to 16][weight rows rounded to 256] fp32 partial sums behind the operand bytes
    assert gemm_ws(16, 4096, 11008) == 16 * 11008 + 4 * 16 * 4096 * 4 > records(11008)
    assert gemm_ws(5, 300, 2144) == 256 * ((5 * 2144 + 255) // 256) + 4 * 16 * 512 * 4 > records(2144)
    assert gemm_ws(128, 9472, 4096) == 128 * 4096 + 4 * 128 * 9472 * 4
    # more weight rows than that, or more tokens: no split, no scratch
    assert gemm_ws(16, 11008, 4096) == records(4096) > 16 * 4096
    assert gemm_ws(17, 11008, 4096) == 17 * 4096
    assert gemm_ws(128, 9473, 4096) == 128 * 4096
    assert gemm_ws(129, 4096, 11008) == 256 * ((129 * 11008 + 255) // 256)


def test_null_and_misaligned_arguments_rejected_before_any_launch():
    lib = bd.load()
    q = bd.binding._CQTensor(0, 0, 0, 16, 64)
    assert lib.bd_quantize_act(None, bd.BF16, 16, 64, 64, 0, ctypes.byref(q), None) == 1
    buf = np.zeros(4096, np.uint8)
    base = buf.ctypes.data + (-buf.ctypes.data % 16)          # host memory: only the checks run
    q = bd.binding._CQTensor(base, base + 1024, base + 2048, 16, 64)
    assert lib.bd_quantize_act(ctypes.c_void_p(base + 4), bd.BF16, 16, 64, 64, 0, ctypes.byref(q), None) == 3
    assert lib.bd_quantize_act(ctypes.c_void_p(base), bd.BF16, 16, 64, 60, 0, ctypes.byref(q), None) == 2
    assert lib.bd_quantize_act(ctypes.c_void_p(base), 9, 16, 64, 64, 0, ctypes.byref(q), None) == 1
    q2 = bd.binding._CQTensor(base, base + 1024, base + 2048, 8, 64)
    assert lib.bd_quantize_act(ctypes.c_void_p(base), bd.BF16, 16, 64, 64, 0, ctypes.byref(q2), None) == 2
    qa = bd.binding._CQTensor(base, base + 1024, base + 2048, 16, 64)
    qb = bd.binding._CQTensor(base, base + 1024, base + 2048, 16, 96)
    assert lib.bd_gemm(ctypes.byref(qa), ctypes.byref(qb), ctypes.c_void_p(base), bd.F32, 16, None, 0, None) == 2
    assert lib.bd_gemm(ctypes.byref(qa), ctypes.byref(qa), ctypes.c_void_p(base), bd.F16, 16, None, 0, None) == 1


def test_batched_product_rejects_operands_of_different_shapes():
    # argument checks come before any launch, so made-up (aligned, non-null) addresses are enough here
    lib = bd.load()
    Q = bd.binding._CQTensor
    a = (Q * 2)(Q(0x1000, 0x2000, 0x3000, 128, 128), Q(0x1000, 0x2000, 0x3000, 64, 128))
    b = (Q * 1)(Q(0x1000, 0x2000, 0x3000, 256, 128))
    rc = lib.bd_gemm_batched(a, b, 2, 2, ctypes.c_void_p(0x4000), 0, 256, 128 * 256, None, 0, None)
    assert rc == 2                                            # BD_ERR_SHAPE: A[1] is shorter than A[0]
