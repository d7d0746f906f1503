"""BlockDialect CPU oracle: ctypes binding of ``bd_oracle.c`` (test infrastructure).

Only tests, the smoke check and the benchmark's CPU-baseline / reference arm may
import this package.  It shares nothing with the CUDA library: its own C file,
its own table, its own build.  Arrays go in and out as numpy; 16-bit inputs are
passed as ``uint16`` bit patterns.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bd_oracle.c")
_LIB = os.path.join(_HERE, "libbd_oracle.so")

F32, BF16, F16 = 0, 1, 2
SELECT_TWO_STAGE, SELECT_MSE = 0, 1
BLOCK = 32

_lib = None


def build(force=False):
    """Compile the oracle with gcc (fp contraction off, so sums keep the written order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        _lib.bdo_quantize.argtypes = [vp, ci, i64, i64, i64, ci, vp, vp, vp]
        _lib.bdo_quantize_bs.argtypes = [vp, ci, i64, i64, i64, ci, ci, vp, vp, vp]
        _lib.bdo_dequantize_bs.argtypes = [vp, vp, vp, i64, i64, ci, vp]
        _lib.bdo_gemm_blockmac_bs.argtypes = [vp] * 6 + [i64] * 3 + [ci, vp]
        _lib.bdo_dequantize.argtypes = [vp, vp, vp, i64, i64, vp]
        _lib.bdo_gemm.argtypes = [vp, vp, i64, i64, i64, vp, vp]
        _lib.bdo_gemm_blockmac.argtypes = [vp] * 6 + [i64] * 3 + [vp]
        _lib.bdo_beneficial_range.argtypes = [ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
        _lib.bdo_round_code.argtypes = [ci, ci]
        _lib.bdo_formatbook.argtypes = [vp]
        _lib.bdo_set_formatbook.argtypes = [vp]
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def threads():
    return int(lib().bdo_threads())


def formatbook():
    """The 16 x 8 DialectFP4 table in half-units (Sec. 3.1, Fig. 4)."""
    out = np.zeros((16, 8), np.uint8)
    lib().bdo_formatbook(_ptr(out))
    return out


def set_formatbook(table=None):
    """Replace the table in use (None restores the reconstruction of Fig. 4).  Raises on a table without
    the pair structure of Sec. 3.1 / 3.2."""
    if table is None:
        rc = lib().bdo_set_formatbook(None)
    else:
        t = np.ascontiguousarray(np.asarray(table, np.uint8).reshape(16, 8))
        rc = lib().bdo_set_formatbook(_ptr(t))
    if rc:
        raise ValueError("formatbook rejected")


def beneficial_range(dialect):
    """[lo, hi) of a dialect's beneficial range on the 5-bit code (Sec. 3.2, Fig. 5c)."""
    lo, hi = ctypes.c_int(), ctypes.c_int()
    if lib().bdo_beneficial_range(dialect, ctypes.byref(lo), ctypes.byref(hi)):
        raise ValueError("bad dialect")
    return lo.value, hi.value


def round_code(dialect, q5):
    """Index of the dialect value nearest to a 5-bit code, ties to the larger (Sec. 3.3)."""
    return int(lib().bdo_round_code(dialect, q5))


def _dtype_of(x):
    if x.dtype == np.float32:
        return F32
    if x.dtype == np.uint16:
        raise TypeError("16-bit input: pass dtype=BF16 or F16 explicitly")
    raise TypeError(f"unsupported input dtype {x.dtype}")


def quantize(x, select=SELECT_TWO_STAGE, dtype=None, block=BLOCK):
    """Quantise a [rows, K] array along K in blocks of `block` elements (32 unless the block-size study of
    Sec. 4.2 / Table 3 is meant: 16 or 64).  Returns canonical (codes, ids, scales)."""
    x = np.ascontiguousarray(x)
    if dtype is None:
        dtype = _dtype_of(x)
    rows, K = x.shape
    codes = np.zeros((rows, K // 2), np.uint8)
    ids = np.zeros((rows, K // block), np.uint8)
    scales = np.zeros((rows, K // block), np.uint8)
    st = lib().bdo_quantize_bs(_ptr(x), dtype, rows, K, K, select, block, _ptr(codes), _ptr(ids), _ptr(scales))
    if st == 2:
        raise FloatingPointError("non-finite input")
    if st:
        raise ValueError("bad arguments")
    return codes, ids, scales


def requantize(y):
    """A product's fp32 result [M, N] back into DialectFP4 for the next product (Sec. 3.3, last paragraph: the
    accumulated sums are requantised "for the next matrix multiplication").  The paper defines no separate
    arithmetic for this step: it is the online two-stage rule applied to the result's rows, blocks of 32 along N."""
    y = np.ascontiguousarray(y)
    if y.dtype != np.float32:
        raise TypeError("requantize takes the fp32 result")
    return quantize(y, SELECT_TWO_STAGE)


def dequantize(codes, ids, scales):
    """Canonical (codes, ids, scales) -> fp64 [rows, K] (Sec. 3.3, Fig. 6); the block size follows from the
    shapes (K / number of ids per row)."""
    rows, K = codes.shape[0], codes.shape[1] * 2
    block = K // ids.shape[1]
    out = np.zeros((rows, K), np.float64)
    if lib().bdo_dequantize_bs(_ptr(np.ascontiguousarray(codes)), _ptr(np.ascontiguousarray(ids)),
                               _ptr(np.ascontiguousarray(scales)), rows, K, block, _ptr(out)):
        raise ValueError("bad arguments")
    return out


def gemm(a, b):
    """Y = a @ b.T in fp64 plus T = |a| @ |b|.T, for dequantised a [M,K], b [N,K]."""
    a = np.ascontiguousarray(a, np.float64)
    b = np.ascontiguousarray(b, np.float64)
    M, K = a.shape
    N = b.shape[0]
    assert b.shape[1] == K
    Y = np.zeros((M, N), np.float64)
    T = np.zeros((M, N), np.float64)
    lib().bdo_gemm(_ptr(a), _ptr(b), M, N, K, _ptr(Y), _ptr(T))
    return Y, T


def gemm_blockmac(qa, qb):
    """The paper's block MAC (integer in-block sums, one rescale per block) on canonical operands."""
    ca, ia, sa = (np.ascontiguousarray(t) for t in qa)
    cb, ib, sb = (np.ascontiguousarray(t) for t in qb)
    M, K = ca.shape[0], ca.shape[1] * 2
    N = cb.shape[0]
    block = K // ia.shape[1]
    assert K // ib.shape[1] == block, "both operands of a product use one block size"
    Y = np.zeros((M, N), np.float64)
    if lib().bdo_gemm_blockmac_bs(_ptr(ca), _ptr(ia), _ptr(sa), _ptr(cb), _ptr(ib), _ptr(sb), M, N, K, block, _ptr(Y)):
        raise ValueError("bad arguments")
    return Y
