"""ctypes binding of the C ABI in include/bd.h (same names without the bd_ prefix)."""
import ctypes
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libblockdialect.so")
_SRC = os.path.join(_HERE, "csrc", "bd_lib.cu")

F32, BF16, F16 = 0, 1, 2
SELECT_TWO_STAGE, SELECT_MSE = 0, 1
AXIS_CONTIG, AXIS_STRIDED = 0, 1
GEMM_AUTO, GEMM_SIMT, GEMM_TCGEN05, GEMM_WARP = 0, 1, 2, 3

_TORCH_DTYPE = {torch.float32: F32, torch.bfloat16: BF16, torch.float16: F16}

_lib = None


class BdError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"libblockdialect: status {status}: {text}")
        self.status = status


class _CQTensor(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("ids", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("rows", ctypes.c_int64), ("K", ctypes.c_int64)]


class _CAttentionDump(ctypes.Structure):
    _fields_ = [("S", ctypes.c_void_p), ("P", ctypes.c_void_p), ("codes", ctypes.c_void_p), ("ids", ctypes.c_void_p),
                ("scales", ctypes.c_void_p)]


class _CKVCache(ctypes.Structure):
    _fields_ = [("k", _CQTensor), ("v", _CQTensor), ("v_recent", ctypes.c_void_p), ("dtype", ctypes.c_int),
                ("capacity", ctypes.c_int64), ("head_dim", ctypes.c_int64), ("length", ctypes.c_int64)]


def library_path():
    return _LIB_PATH


def build(verbose=False):
    """Compile the CUDA library in-tree for sm_100a."""
    srcs = [os.path.join(_HERE, "csrc", f) for f in os.listdir(os.path.join(_HERE, "csrc"))]
    if os.path.exists(_LIB_PATH) and all(os.path.getmtime(_LIB_PATH) >= os.path.getmtime(s) for s in srcs):
        return _LIB_PATH
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-o", _LIB_PATH, _SRC]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return _LIB_PATH


def load():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise BdError(-1, f"{_LIB_PATH} is missing: run __graft_entry__.build() (nvcc, sm_100a) first")
    lib = ctypes.CDLL(_LIB_PATH)
    i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    qp = ctypes.POINTER(_CQTensor)
    szp = ctypes.POINTER(sz)
    lib.bd_qtensor_sizes.argtypes = [i64, i64, szp, szp, szp]
    lib.bd_quantize_weights.argtypes = [vp, ci, i64, i64, i64, ci, qp, vp]
    lib.bd_quantize_act.argtypes = [vp, ci, i64, i64, i64, ci, qp, vp]
    lib.bd_gemm_workspace_size.argtypes = [i64, i64, i64, szp]
    lib.bd_gemm.argtypes = [qp, qp, vp, ci, i64, vp, sz, vp]
    lib.bd_gemm_batched_workspace_size.argtypes = [i64, i64, i64, i64, szp]
    lib.bd_gemm_batched.argtypes = [qp, qp, i64, i64, vp, ci, i64, i64, vp, sz, vp]
    lib.bd_linear_workspace_size.argtypes = [i64, i64, i64, szp]
    lib.bd_linear.argtypes = [vp, ci, i64, i64, i64, qp, vp, ci, i64, vp, sz, vp]
    lib.bd_linear_noalloc.argtypes = [vp, ci, i64, i64, i64, qp, vp, ci, i64, vp]
    kp = ctypes.POINTER(_CKVCache)
    lib.bd_kvcache_recent_bytes.argtypes = [i64, ci, szp]
    lib.bd_kvcache_reset.argtypes = [kp, vp]
    lib.bd_kvcache_append.argtypes = [kp, vp, vp, i64, i64, i64, vp]
    lib.bd_kvcache_workspace_size.argtypes = [i64, i64, i64, szp]
    lib.bd_kvcache_scores.argtypes = [kp, qp, vp, ci, i64, vp, sz, vp]
    lib.bd_kvcache_pv.argtypes = [kp, vp, i64, i64, vp, ci, i64, vp, sz, vp]
    lib.bd_kvcache_append_batched.argtypes = [kp, i64, vp, vp, i64, i64, i64, i64, i64, vp]
    lib.bd_kvcache_batched_workspace_size.argtypes = [i64, i64, i64, i64, szp]
    lib.bd_kvcache_attention_workspace_size.argtypes = [i64, i64, i64, i64, szp]
    lib.bd_kvcache_attention.argtypes = [kp, i64, qp, ctypes.c_float, vp, ci, i64, i64, vp, i64, i64, vp, sz, vp]
    lib.bd_kvcache_scores_batched.argtypes = [kp, i64, qp, vp, ci, i64, i64, vp, sz, vp]
    lib.bd_kvcache_pv_batched.argtypes = [kp, i64, vp, i64, i64, i64, vp, ci, i64, i64, vp, sz, vp]
    lib.bd_attention_workspace_size.argtypes = [i64, i64, i64, i64, szp]
    lib.bd_attention.argtypes = [qp, qp, qp, i64, i64, ctypes.c_float, vp, ci, i64, i64, ctypes.POINTER(_CAttentionDump), vp, sz, vp]
    lib.bd_qtensor_sizes_bs.argtypes = [i64, i64, ci, szp, szp, szp]
    lib.bd_quantize_bs.argtypes = [vp, ci, i64, i64, i64, ci, ci, qp, vp]
    lib.bd_export_canonical_bs.argtypes = [qp, ci, vp, vp, vp, vp]
    lib.bd_linear_bs_workspace_size.argtypes = [i64, i64, i64, ci, szp]
    lib.bd_linear_bs.argtypes = [vp, ci, i64, i64, i64, ci, qp, vp, ci, i64, vp, sz, vp]
    lib.bd_linear_requant_workspace_size.argtypes = [i64, i64, i64, szp]
    lib.bd_linear_requant.argtypes = [vp, ci, i64, i64, i64, qp, qp, vp, sz, vp]
    lib.bd_gemm_requant_workspace_size.argtypes = [i64, i64, i64, szp]
    lib.bd_gemm_requant.argtypes = [qp, qp, qp, vp, sz, vp]
    lib.bd_export_canonical.argtypes = [qp, vp, vp, vp, vp]
    lib.bd_import_canonical.argtypes = [vp, vp, vp, qp, vp]
    lib.bd_dequantize.argtypes = [qp, vp, i64, vp]
    lib.bd_get_formatbook.argtypes = [vp]
    lib.bd_set_formatbook.argtypes = [vp]
    lib.bd_poll_status.argtypes = [vp]
    lib.bd_set_gemm_impl.argtypes = [ci]
    lib.bd_debug_fault.argtypes = [ctypes.c_uint32, ci]
    lib.bd_launch_count.restype = ctypes.c_uint64
    lib.bd_status_string.argtypes = [ci]
    lib.bd_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _check(status):
    if status:
        lib = load()
        text = lib.bd_status_string(status).decode()
        if status == 5:
            text += f" (cuda error {lib.bd_last_cuda_error()})"
        raise BdError(status, text)


def _stream(stream=None):
    if stream is None:
        return ctypes.c_void_p(torch._C._cuda_getCurrentRawStream(torch.cuda.current_device()))
    return ctypes.c_void_p(stream.cuda_stream)


def version():
    return load().bd_version()


def launch_count():
    """Kernels launched by the library so far in this process."""
    return int(load().bd_launch_count())


def debug_fault(poll_limit=0, skip_first_code_stage=False):
    """Test hook: shorten the bounded device-side waits and make one of them run out (see bd.h)."""
    _check(load().bd_debug_fault(ctypes.c_uint32(poll_limit), 1 if skip_first_code_stage else 0))


def set_gemm_impl(impl):
    _check(load().bd_set_gemm_impl(impl))


def get_formatbook():
    """The DialectFP4 table, 16 x 8, magnitudes in units of 0.5 (Sec. 3.1, Fig. 4)."""
    buf = (ctypes.c_uint8 * 128)()
    _check(load().bd_get_formatbook(buf))
    return torch.tensor(list(buf), dtype=torch.uint8).reshape(16, 8)


def set_formatbook(table=None):
    """Replace the DialectFP4 table on the current device (None restores the built-in one)."""
    if table is None:
        _check(load().bd_set_formatbook(None))
        return
    vals = [int(v) for v in torch.as_tensor(table).reshape(-1).tolist()]
    if len(vals) != 128:
        raise ValueError("formatbook must be 16 x 8")
    buf = (ctypes.c_uint8 * 128)(*vals)
    _check(load().bd_set_formatbook(buf))


def poll_status(stream=None):
    """Synchronise the stream and raise if a kernel recorded a device-side condition."""
    _check(load().bd_poll_status(_stream(stream)))


class QTensor:
    """A quantised [rows, K] operand: three device byte buffers in the library's layout."""

    def __init__(self, rows, K, device="cuda"):
        c, i, s = (ctypes.c_size_t() for _ in range(3))
        _check(load().bd_qtensor_sizes(rows, K, ctypes.byref(c), ctypes.byref(i), ctypes.byref(s)))
        self.rows, self.K = rows, K
        self.codes = torch.empty(c.value, dtype=torch.uint8, device=device)
        self.ids = torch.empty(i.value, dtype=torch.uint8, device=device)
        self.scales = torch.empty(s.value, dtype=torch.uint8, device=device)

    def __setattr__(self, name, value):
        object.__setattr__(self, name, value)
        object.__setattr__(self, "_c", None)                      # a buffer or a shape changed: the descriptor is rebuilt

    def c_struct(self):
        """The C descriptor (kept until a member changes: a decode step passes dozens of these per call)."""
        if self._c is None:
            object.__setattr__(self, "_c", _CQTensor(self.codes.data_ptr(), self.ids.data_ptr(), self.scales.data_ptr(), self.rows, self.K))
        return self._c

    def nbytes(self):
        return self.codes.numel() + self.ids.numel() + self.scales.numel()


def _src(x):
    if x.dtype not in _TORCH_DTYPE or x.dim() != 2 or x.stride(1) != 1 or not x.is_cuda:
        raise ValueError("source must be a 2-D CUDA tensor of fp32/bf16/fp16 with a contiguous last axis")
    return ctypes.c_void_p(x.data_ptr()), _TORCH_DTYPE[x.dtype], x.stride(0)


def quantize_weights(W, select=SELECT_MSE, out=None, stream=None):
    """Offline weight quantisation of W [N, K] along K (Sec. 3.3)."""
    ptr, dt, ld = _src(W)
    N, K = W.shape
    out = out or QTensor(N, K, W.device)
    cq = out.c_struct()
    _check(load().bd_quantize_weights(ptr, dt, N, K, ld, select, ctypes.byref(cq), _stream(stream)))
    return out


def quantize_act(X, axis=AXIS_CONTIG, out=None, stream=None):
    """Online two-stage quantisation (Sec. 3.2).  AXIS_CONTIG: X [M, K]; AXIS_STRIDED: X [K, M]."""
    ptr, dt, ld = _src(X)
    M, K = X.shape if axis == AXIS_CONTIG else (X.shape[1], X.shape[0])
    out = out or QTensor(M, K, X.device)
    cq = out.c_struct()
    _check(load().bd_quantize_act(ptr, dt, M, K, ld, axis, ctypes.byref(cq), _stream(stream)))
    return out


def gemm_workspace_size(M, N, K):
    b = ctypes.c_size_t()
    _check(load().bd_gemm_workspace_size(M, N, K, ctypes.byref(b)))
    return b.value


def linear_workspace_size(M, N, K):
    b = ctypes.c_size_t()
    _check(load().bd_linear_workspace_size(M, N, K, ctypes.byref(b)))
    return b.value


def _ydtype(dtype):
    if dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("output dtype must be float32 or bfloat16")
    return _TORCH_DTYPE[dtype]


def _ws(workspace, need, device):
    """`need` may be a callable: the size query is skipped when the caller brings a workspace."""
    if workspace is None:
        need = need() if callable(need) else need
        if need:
            workspace = torch.empty(need, dtype=torch.uint8, device=device)
    ptr = ctypes.c_void_p(workspace.data_ptr() if workspace is not None else 0)
    return workspace, ptr, (workspace.numel() if workspace is not None else 0)


def gemm(A, B, out=None, dtype=torch.float32, workspace=None, stream=None):
    """Y [M, N] = dq(A) dq(B)^T (Sec. 3.3, Fig. 6)."""
    if out is None:
        out = torch.empty(A.rows, B.rows, dtype=dtype, device=A.codes.device)
    workspace, wptr, wbytes = _ws(workspace, lambda: gemm_workspace_size(A.rows, B.rows, A.K), A.codes.device)
    ca, cb = A.c_struct(), B.c_struct()
    _check(load().bd_gemm(ctypes.byref(ca), ctypes.byref(cb), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                          out.stride(0), wptr, wbytes, _stream(stream)))
    return out


def gemm_batched_workspace_size(M, N, K, b_group):
    b = ctypes.c_size_t()
    _check(load().bd_gemm_batched_workspace_size(M, N, K, b_group, ctypes.byref(b)))
    return b.value


def gemm_batched(As, Bs, b_group=1, out=None, dtype=torch.float32, workspace=None, stream=None):
    """Batched product; A[b] pairs with B[b // b_group] (grouped-query attention)."""
    batch = len(As)
    M, N, K = As[0].rows, Bs[0].rows, As[0].K
    if out is None:
        out = torch.empty(batch, M, N, dtype=dtype, device=As[0].codes.device)
    workspace, wptr, wbytes = _ws(workspace, gemm_batched_workspace_size(M, N, K, b_group), As[0].codes.device)
    ca = (_CQTensor * batch)(*[a.c_struct() for a in As])
    cb = (_CQTensor * len(Bs))(*[b.c_struct() for b in Bs])
    _check(load().bd_gemm_batched(ca, cb, batch, b_group, ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                                  out.stride(1), out.stride(0), wptr, wbytes, _stream(stream)))
    return out


def linear(X, Wq, out=None, dtype=torch.bfloat16, workspace=None, stream=None):
    """The quantised linear layer: two-stage quantisation of X [M, K], then the product with Wq [N, K]."""
    ptr, dt, ld = _src(X)
    M, K = X.shape
    if out is None:
        out = torch.empty(M, Wq.rows, dtype=dtype, device=X.device)
    workspace, wptr, wbytes = _ws(workspace, lambda: linear_workspace_size(M, Wq.rows, K), X.device)
    cw = Wq.c_struct()
    _check(load().bd_linear(ptr, dt, M, K, ld, ctypes.byref(cw), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                            out.stride(0), wptr, wbytes, _stream(stream)))
    return out


def linear_requant_workspace_size(M, N, K):
    b = ctypes.c_size_t()
    _check(load().bd_linear_requant_workspace_size(M, N, K, ctypes.byref(b)))
    return b.value


def gemm_requant_workspace_size(M, N, K):
    b = ctypes.c_size_t()
    _check(load().bd_gemm_requant_workspace_size(M, N, K, ctypes.byref(b)))
    return b.value


def linear_requant(X, Wq, out=None, workspace=None, stream=None):
    """The quantised linear layer with its result requantised for the next product (Sec. 3.3, last
    paragraph): returns the QTensor [M, N] instead of Y."""
    ptr, dt, ld = _src(X)
    M, K = X.shape
    out = out or QTensor(M, Wq.rows, X.device)
    workspace, wptr, wbytes = _ws(workspace, linear_requant_workspace_size(M, Wq.rows, K), X.device)
    cw, cy = Wq.c_struct(), out.c_struct()
    _check(load().bd_linear_requant(ptr, dt, M, K, ld, ctypes.byref(cw), ctypes.byref(cy), wptr, wbytes, _stream(stream)))
    return out


def gemm_requant(A, B, out=None, workspace=None, stream=None):
    """dq(A) dq(B)^T requantised along N for the next product (Sec. 3.3, last paragraph)."""
    out = out or QTensor(A.rows, B.rows, A.codes.device)
    workspace, wptr, wbytes = _ws(workspace, gemm_requant_workspace_size(A.rows, B.rows, A.K), A.codes.device)
    ca, cb, cy = A.c_struct(), B.c_struct(), out.c_struct()
    _check(load().bd_gemm_requant(ctypes.byref(ca), ctypes.byref(cb), ctypes.byref(cy), wptr, wbytes, _stream(stream)))
    return out


def physical_k(K, block):
    """K of the stored operand for a block size: block 16 is stored zero-padded to 32-element blocks."""
    return 2 * K if block == 16 else K


def quantize_bs(X, block, select=SELECT_TWO_STAGE, out=None, stream=None):
    """Quantise X [rows, K] along K in blocks of 16, 32 or 64 elements (Sec. 4.2, Table 3).  The result is an
    ordinary QTensor with K' = physical_k(K, block) that every product takes as it is."""
    ptr, dt, ld = _src(X)
    rows, K = X.shape
    out = out or QTensor(rows, physical_k(K, block), X.device)
    cq = out.c_struct()
    _check(load().bd_quantize_bs(ptr, dt, rows, K, ld, select, block, ctypes.byref(cq), _stream(stream)))
    return out


def export_canonical_bs(q, block, stream=None):
    """(codes [rows, K/2], ids [rows, K/block], scales [rows, K/block]) of an operand stored for `block`."""
    dev = q.codes.device
    K = q.K // 2 if block == 16 else q.K
    codes = torch.empty(q.rows, K // 2, dtype=torch.uint8, device=dev)
    ids = torch.empty(q.rows, K // block, dtype=torch.uint8, device=dev)
    scales = torch.empty(q.rows, K // block, dtype=torch.uint8, device=dev)
    cq = q.c_struct()
    _check(load().bd_export_canonical_bs(ctypes.byref(cq), block, ctypes.c_void_p(codes.data_ptr()),
                                         ctypes.c_void_p(ids.data_ptr()), ctypes.c_void_p(scales.data_ptr()), _stream(stream)))
    return codes, ids, scales


def linear_bs_workspace_size(M, N, K, block):
    b = ctypes.c_size_t()
    _check(load().bd_linear_bs_workspace_size(M, N, K, block, ctypes.byref(b)))
    return b.value


def linear_bs(X, Wq, block, out=None, dtype=torch.bfloat16, workspace=None, stream=None):
    """The quantised linear layer with blocks of 16, 32 or 64 elements; Wq from quantize_bs with the same block."""
    ptr, dt, ld = _src(X)
    M, K = X.shape
    if out is None:
        out = torch.empty(M, Wq.rows, dtype=dtype, device=X.device)
    workspace, wptr, wbytes = _ws(workspace, linear_bs_workspace_size(M, Wq.rows, K, block), X.device)
    cw = Wq.c_struct()
    _check(load().bd_linear_bs(ptr, dt, M, K, ld, block, ctypes.byref(cw), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                               out.stride(0), wptr, wbytes, _stream(stream)))
    return out


def attention_workspace_size(heads, group, sk, head_dim):
    b = ctypes.c_size_t()
    _check(load().bd_attention_workspace_size(heads, group, sk, head_dim, ctypes.byref(b)))
    return b.value


def attention(Qs, Ks, Vs, group=1, scale=None, out=None, dtype=torch.bfloat16, dump=False, workspace=True, stream=None):
    """Full-path attention in one kernel (Sec. 4.1 scope "all"; Sec. 3.3 softmax in high precision): Qs are `heads`
    operands [Sq, d], Ks heads / group operands [Sk, d], Vs heads / group operands [d, Sk] (quantize_act with
    AXIS_STRIDED).  Returns O [heads, Sq, d]; with dump=True also a dict of S, P (fp32 [heads, Sq, Sk]) and the
    canonical codes, ids, scales of the quantised P, which the kernel then writes for checking.  workspace: True = allocate
    the scratch in which K and V are expanded to bf16 once (faster), False / None = none, or a uint8 CUDA tensor."""
    heads, sq, d, sk = len(Qs), Qs[0].rows, Qs[0].K, Ks[0].rows
    dev = Qs[0].codes.device
    if scale is None:
        scale = d ** -0.5
    if out is None:
        out = torch.empty(heads, sq, d, dtype=dtype, device=dev)
    cq = (_CQTensor * heads)(*[q.c_struct() for q in Qs])
    ck = (_CQTensor * len(Ks))(*[k.c_struct() for k in Ks])
    cv = (_CQTensor * len(Vs))(*[v.c_struct() for v in Vs])
    extra, cd = None, None
    if dump:
        extra = {"S": torch.empty(heads, sq, sk, dtype=torch.float32, device=dev), "P": torch.empty(heads, sq, sk, dtype=torch.float32, device=dev),
                 "codes": torch.empty(heads, sq, sk // 2, dtype=torch.uint8, device=dev),
                 "ids": torch.empty(heads, sq, sk // 32, dtype=torch.uint8, device=dev),
                 "scales": torch.empty(heads, sq, sk // 32, dtype=torch.uint8, device=dev)}
        cd = ctypes.pointer(_CAttentionDump(*[extra[k].data_ptr() for k in ("S", "P", "codes", "ids", "scales")]))
    if workspace is True:
        b = ctypes.c_size_t()
        _check(load().bd_attention_workspace_size(heads, group, sk, d, ctypes.byref(b)))
        workspace = torch.empty(b.value, dtype=torch.uint8, device=dev)
    wptr, wbytes = (ctypes.c_void_p(workspace.data_ptr()), workspace.numel()) if isinstance(workspace, torch.Tensor) else (None, 0)
    _check(load().bd_attention(cq, ck, cv, heads, group, ctypes.c_float(scale), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                               out.stride(1), out.stride(0), cd, wptr, wbytes, _stream(stream)))
    return (out, extra) if dump else out


class KVCache:
    """KV cache of one KV head (appendix "Quantization Dimension", Fig. 9b): keys quantised per token along
    head_dim, values in 4-bit chunks of 32 tokens along the token axis, the newest length % 32 value rows in
    high precision.  Buffers are torch tensors; every step runs in the library."""

    def __init__(self, capacity, head_dim, dtype=torch.bfloat16, device="cuda"):
        self.capacity, self.head_dim, self.dtype = capacity, head_dim, dtype
        self.k = QTensor(capacity, head_dim, device)
        self.v = QTensor(head_dim, capacity, device)
        self.v_recent = torch.zeros(32, head_dim, dtype=dtype, device=device)
        self._c = _CKVCache(self.k.c_struct(), self.v.c_struct(), self.v_recent.data_ptr(), _TORCH_DTYPE[dtype], capacity, head_dim, 0)
        self._ws = None
        _check(load().bd_kvcache_reset(ctypes.byref(self._c), _stream()))

    @property
    def length(self):
        return int(self._c.length)

    def append(self, k_new, v_new, stream=None):
        kp, kdt, ldk = _src(k_new)
        vp_, vdt, ldv = _src(v_new)
        if kdt != self._c.dtype or vdt != self._c.dtype or k_new.shape != v_new.shape or k_new.shape[1] != self.head_dim:
            raise ValueError("key / value rows must be [t, head_dim] of the cache's dtype")
        _check(load().bd_kvcache_append(ctypes.byref(self._c), kp, vp_, k_new.shape[0], ldk, ldv, _stream(stream)))

    def _workspace(self, q_rows):
        b = ctypes.c_size_t()
        _check(load().bd_kvcache_workspace_size(self.capacity, self.head_dim, q_rows, ctypes.byref(b)))
        if self._ws is None or self._ws.numel() < b.value:
            self._ws = torch.empty(max(b.value, 256), dtype=torch.uint8, device=self.k.codes.device)
        return ctypes.c_void_p(self._ws.data_ptr()), self._ws.numel()

    def scores(self, Q, out=None, dtype=torch.float32, stream=None):
        """S [q, length] = dq(Q) dq(K)^T for a quantised query operand Q [q, head_dim]."""
        if out is None:
            out = torch.empty(Q.rows, self.length, dtype=dtype, device=self.k.codes.device)
        wptr, wbytes = self._workspace(Q.rows)
        cq = Q.c_struct()
        _check(load().bd_kvcache_scores(ctypes.byref(self._c), ctypes.byref(cq), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype),
                                        out.stride(0), wptr, wbytes, _stream(stream)))
        return out

    def pv(self, P, out=None, dtype=torch.float32, stream=None):
        """O [q, head_dim] = P V for fp32 probabilities P [q, length]."""
        if P.dtype != torch.float32 or P.dim() != 2 or P.stride(1) != 1 or P.shape[1] != self.length:
            raise ValueError("P must be fp32 [q, length] with a contiguous last axis")
        if out is None:
            out = torch.empty(P.shape[0], self.head_dim, dtype=dtype, device=P.device)
        wptr, wbytes = self._workspace(P.shape[0])
        _check(load().bd_kvcache_pv(ctypes.byref(self._c), ctypes.c_void_p(P.data_ptr()), P.shape[0], P.stride(0),
                                    ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype), out.stride(0), wptr, wbytes, _stream(stream)))
        return out


def _kv_batch(caches, q_rows):
    n, c0 = len(caches), caches[0]
    arr = (_CKVCache * n)(*[c._c for c in caches])
    b = ctypes.c_size_t()
    _check(load().bd_kvcache_batched_workspace_size(n, c0.capacity, c0.head_dim, q_rows, ctypes.byref(b)))
    if c0._ws is None or c0._ws.numel() < b.value:
        c0._ws = torch.empty(max(b.value, 256), dtype=torch.uint8, device=c0.k.codes.device)
    return arr, ctypes.c_void_p(c0._ws.data_ptr()), c0._ws.numel()


def kvcache_append_batched(caches, k_new, v_new, stream=None):
    """t new tokens for n KV heads of the same length in one call: k_new, v_new [n, t, head_dim] of the caches' dtype."""
    n, c0 = len(caches), caches[0]
    if k_new.shape != v_new.shape or k_new.dim() != 3 or k_new.shape[0] != n or k_new.shape[2] != c0.head_dim or k_new.stride(2) != 1 or v_new.stride(2) != 1:
        raise ValueError("key / value rows must be [n, t, head_dim] with a contiguous last axis")
    if _TORCH_DTYPE[k_new.dtype] != c0._c.dtype or v_new.dtype != k_new.dtype:
        raise ValueError("key / value rows must have the caches' dtype")
    arr = (_CKVCache * n)(*[c._c for c in caches])
    _check(load().bd_kvcache_append_batched(arr, n, ctypes.c_void_p(k_new.data_ptr()), ctypes.c_void_p(v_new.data_ptr()), k_new.shape[1],
                                            k_new.stride(1), v_new.stride(1), k_new.stride(0), v_new.stride(0), _stream(stream)))
    for c, done in zip(caches, arr):
        c._c.length = done.length


def kvcache_scores_batched(caches, Qs, out=None, dtype=torch.float32, stream=None):
    """S [n, q, length]: the scores of n KV heads (same length) in one call; Qs[i] is head i's quantised query operand."""
    n, q, length = len(caches), Qs[0].rows, caches[0].length
    if out is None:
        out = torch.empty(n, q, length, dtype=dtype, device=caches[0].k.codes.device)
    arr, wptr, wbytes = _kv_batch(caches, q)
    cq = (_CQTensor * n)(*[x.c_struct() for x in Qs])
    _check(load().bd_kvcache_scores_batched(arr, n, cq, ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype), out.stride(1), out.stride(0),
                                            wptr, wbytes, _stream(stream)))
    return out


def kvcache_pv_batched(caches, P, out=None, dtype=torch.float32, stream=None):
    """O [n, q, head_dim] = P[i] V[i] for fp32 probabilities P [n, q, length] of n KV heads (same length) in one call."""
    n = len(caches)
    if P.dtype != torch.float32 or P.dim() != 3 or P.stride(2) != 1 or P.shape[0] != n or P.shape[2] != caches[0].length:
        raise ValueError("P must be fp32 [n, q, length] with a contiguous last axis")
    if out is None:
        out = torch.empty(n, P.shape[1], caches[0].head_dim, dtype=dtype, device=P.device)
    arr, wptr, wbytes = _kv_batch(caches, P.shape[1])
    _check(load().bd_kvcache_pv_batched(arr, n, ctypes.c_void_p(P.data_ptr()), P.shape[1], P.stride(1), P.stride(0),
                                        ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype), out.stride(1), out.stride(0), wptr, wbytes,
                                        _stream(stream)))
    return out


def kvcache_attention(caches, Qs, scale, out=None, dtype=torch.float32, probs=None, stream=None):
    """O [n, q, head_dim] of one decode step over n cached heads: scores, fp32 softmax of scale * S, P V.  `probs`
    (fp32 [n, q, pitch >= length], pitch a multiple of 4) receives the probabilities when given."""
    n, c0, q = len(caches), caches[0], Qs[0].rows
    if out is None:
        out = torch.empty(n, q, c0.head_dim, dtype=dtype, device=c0.k.codes.device)
    arr = (_CKVCache * n)(*[c._c for c in caches])
    b = ctypes.c_size_t()
    _check(load().bd_kvcache_attention_workspace_size(n, c0.capacity, c0.head_dim, q, ctypes.byref(b)))
    if c0._ws is None or c0._ws.numel() < b.value:
        c0._ws = torch.empty(max(b.value, 256), dtype=torch.uint8, device=c0.k.codes.device)
    cq = (_CQTensor * n)(*[x.c_struct() for x in Qs])
    pp, ldp, sp = (ctypes.c_void_p(probs.data_ptr()), probs.stride(1), probs.stride(0)) if probs is not None else (None, 0, 0)
    _check(load().bd_kvcache_attention(arr, n, cq, ctypes.c_float(scale), ctypes.c_void_p(out.data_ptr()), _ydtype(out.dtype), out.stride(1),
                                       out.stride(0), pp, ldp, sp, ctypes.c_void_p(c0._ws.data_ptr()), c0._ws.numel(), _stream(stream)))
    return out


NOALLOC_SCRATCH_BYTES = 32 << 20


def linear_noalloc(X, Wq, out, stream=None):
    """bd_linear without a workspace argument and without any allocation: for callers that may not
    allocate device memory (frozen memory plans, plugins handed only inputs and outputs).  `out`
    must be preallocated; problems whose scratch need exceeds NOALLOC_SCRATCH_BYTES raise status 9.
    Calls share one built-in device buffer, so calls that overlap on the GPU must be serialised."""
    ptr, dt, ld = _src(X)
    M, K = X.shape
    cw = Wq.c_struct()
    _check(load().bd_linear_noalloc(ptr, dt, M, K, ld, ctypes.byref(cw), ctypes.c_void_p(out.data_ptr()),
                                    _ydtype(out.dtype), out.stride(0), _stream(stream)))
    return out


def export_canonical(q, stream=None):
    """(codes [rows, K/2], ids [rows, K/32], scales [rows, K/32]) as uint8 CUDA tensors."""
    dev = q.codes.device
    codes = torch.empty(q.rows, q.K // 2, dtype=torch.uint8, device=dev)
    ids = torch.empty(q.rows, q.K // 32, dtype=torch.uint8, device=dev)
    scales = torch.empty(q.rows, q.K // 32, dtype=torch.uint8, device=dev)
    cq = q.c_struct()
    _check(load().bd_export_canonical(ctypes.byref(cq), ctypes.c_void_p(codes.data_ptr()),
                                      ctypes.c_void_p(ids.data_ptr()), ctypes.c_void_p(scales.data_ptr()),
                                      _stream(stream)))
    return codes, ids, scales


def import_canonical(codes, ids, scales, stream=None):
    """Build a QTensor from canonical uint8 CUDA tensors."""
    rows, K = codes.shape[0], codes.shape[1] * 2
    q = QTensor(rows, K, codes.device)
    cq = q.c_struct()
    codes, ids, scales = codes.contiguous(), ids.contiguous(), scales.contiguous()
    _check(load().bd_import_canonical(ctypes.c_void_p(codes.data_ptr()), ctypes.c_void_p(ids.data_ptr()),
                                      ctypes.c_void_p(scales.data_ptr()), ctypes.byref(cq), _stream(stream)))
    return q


def dequantize(q, stream=None):
    """fp32 [rows, K] values of a quantised operand (Sec. 3.3, Fig. 6)."""
    out = torch.empty(q.rows, q.K, dtype=torch.float32, device=q.codes.device)
    cq = q.c_struct()
    _check(load().bd_dequantize(ctypes.byref(cq), ctypes.c_void_p(out.data_ptr()), out.stride(0), _stream(stream)))
    return out
