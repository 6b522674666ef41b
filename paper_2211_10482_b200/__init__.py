"""Python binding of libstructtensor (C ABI in include/structtensor.h).

Argument marshalling only: every function takes torch CUDA tensors, passes their raw device
pointers, extents and the current CUDA stream to the C entry point of the same name, and
raises ``StError`` when the call returns a non-zero status.  torch is used for device
memory and streams only; there is no CPU or torch fallback -- if the shared library has not
been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# STRUCTTENSOR_LIB selects another build of the library, e.g. the range-checking debug build
# libstructtensor_check.so (python -m paper_2211_10482_b200._build --check)
LIB_PATH = os.environ.get("STRUCTTENSOR_LIB") or os.path.join(_HERE, "libstructtensor.so")

# st_status
ST_OK, ST_ERR_NULL, ST_ERR_SHAPE, ST_ERR_ALIGN, ST_ERR_DTYPE, ST_ERR_WORKSPACE, ST_ERR_UNSUPPORTED, \
    ST_ERR_CUDA, ST_ERR_DEV_TIMEOUT, ST_ERR_DEV_BOUNDS, ST_ERR_STATIC_SCRATCH = range(11)
ST_STATIC_SCRATCH_BYTES = 16 << 20
# st_dtype
ST_F32, ST_BF16, ST_F64 = 0, 1, 2
# st_kind
ST_TRI_UPPER, ST_TET, ST_BAND, ST_BLOCKDIAG, ST_FIXED_ROW, ST_FIXED_COL, ST_SIMPLEX4 = 0, 1, 2, 3, 4, 5, 6
# st_fill
ST_FILL_ZERO, ST_FILL_SYMMETRIC = 0, 1
# st_op
ST_OP_SYM_MOMENT2, ST_OP_SYM_MOMENT3, ST_OP_MTTKRP_TRI, ST_OP_TTM_BLOCKDIAG, ST_OP_SYM_MOMENT4, \
    ST_OP_MTTKRP_SLICE = 0, 1, 2, 3, 4, 5
# flags
ST_FLAG_DENSE_CONTROL = 1
ST_FLAG_TC_TF32 = 2
ST_FLAG_TC_BF16 = 4
ST_FLAG_TC_SPLIT = 8

EXPORTS = [
    "st_packed_elems", "st_dense_elems", "st_pack", "st_unpack", "st_workspace_bytes", "st_sym_moment2",
    "st_sym_moment3", "st_sym_moment3_static", "st_sym_moment4", "st_mttkrp_tri", "st_mttkrp_slice", "st_ttm_blockdiag", "st_ttm_packed",
    "st_thp", "st_packed_axpby", "st_packed_mul", "st_check_status", "st_status_string",
    "st_abi_version", "st_bounds_checked_build", "st_bounds_self_test",
]


class StLayout(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("reserved", ctypes.c_int32), ("d", ctypes.c_int64),
                ("inner", ctypes.c_int64), ("kl", ctypes.c_int64), ("ku", ctypes.c_int64),
                ("nblocks", ctypes.c_int64), ("bs", ctypes.c_int64)]


@dataclass(frozen=True)
class Layout:
    kind: int
    d: int
    inner: int = 1
    kl: int = 0
    ku: int = 0
    nblocks: int = 0
    bs: int = 0

    def c(self) -> StLayout:
        return StLayout(self.kind, 0, self.d, self.inner, self.kl, self.ku, self.nblocks, self.bs)


class StError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libstructtensor.so is missing: build it with `python -m paper_2211_10482_b200._build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        i64, vp, ci, cu, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_uint, ctypes.c_size_t
        LP = ctypes.POINTER(StLayout)
        L.st_packed_elems.argtypes = [LP]
        L.st_packed_elems.restype = i64
        L.st_dense_elems.argtypes = [LP]
        L.st_dense_elems.restype = i64
        L.st_pack.argtypes = [LP, ci, vp, vp, vp]
        L.st_unpack.argtypes = [LP, ci, vp, vp, ci, vp]
        L.st_workspace_bytes.argtypes = [ci, i64, i64, i64, i64, cu]
        L.st_workspace_bytes.restype = sz
        L.st_bounds_self_test.argtypes = [vp]
        L.st_sym_moment2.argtypes = [vp, ci, i64, i64, i64, vp, vp, sz, cu, vp]
        L.st_sym_moment3.argtypes = [vp, i64, i64, i64, vp, vp, sz, cu, vp]
        L.st_sym_moment3_static.argtypes = [vp, i64, i64, i64, vp, cu, vp]
        L.st_sym_moment4.argtypes = [vp, i64, i64, i64, vp, vp, sz, cu, vp]
        L.st_mttkrp_tri.argtypes = [vp, i64, i64, vp, vp, i64, vp, vp, sz, cu, vp]
        L.st_ttm_blockdiag.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp, sz, cu, vp]
        L.st_mttkrp_slice.argtypes = [vp, i64, i64, i64, i64, i64, vp, vp, i64, vp, vp, sz, cu, vp]
        L.st_ttm_packed.argtypes = [LP, vp, vp, i64, vp, vp, sz, cu, vp]
        L.st_thp.argtypes = [LP, vp, vp, vp, vp]
        L.st_packed_axpby.argtypes = [i64, ctypes.c_float, vp, ctypes.c_float, vp, vp, vp]
        L.st_packed_mul.argtypes = [i64, vp, vp, vp, vp]
        L.st_check_status.argtypes = [vp, vp]
        L.st_status_string.argtypes = [ci]
        L.st_status_string.restype = ctypes.c_char_p
        L.st_abi_version.restype = ci
        for name in ("st_pack", "st_unpack", "st_sym_moment2", "st_sym_moment3", "st_sym_moment3_static", "st_sym_moment4", "st_mttkrp_tri",
                     "st_mttkrp_slice", "st_ttm_blockdiag", "st_ttm_packed", "st_thp", "st_packed_axpby", "st_packed_mul", "st_check_status"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().st_status_string(int(status)).decode()


_DTYPES = {torch.float32: ST_F32, torch.bfloat16: ST_BF16, torch.float64: ST_F64}


def _dtype(t: torch.Tensor) -> int:
    if t.dtype in _DTYPES:
        return _DTYPES[t.dtype]
    if t.dtype in (torch.int32, torch.uint32):
        return ST_F32    # pack/unpack are bit copies: any 4-byte type travels as ST_F32
    if t.dtype in (torch.int16, torch.uint16, torch.float16):
        return ST_BF16
    if t.dtype == torch.int64:
        return ST_F64
    raise TypeError("unsupported dtype %s" % t.dtype)


def _dev(t: torch.Tensor, name: str) -> int:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str) -> None:
    if status != ST_OK:
        raise StError(status, where)


def st_packed_elems(layout: Layout) -> int:
    return int(lib().st_packed_elems(ctypes.byref(layout.c())))


def st_dense_elems(layout: Layout) -> int:
    return int(lib().st_dense_elems(ctypes.byref(layout.c())))


def st_workspace_bytes(op: int, a: int, b: int, c: int = 0, e: int = 0, flags: int = 0) -> int:
    return int(lib().st_workspace_bytes(op, a, b, c, e, flags))


_allocator = None          # callable (numel, dtype, device) -> tensor, or None for torch.empty
_last_ws: dict = {}        # device index -> the workspace of the most recent compute call on that device


def set_allocator(fn) -> None:
    """Device memory for the outputs and workspaces that a caller does not pass comes from
    ``fn(numel, dtype, device)`` (a 1-d tensor whose data pointer is 256-byte aligned); ``None``
    restores ``torch.empty``.  For callers that manage their own pool, and for tests that
    surround every buffer with guard bands."""
    global _allocator
    _allocator = fn


def _alloc(numel: int, dtype, device) -> torch.Tensor:
    if _allocator is not None:
        return _allocator(int(numel), dtype, device)
    return torch.empty(int(numel), dtype=dtype, device=device)


def _workspace(query, device, ws: torch.Tensor | None) -> torch.Tensor:
    """The caller's workspace, or a fresh one of the size that `query()` reports.  Either way it is
    remembered as the device's last workspace, so that st_check_status() can read the status word
    that the call's kernels may have written."""
    if ws is None:
        ws = _alloc(max(int(query()), 256), torch.uint8, device)
    _last_ws[ws.device.index] = ws
    return ws


def st_pack(dense: torch.Tensor, layout: Layout, out: torch.Tensor | None = None) -> torch.Tensor:
    n = st_packed_elems(layout)
    if n < 0:
        raise StError(ST_ERR_SHAPE, "st_packed_elems")
    if dense.numel() != st_dense_elems(layout):
        raise ValueError("dense has %d elements, layout needs %d" % (dense.numel(), st_dense_elems(layout)))
    if out is None:
        out = _alloc(n, dense.dtype, dense.device)
    _check(lib().st_pack(ctypes.byref(layout.c()), _dtype(dense), _dev(dense, "dense"), _dev(out, "out"),
                         _stream()), "st_pack")
    return out


def st_unpack(packed: torch.Tensor, layout: Layout, fill: int = ST_FILL_ZERO,
              out: torch.Tensor | None = None) -> torch.Tensor:
    n = st_dense_elems(layout)
    if n < 0:
        raise StError(ST_ERR_SHAPE, "st_dense_elems")
    if packed.numel() != st_packed_elems(layout):
        raise ValueError("packed has %d elements, layout needs %d" % (packed.numel(), st_packed_elems(layout)))
    if out is None:
        out = _alloc(n, packed.dtype, packed.device)
    _check(lib().st_unpack(ctypes.byref(layout.c()), _dtype(packed), _dev(packed, "packed"), _dev(out, "out"),
                           int(fill), _stream()), "st_unpack")
    return out


def st_sym_moment2(X: torch.Tensor, out: torch.Tensor | None = None, ws: torch.Tensor | None = None,
                   flags: int = 0) -> torch.Tensor:
    """Packed upper triangle of X^T X; X is [N, d] float32 or bfloat16."""
    N, d = X.shape
    if X.dtype not in (torch.float32, torch.bfloat16):
        raise TypeError("X must be float32 or bfloat16")
    xdt = _DTYPES[X.dtype]
    if out is None:
        out = _alloc(d * (d + 1) // 2, torch.float32, X.device)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_SYM_MOMENT2, N, d, xdt, 0, flags), X.device, ws)
    _check(lib().st_sym_moment2(_dev(X, "X"), xdt, N, d, X.stride(0), _dev(out, "out"), ws.data_ptr(),
                                ws.numel() * ws.element_size(), flags, _stream()), "st_sym_moment2")
    return out


def st_sym_moment3(X: torch.Tensor, out: torch.Tensor | None = None, ws: torch.Tensor | None = None,
                   flags: int = 0) -> torch.Tensor:
    """Packed tetrahedron sum_n X[n,i] X[n,j] X[n,k], i<=j<=k; X is [N, d] float32."""
    N, d = X.shape
    if X.dtype != torch.float32:
        raise TypeError("X must be float32")
    if out is None:
        out = _alloc(d * (d + 1) * (d + 2) // 6, torch.float32, X.device)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_SYM_MOMENT3, N, d, 0, 0, flags), X.device, ws)
    _check(lib().st_sym_moment3(_dev(X, "X"), N, d, X.stride(0), _dev(out, "out"), ws.data_ptr(),
                                ws.numel() * ws.element_size(), flags, _stream()), "st_sym_moment3")
    return out


def st_sym_moment4(X: torch.Tensor, out: torch.Tensor | None = None, ws: torch.Tensor | None = None,
                   flags: int = 0) -> torch.Tensor:
    """Packed 4-simplex sum_n X[n,i] X[n,j] X[n,k] X[n,l], i<=j<=k<=l; X is [N, d] float32."""
    N, d = X.shape
    if X.dtype != torch.float32:
        raise TypeError("X must be float32")
    if out is None:
        out = _alloc(d * (d + 1) * (d + 2) * (d + 3) // 24, torch.float32, X.device)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_SYM_MOMENT4, N, d, 0, 0, flags), X.device, ws)
    _check(lib().st_sym_moment4(_dev(X, "X"), N, d, X.stride(0), _dev(out, "out"), ws.data_ptr(),
                                ws.numel() * ws.element_size(), flags, _stream()), "st_sym_moment4")
    return out


def st_sym_moment3_static(X: torch.Tensor, out: torch.Tensor, flags: int = 0) -> torch.Tensor:
    """st_sym_moment3 with the library's built-in scratch, for callers that must not allocate:
    the caller passes the input and the output tensor, and nothing is allocated here either.
    Calls that overlap on the GPU race on the shared scratch; keep them on one stream."""
    N, d = X.shape
    if X.dtype != torch.float32 or out.dtype != torch.float32:
        raise TypeError("X and out must be float32")
    if out.numel() != d * (d + 1) * (d + 2) // 6:
        raise ValueError("out must hold d(d+1)(d+2)/6 elements")
    _check(lib().st_sym_moment3_static(_dev(X, "X"), N, d, X.stride(0), _dev(out, "out"), flags, _stream()),
           "st_sym_moment3_static")
    return out


def st_mttkrp_tri(Bp: torch.Tensor, C: torch.Tensor, D: torch.Tensor, out: torch.Tensor | None = None,
                  ws: torch.Tensor | None = None, flags: int = 0) -> torch.Tensor:
    """A[i,r] = sum_{j>=i,k} Bp[p(i,j),k] C[j,r] D[k,r]; Bp is [I(I+1)/2, K] (dense [I,I,K] with the
    dense-control flag)."""
    I, R = C.shape
    K = D.shape[0]
    for t in (Bp, C, D):
        if t.dtype != torch.float32:
            raise TypeError("inputs must be float32")
    want = I * I * K if (flags & ST_FLAG_DENSE_CONTROL) else I * (I + 1) // 2 * K
    if Bp.numel() != want or D.shape[1] != R:
        raise ValueError("shape mismatch")
    if out is None:
        out = _alloc(I * R, torch.float32, Bp.device).view(I, R)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_MTTKRP_TRI, I, K, R, 0, flags), Bp.device, ws)
    _check(lib().st_mttkrp_tri(_dev(Bp, "Bp"), I, K, _dev(C, "C"), _dev(D, "D"), R, _dev(out, "out"),
                               ws.data_ptr(), ws.numel() * ws.element_size(), flags, _stream()),
           "st_mttkrp_tri")
    return out


def st_mttkrp_slice(Bp: torch.Tensor, C: torch.Tensor, D: torch.Tensor, I: int, fixed_i: int = -1, fixed_j: int = -1,
                    out: torch.Tensor | None = None, ws: torch.Tensor | None = None, flags: int = 0) -> torch.Tensor:
    """MTTKRP on a tensor that is non-zero only where i == fixed_i and / or j == fixed_j; Bp is that slice."""
    J, R = C.shape
    K = D.shape[0]
    for t in (Bp, C, D):
        if t.dtype != torch.float32:
            raise TypeError("inputs must be float32")
    rows = (1 if fixed_j >= 0 else J) if fixed_i >= 0 else I
    if Bp.numel() != rows * K or D.shape[1] != R:
        raise ValueError("shape mismatch")
    if out is None:
        out = _alloc(I * R, torch.float32, Bp.device).view(I, R)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_MTTKRP_SLICE, I, J, K, R, flags), Bp.device, ws)
    _check(lib().st_mttkrp_slice(_dev(Bp, "Bp"), I, J, K, fixed_i, fixed_j, _dev(C, "C"), _dev(D, "D"), R,
                                 _dev(out, "out"), ws.data_ptr(), ws.numel() * ws.element_size(), flags, _stream()),
           "st_mttkrp_slice")
    return out


def st_ttm_blockdiag(Bp: torch.Tensor, U: torch.Tensor, nblocks: int, bs: int,
                     out: torch.Tensor | None = None, ws: torch.Tensor | None = None,
                     flags: int = 0) -> torch.Tensor:
    """Ap[b,i',j',r] = sum_k Bp[b,i',j',k] U[k,r] on the diagonal blocks only."""
    K, R = U.shape
    if Bp.dtype != torch.float32 or U.dtype != torch.float32:
        raise TypeError("inputs must be float32")
    d = nblocks * bs
    rows = d * d if (flags & ST_FLAG_DENSE_CONTROL) else nblocks * bs * bs
    if Bp.numel() != rows * K:
        raise ValueError("shape mismatch")
    if out is None:
        out = _alloc(rows * R, torch.float32, Bp.device).view(rows, R)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_TTM_BLOCKDIAG, nblocks, bs, K, R, flags), Bp.device, ws)
    _check(lib().st_ttm_blockdiag(_dev(Bp, "Bp"), nblocks, bs, K, _dev(U, "U"), R, _dev(out, "out"),
                                  ws.data_ptr(), ws.numel() * ws.element_size(), flags, _stream()),
           "st_ttm_blockdiag")
    return out


def st_ttm_packed(Bp: torch.Tensor, U: torch.Tensor, layout: Layout, out: torch.Tensor | None = None,
                  ws: torch.Tensor | None = None, flags: int = 0) -> torch.Tensor:
    """Ap[p,r] = sum_k Bp[p,k] U[k,r] for every packed position p of `layout` (inner = K)."""
    K, R = U.shape
    if Bp.dtype != torch.float32 or U.dtype != torch.float32:
        raise TypeError("inputs must be float32")
    if layout.inner != K or Bp.numel() != st_packed_elems(layout):
        raise ValueError("shape mismatch")
    rows = Bp.numel() // K
    if out is None:
        out = _alloc(rows * R, torch.float32, Bp.device).view(rows, R)
    ws = _workspace(lambda: st_workspace_bytes(ST_OP_TTM_BLOCKDIAG, rows, 1, K, R, flags), Bp.device, ws)
    _check(lib().st_ttm_packed(ctypes.byref(layout.c()), _dev(Bp, "Bp"), _dev(U, "U"), R, _dev(out, "out"),
                               ws.data_ptr(), ws.numel() * ws.element_size(), flags, _stream()), "st_ttm_packed")
    return out


def st_thp(Bp: torch.Tensor, C: torch.Tensor, layout: Layout, out: torch.Tensor | None = None) -> torch.Tensor:
    """Ap = Bp * (C at the unique positions of `layout`): packed B, dense C, packed result."""
    if Bp.dtype != torch.float32 or C.dtype != torch.float32:
        raise TypeError("inputs must be float32")
    if Bp.numel() != st_packed_elems(layout) or C.numel() != st_dense_elems(layout):
        raise ValueError("shape mismatch")
    if out is None:
        out = _alloc(Bp.numel(), torch.float32, Bp.device).view(Bp.shape)
    _check(lib().st_thp(ctypes.byref(layout.c()), _dev(Bp, "Bp"), _dev(C, "C"), _dev(out, "out"), _stream()), "st_thp")
    return out


def st_packed_axpby(alpha: float, a: torch.Tensor, beta: float, b: torch.Tensor,
                    out: torch.Tensor | None = None) -> torch.Tensor:
    """out = alpha * a + beta * b for two packed float32 arrays of the same layout (out may be a or b)."""
    if a.dtype != torch.float32 or b.dtype != torch.float32 or a.numel() != b.numel():
        raise ValueError("two float32 arrays of the same size are needed")
    if out is None:
        out = _alloc(a.numel(), torch.float32, a.device).view(a.shape)
    _check(lib().st_packed_axpby(a.numel(), alpha, _dev(a, "a"), beta, _dev(b, "b"), _dev(out, "out"), _stream()),
           "st_packed_axpby")
    return out


def st_packed_mul(a: torch.Tensor, b: torch.Tensor, out: torch.Tensor | None = None) -> torch.Tensor:
    """out = a * b for two packed float32 arrays of the same layout (out may be a or b)."""
    if a.dtype != torch.float32 or b.dtype != torch.float32 or a.numel() != b.numel():
        raise ValueError("two float32 arrays of the same size are needed")
    if out is None:
        out = _alloc(a.numel(), torch.float32, a.device).view(a.shape)
    _check(lib().st_packed_mul(a.numel(), _dev(a, "a"), _dev(b, "b"), _dev(out, "out"), _stream()), "st_packed_mul")
    return out


def st_check_status(ws: torch.Tensor | None = None) -> int:
    """Synchronises the current stream and returns the device-side status of `ws`; without an
    argument, of the workspace used by the most recent compute call on the current device."""
    if ws is None:
        ws = _last_ws.get(torch.cuda.current_device())
    return int(lib().st_check_status(ws.data_ptr() if ws is not None else None, _stream()))
