"""Thin ctypes binding of the C-ABI library (include/gwq.h).

Argument marshalling only: every step of the method runs in the CUDA kernels of
libgwq.so.  PyTorch tensors are used as plain device buffers (data_ptr) and for
the current stream.  There is no CPU fallback: a missing library or a missing
CUDA device raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgwq.so")

GWQ_OK = 0
(GWQ_ERR_INVALID_ARG, GWQ_ERR_UNSUPPORTED, GWQ_ERR_ALLOC, GWQ_ERR_NONFINITE, GWQ_ERR_TIMEOUT,
 GWQ_ERR_CUDA, GWQ_ERR_WORKSPACE) = range(1, 8)
GWQ_F16, GWQ_BF16, GWQ_F32 = 0, 1, 2
STATUS_NAMES = {
    0: "GWQ_OK", 1: "GWQ_ERR_INVALID_ARG", 2: "GWQ_ERR_UNSUPPORTED", 3: "GWQ_ERR_ALLOC",
    4: "GWQ_ERR_NONFINITE", 5: "GWQ_ERR_TIMEOUT", 6: "GWQ_ERR_CUDA", 7: "GWQ_ERR_WORKSPACE",
}
EXPORTS = ("gwq_select_outliers", "gwq_select_outliers_static", "gwq_outliers_rows", "gwq_pack", "gwq_linear", "gwq_linear_ws",
           "gwq_linear_workspace_bytes", "gwq_linear_multi",
           "gwq_gradient_mean", "gwq_quality", "gwq_linear_host", "gwq_linear_host_async", "gwq_device_status", "gwq_set_wait_limit", "gwq_free", "gwq_status_string")
GWQ_MULTI_MAX = 4


class GwqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class gwq_outliers(C.Structure):
    _fields_ = [("tag", C.c_uint32), ("N", C.c_int32), ("K", C.c_int32), ("nnz", C.c_int64),
                ("row_ptr", C.c_void_p), ("col_idx", C.c_void_p), ("val", C.c_void_p)]


class gwq_packed(C.Structure):
    _fields_ = [("tag", C.c_uint32), ("N", C.c_int32), ("K", C.c_int32), ("bits", C.c_int32),
                ("group", C.c_int32), ("codes", C.c_void_p), ("scales", C.c_void_p),
                ("zeros", C.c_void_p), ("S", C.POINTER(gwq_outliers)), ("priv", C.c_void_p)]


_lib = None


def load_library(path: str = LIB_PATH) -> C.CDLL:
    """Load libgwq.so and declare the prototypes of include/gwq.h."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2411_00850_b200.build` "
                           "(there is no fallback path)")
    lib = C.CDLL(path)
    lib.gwq_select_outliers.restype = C.c_int
    lib.gwq_select_outliers.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_double,
                                        C.POINTER(C.POINTER(gwq_outliers)), C.c_void_p]
    lib.gwq_select_outliers_static.restype = C.c_int
    lib.gwq_select_outliers_static.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_double,
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64,
                                               C.POINTER(C.c_int64), C.c_void_p]
    lib.gwq_outliers_rows.restype = C.c_int
    lib.gwq_outliers_rows.argtypes = [C.POINTER(gwq_outliers), C.c_int32, C.c_int32, C.POINTER(C.POINTER(gwq_outliers)),
                                      C.c_void_p]
    lib.gwq_pack.restype = C.c_int
    lib.gwq_pack.argtypes = [C.c_void_p, C.POINTER(gwq_outliers), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                             C.POINTER(C.POINTER(gwq_packed)), C.c_void_p]
    lib.gwq_linear.restype = C.c_int
    lib.gwq_linear.argtypes = [C.POINTER(gwq_packed), C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int,
                               C.c_void_p]
    lib.gwq_linear_ws.restype = C.c_int
    lib.gwq_linear_ws.argtypes = [C.POINTER(gwq_packed), C.c_void_p, C.c_int, C.c_int32, C.c_void_p, C.c_int,
                                  C.c_void_p, C.c_size_t, C.c_void_p]
    lib.gwq_linear_workspace_bytes.restype = C.c_size_t
    lib.gwq_linear_workspace_bytes.argtypes = [C.POINTER(gwq_packed), C.c_int, C.c_int32]
    lib.gwq_linear_multi.restype = C.c_int
    lib.gwq_linear_multi.argtypes = [C.POINTER(C.POINTER(gwq_packed)), C.c_int32, C.c_void_p, C.c_int, C.c_int32,
                                     C.POINTER(C.c_void_p), C.c_int, C.c_void_p]
    lib.gwq_gradient_mean.restype = C.c_int
    lib.gwq_gradient_mean.argtypes = [C.POINTER(C.c_void_p), C.c_int32, C.c_int64, C.c_void_p, C.c_void_p]
    lib.gwq_quality.restype = C.c_int
    lib.gwq_quality.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(gwq_packed), C.POINTER(C.c_double),
                                C.POINTER(C.c_double), C.c_void_p]
    lib.gwq_linear_host.restype = C.c_int
    lib.gwq_linear_host.argtypes = lib.gwq_linear.argtypes
    lib.gwq_linear_host_async.restype = C.c_int
    lib.gwq_linear_host_async.argtypes = lib.gwq_linear.argtypes
    lib.gwq_device_status.restype = C.c_int
    lib.gwq_device_status.argtypes = [C.POINTER(gwq_packed), C.c_void_p]
    lib.gwq_set_wait_limit.restype = C.c_int
    lib.gwq_set_wait_limit.argtypes = [C.POINTER(gwq_packed), C.c_int64]
    lib.gwq_free.restype = None
    lib.gwq_free.argtypes = [C.c_void_p]
    lib.gwq_status_string.restype = C.c_char_p
    lib.gwq_status_string.argtypes = [C.c_int]
    _lib = lib
    return lib


def _stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float16:
        return GWQ_F16
    if t == torch.bfloat16:
        return GWQ_BF16
    if t == torch.float32:
        return GWQ_F32
    raise TypeError(f"unsupported dtype {t}")


def _check(st: int, where: str):
    if st != GWQ_OK:
        raise GwqError(st, where)


_rt = None


def _cudart() -> C.CDLL:
    """The CUDA runtime that torch has already loaded (used only to copy results out)."""
    global _rt
    if _rt is None:
        last = None
        for name in ("libcudart.so.12", "libcudart.so.13", "libcudart.so"):
            try:
                _rt = C.CDLL(name)
                break
            except OSError as e:
                last = e
        if _rt is None:
            raise RuntimeError(f"CUDA runtime library not found: {last}")
        _rt.cudaMemcpy.restype = C.c_int
    return _rt


def _view(ptr: int, n: int, dtype: torch.dtype, device) -> torch.Tensor:
    """Copy n elements at device address ptr into a new tensor (D2D copy)."""
    out = torch.empty(n, dtype=dtype, device=device)
    if n:
        nbytes = n * out.element_size()
        torch.cuda.current_stream().synchronize()
        rc = _cudart().cudaMemcpy(C.c_void_p(out.data_ptr()), C.c_void_p(ptr), C.c_size_t(nbytes), 3)  # 3 = D2D
        if int(rc) != 0:
            raise RuntimeError(f"cudaMemcpy failed: {rc}")
    return out


class Outliers:
    """Owner of a gwq_outliers* (CSR of the FP16 outlier matrix S)."""

    def __init__(self, handle, device):
        self._h = handle
        self.device = device

    @property
    def N(self): return self._h.contents.N
    @property
    def K(self): return self._h.contents.K
    @property
    def nnz(self): return self._h.contents.nnz

    def arrays(self):
        """(row_ptr int32 [N+1], col_idx int32 [nnz], val int16-bit patterns [nnz]) as tensors."""
        c = self._h.contents
        return (_view(c.row_ptr, c.N + 1, torch.int32, self.device),
                _view(c.col_idx, c.nnz, torch.int32, self.device),
                _view(c.val, c.nnz, torch.int16, self.device))

    def free(self):
        if self._h is not None:
            load_library().gwq_free(C.cast(self._h, C.c_void_p))
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


class Packed:
    """Owner of a gwq_packed* (codes, scales, zero-points and the outliers)."""

    def __init__(self, handle, device):
        self._h = handle
        self.device = device

    @property
    def N(self): return self._h.contents.N
    @property
    def K(self): return self._h.contents.K
    @property
    def bits(self): return self._h.contents.bits
    @property
    def group(self): return self._h.contents.group
    @property
    def nnz(self): return self._h.contents.S.contents.nnz

    def arrays(self):
        """dict of tensors copied out of the packed object (for inspection and parity)."""
        c = self._h.contents
        s = c.S.contents
        nw = c.N * (c.K // 32) * c.bits
        ng = c.N * (c.K // c.group)
        return dict(
            words=_view(c.codes, nw, torch.int32, self.device).view(c.N, -1),
            scales=_view(c.scales, ng, torch.int16, self.device).view(c.N, -1),
            zeros=_view(c.zeros, ng, torch.uint8, self.device).view(c.N, -1),
            row_ptr=_view(s.row_ptr, s.N + 1, torch.int32, self.device),
            col_idx=_view(s.col_idx, s.nnz, torch.int32, self.device),
            val=_view(s.val, s.nnz, torch.int16, self.device),
        )

    def packed_bytes(self) -> int:
        """Bytes of codes + scales + zero-points + CSR as stored by the ABI-visible format."""
        c = self._h.contents
        nnz = c.S.contents.nnz
        return (c.N * (c.K // 32) * c.bits * 4 + c.N * (c.K // c.group) * 3 + (c.N + 1) * 4 + nnz * 6)

    def free(self):
        if self._h is not None:
            load_library().gwq_free(C.cast(self._h, C.c_void_p))
            self._h = None

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass


def _require_cuda(t: torch.Tensor, name: str):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")


def gwq_select_outliers(W: torch.Tensor, G: torch.Tensor, frac: float) -> Outliers:
    """W fp16 [N,K], G fp32 [N,K] on the GPU -> CSR of the ceil(frac*N*K) largest-|G| weights."""
    lib = load_library()
    _require_cuda(W, "W"); _require_cuda(G, "G")
    if W.dtype != torch.float16 or G.dtype != torch.float32 or W.shape != G.shape or W.dim() != 2:
        raise ValueError("W must be fp16 [N,K] and G fp32 [N,K]")
    N, K = W.shape
    out = C.POINTER(gwq_outliers)()
    with torch.cuda.device(W.device):
        st = lib.gwq_select_outliers(W.data_ptr(), G.data_ptr(), N, K, float(frac), C.byref(out), _stream_ptr())
    _check(st, "gwq_select_outliers")
    return Outliers(out, W.device)


def gwq_select_outliers_static(W: torch.Tensor, G: torch.Tensor, frac: float, row_ptr: torch.Tensor,
                               col_idx: torch.Tensor, val: torch.Tensor) -> int:
    """Selection into caller-owned device tensors (row_ptr int32 [N+1], col_idx int32 [cap],
    val int16 [cap]) without any device allocation inside the library; returns nnz.
    For processes whose device memory is fully owned by their own pool, or that may not
    take the stall of a cudaMalloc.  Calls must not overlap on one GPU; N <= 32768."""
    lib = load_library()
    for t, name in ((W, "W"), (G, "G"), (row_ptr, "row_ptr"), (col_idx, "col_idx"), (val, "val")):
        _require_cuda(t, name)
    N, K = W.shape
    if row_ptr.dtype != torch.int32 or col_idx.dtype != torch.int32 or val.element_size() != 2:
        raise ValueError("row_ptr / col_idx must be int32 and val 16-bit")
    if row_ptr.numel() < N + 1:
        raise ValueError("row_ptr too short")
    cap = min(col_idx.numel(), val.numel())
    nnz = C.c_int64(0)
    with torch.cuda.device(W.device):
        st = lib.gwq_select_outliers_static(W.data_ptr(), G.data_ptr(), N, K, float(frac), row_ptr.data_ptr(),
                                            col_idx.data_ptr(), val.data_ptr(), cap, C.byref(nnz), _stream_ptr())
    _check(st, "gwq_select_outliers_static")
    return int(nnz.value)


def gwq_outliers_rows(S: Outliers, row0: int, row1: int) -> Outliers:
    """Rows [row0, row1) of S as an outlier matrix of its own (for a layer whose rows are split over ranks)."""
    out = C.POINTER(gwq_outliers)()
    with torch.cuda.device(S.device):
        st = load_library().gwq_outliers_rows(S._h, int(row0), int(row1), C.byref(out), _stream_ptr())
    _check(st, "gwq_outliers_rows")
    return Outliers(out, S.device)


def gwq_pack(W: torch.Tensor, S: Outliers, bits: int, group: int) -> Packed:
    """Quantize the non-outliers of W and pack; S is consumed (owned by the result)."""
    lib = load_library()
    _require_cuda(W, "W")
    if W.dtype != torch.float16 or W.dim() != 2:
        raise ValueError("W must be fp16 [N,K]")
    N, K = W.shape
    out = C.POINTER(gwq_packed)()
    with torch.cuda.device(W.device):
        st = lib.gwq_pack(W.data_ptr(), S._h, N, K, int(bits), int(group), C.byref(out), _stream_ptr())
    _check(st, "gwq_pack")
    S._h = None  # ownership moved
    return Packed(out, W.device)


def gwq_linear(P: Packed, x: torch.Tensor, out_dtype: torch.dtype | None = None,
               out: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """y = x (deq(Wq) + S)^T for x [M,K] fp16/bf16 on the GPU; asynchronous on the current stream.
    Where the product needs scratch memory (gwq_linear_workspace_bytes > 0) it is taken from `workspace`
    (a CUDA uint8 tensor) or, by default, from a new torch tensor: the library itself never allocates here."""
    lib = load_library()
    _require_cuda(x, "x")
    if x.dim() != 2 or x.shape[1] != P.K:
        raise ValueError("x must be [M, K]")
    M = x.shape[0]
    if out is None:
        out = torch.empty((M, P.N), dtype=out_dtype or x.dtype, device=x.device)
    else:
        _require_cuda(out, "out")
    xd = _dtype_code(x.dtype)
    need = 0 if xd == GWQ_F32 else int(lib.gwq_linear_workspace_bytes(P._h, xd, M))
    if need > 0 and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
    if workspace is not None:
        st = lib.gwq_linear_ws(P._h, x.data_ptr(), xd, M, out.data_ptr(), _dtype_code(out.dtype),
                               workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream_ptr())
    else:
        st = lib.gwq_linear(P._h, x.data_ptr(), xd, M, out.data_ptr(), _dtype_code(out.dtype), _stream_ptr())
    _check(st, "gwq_linear")
    return out


def gwq_linear_multi(Ps, x: torch.Tensor, out_dtype: torch.dtype | None = None, outs=None,
                     workspace: torch.Tensor | None = None):
    """[x (deq(P) + S_P)^T for P in Ps] for layers that read the same x [M,K]: one call, and for M <= 32 one launch."""
    lib = load_library()
    _require_cuda(x, "x")
    n = len(Ps)
    if x.dim() != 2 or any(P.K != x.shape[1] for P in Ps):
        raise ValueError("x must be [M, K] with the K of every layer")
    M = x.shape[0]
    if outs is None:
        outs = [torch.empty((M, P.N), dtype=out_dtype or x.dtype, device=x.device) for P in Ps]
    for o in outs:
        _require_cuda(o, "out")
    if len(outs) != n or any(o.dtype != outs[0].dtype for o in outs):
        raise ValueError("one output per layer, all of one dtype")
    xd = _dtype_code(x.dtype)
    need = 0 if xd == GWQ_F32 else max(int(lib.gwq_linear_workspace_bytes(P._h, xd, M)) for P in Ps)
    if need > 0:   # products that take scratch memory: one call per layer, all on the same workspace (stream order)
        if workspace is None or workspace.numel() * workspace.element_size() < need:
            workspace = torch.empty(need, dtype=torch.uint8, device=x.device)
        for P, o in zip(Ps, outs):
            gwq_linear(P, x, out=o, workspace=workspace)
        return outs
    handles = (C.POINTER(gwq_packed) * max(n, 1))(*[P._h for P in Ps])
    ys = (C.c_void_p * max(n, 1))(*[o.data_ptr() for o in outs])
    st = lib.gwq_linear_multi(handles, n, x.data_ptr(), _dtype_code(x.dtype), M, ys,
                              _dtype_code(outs[0].dtype) if outs else GWQ_F16, _stream_ptr())
    _check(st, "gwq_linear_multi")
    return outs


def gwq_gradient_mean(Gs, out: torch.Tensor | None = None) -> torch.Tensor:
    """FP32 mean of the gradients of several calibration samples (same shape, on the GPU), added in list order."""
    if len(Gs) < 1:
        raise ValueError("at least one gradient")
    for G in Gs:
        _require_cuda(G, "G")
        if G.dtype != torch.float32 or G.shape != Gs[0].shape or not G.is_contiguous():
            raise ValueError("gradients must be contiguous fp32 tensors of one shape")
    if out is None:
        out = torch.empty_like(Gs[0])
    ptrs = (C.c_void_p * len(Gs))(*[G.data_ptr() for G in Gs])
    with torch.cuda.device(Gs[0].device):
        st = load_library().gwq_gradient_mean(ptrs, len(Gs), Gs[0].numel(), out.data_ptr(), _stream_ptr())
    _check(st, "gwq_gradient_mean")
    return out


def gwq_quality(W: torch.Tensor, G: torch.Tensor, P: Packed):
    """(||W - W_Q||^2, g^T (W - W_Q)) of the packed layer P against W fp16 [N,K] and G fp32 [N,K] on the GPU."""
    _require_cuda(W, "W")
    _require_cuda(G, "G")
    if W.dtype != torch.float16 or G.dtype != torch.float32 or tuple(W.shape) != (P.N, P.K) or W.shape != G.shape:
        raise ValueError("W must be fp16 [N,K] and G fp32 [N,K] of the layer's shape")
    if not (W.is_contiguous() and G.is_contiguous()):
        raise ValueError("W and G must be contiguous")
    a, b = C.c_double(0.0), C.c_double(0.0)
    with torch.cuda.device(P.device):
        st = load_library().gwq_quality(W.data_ptr(), G.data_ptr(), P._h, C.byref(a), C.byref(b), _stream_ptr())
    _check(st, "gwq_quality")
    return float(a.value), float(b.value)


def gwq_linear_host(P: Packed, x_host: torch.Tensor, y_host: torch.Tensor) -> torch.Tensor:
    """Same product with HOST tensors (ideally pinned); copies in, computes, copies out, synchronises."""
    lib = load_library()
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("gwq_linear_host takes host tensors")
    M = x_host.shape[0]
    with torch.cuda.device(P.device):
        st = lib.gwq_linear_host(P._h, x_host.data_ptr(), _dtype_code(x_host.dtype), M, y_host.data_ptr(),
                                 _dtype_code(y_host.dtype), _stream_ptr())
    _check(st, "gwq_linear_host")
    return y_host


def gwq_linear_host_async(P: Packed, x_host: torch.Tensor, y_host: torch.Tensor) -> torch.Tensor:
    """gwq_linear_host without the synchronisation: y_host is valid after the current stream has been synchronised."""
    lib = load_library()
    if x_host.is_cuda or y_host.is_cuda:
        raise ValueError("gwq_linear_host_async takes host tensors")
    M = x_host.shape[0]
    with torch.cuda.device(P.device):
        st = lib.gwq_linear_host_async(P._h, x_host.data_ptr(), _dtype_code(x_host.dtype), M, y_host.data_ptr(),
                                       _dtype_code(y_host.dtype), _stream_ptr())
    _check(st, "gwq_linear_host_async")
    return y_host


def gwq_device_status(P: Packed) -> int:
    """Status recorded by the kernels of earlier gwq_linear calls on P (0 = ok); synchronises."""
    with torch.cuda.device(P.device):
        return int(load_library().gwq_device_status(P._h, _stream_ptr()))


def gwq_set_wait_limit(P: Packed, cycles: int) -> None:
    """SM cycles a bounded device-side wait may spin before the kernel gives up (negative: the default)."""
    _check(int(load_library().gwq_set_wait_limit(P._h, int(cycles))), "gwq_set_wait_limit")


def gwq_free(obj) -> None:
    obj.free()
