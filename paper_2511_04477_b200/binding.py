"""Thin Python binding of the C ABI in ``include/spqt.h``.

Argument marshalling only: every function takes torch CUDA tensors (device
memory and streams are PyTorch's job), checks dtypes, passes raw pointers to the
entry point of the same name and raises :class:`SpqtError` on a non-zero status.
No arithmetic of the method happens in Python and there is no CPU fallback: if
``libspqt.so`` has not been built, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspqt.so")

EXPORTS = (
    "spqt_status_string", "spqt_version", "spqt_packed_sizes", "spqt_pack", "spqt_unpack",
    "spqt_sparsify", "spqt_sparse_gemv", "spqt_sparse_gemv_static", "spqt_static_status", "spqt_sparsify_gemv", "spqt_dense_gemv",
    "spqt_sparse_linear_host", "spqt_sparse_linear_host_async", "spqt_host_step_create", "spqt_host_step_launch", "spqt_host_step_destroy", "spqt_gemm_small_workspace", "spqt_sparse_gemm_small", "spqt_dense_gemm_small", "spqt_rowwise_packed_sizes", "spqt_rowwise_pack", "spqt_rowwise_dense_gemv", "spqt_rowwise_thresholded_gemv", "spqt_kq_packed_sizes", "spqt_kq_pack", "spqt_kq_sparse_gemv", "spqt_kq_dense_gemv", "spqt_kqw_packed_sizes", "spqt_kqw_pack", "spqt_kqw_sparse_gemv", "spqt_kqw_dense_gemv", "spqt_autotune", "spqt_calibrate_threshold", "spqt_set_tuning", "spqt_set_debug", "spqt_workspace_status", "spqt_probe_read", "spqt_probe_arith", "spqt_launch_count",
)

_lib = None


class SpqtError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s failed: %s (%d)" % (where, status_string(status), status))


def lib() -> ctypes.CDLL:
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libspqt.so is missing: build it with `python -m paper_2511_04477_b200.build` "
                "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.spqt_status_string.restype = ctypes.c_char_p
        L.spqt_status_string.argtypes = [i32]
        L.spqt_version.restype = i32
        L.spqt_packed_sizes.argtypes = [i32, i32, i32, i32] + [ctypes.POINTER(sz)] * 3
        L.spqt_pack.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp]
        L.spqt_unpack.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.spqt_sparsify.argtypes = [vp, i32, ctypes.c_float, vp, vp, vp]
        L.spqt_sparse_gemv.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.spqt_sparse_gemv_static.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
        L.spqt_sparse_gemv_static.restype = i32
        L.spqt_static_status.argtypes = [i32, i32, ctypes.POINTER(i32), vp]
        L.spqt_static_status.restype = i32
        L.spqt_sparsify_gemv.argtypes = [vp, vp, i32, i32, i32, i32, vp, ctypes.c_float, vp, vp, vp, vp, sz, vp]
        L.spqt_sparsify_gemv.restype = i32
        L.spqt_dense_gemv.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.spqt_rowwise_packed_sizes.argtypes = [i32, i32, i32, i32] + [ctypes.POINTER(sz)] * 2
        L.spqt_rowwise_pack.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp]
        L.spqt_rowwise_dense_gemv.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp]
        L.spqt_rowwise_thresholded_gemv.argtypes = [vp, vp, i32, i32, i32, i32, vp, ctypes.c_float, vp, vp]
        L.spqt_kq_packed_sizes.argtypes = [i32, i32] + [ctypes.POINTER(sz)] * 2
        L.spqt_kq_pack.argtypes = [vp, i32, i32, i32, vp, vp]
        L.spqt_kq_sparse_gemv.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.spqt_kq_dense_gemv.argtypes = [vp, i32, i32, vp, vp, vp, sz, vp]
        L.spqt_kqw_packed_sizes.argtypes = [i32, i32, i32] + [ctypes.POINTER(sz)] * 2
        L.spqt_kqw_pack.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.spqt_kqw_sparse_gemv.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, sz, vp]
        L.spqt_kqw_dense_gemv.argtypes = [vp, i32, i32, i32, vp, vp, vp, sz, vp]
        for name in ("spqt_kqw_packed_sizes", "spqt_kqw_pack", "spqt_kqw_sparse_gemv", "spqt_kqw_dense_gemv"):
            getattr(L, name).restype = i32
        L.spqt_sparse_linear_host.argtypes = [vp, vp, i32, i32, i32, i32, vp, ctypes.c_float, vp,
                                              vp, vp, vp, vp, vp, sz, vp]
        L.spqt_sparse_linear_host_async.argtypes = L.spqt_sparse_linear_host.argtypes
        L.spqt_host_step_create.argtypes = [vp, i32, ctypes.POINTER(vp)]
        L.spqt_host_step_launch.argtypes = [vp, vp]
        L.spqt_host_step_destroy.argtypes = [vp]
        L.spqt_gemm_small_workspace.argtypes = [i32, i32, i32, i32, ctypes.POINTER(sz)]
        L.spqt_gemm_small_workspace.restype = i32
        L.spqt_sparse_gemm_small.argtypes = [vp, vp, i32, i32, i32, i32, vp, i32, i32, ctypes.c_float, vp, vp, vp, i32, vp, sz, vp]
        L.spqt_sparse_gemm_small.restype = i32
        L.spqt_dense_gemm_small.argtypes = [vp, vp, i32, i32, i32, i32, vp, i32, i32, vp, i32, vp, sz, vp]
        L.spqt_dense_gemm_small.restype = i32
        L.spqt_autotune.argtypes = [vp, vp, i32, i32, i32, i32, vp, ctypes.c_float, vp, vp, vp, vp, sz, vp, sz,
                                    ctypes.POINTER(i32), ctypes.POINTER(i32), vp]
        L.spqt_autotune.restype = i32
        L.spqt_calibrate_threshold.argtypes = [vp, sz, ctypes.c_double, vp, vp, sz, vp]
        L.spqt_calibrate_threshold.restype = i32
        L.spqt_set_tuning.argtypes = [i32, i32]
        L.spqt_set_debug.argtypes = [i32]
        L.spqt_probe_read.argtypes = [vp, sz, i32, vp, vp]
        L.spqt_probe_arith.argtypes = [i32, vp, sz, ctypes.POINTER(ctypes.c_ulonglong), vp]
        L.spqt_probe_arith.restype = i32
        L.spqt_workspace_status.argtypes = [vp, i32, i32, ctypes.POINTER(i32), vp]
        L.spqt_launch_count.restype = ctypes.c_ulonglong
        for name in ("spqt_packed_sizes", "spqt_pack", "spqt_unpack", "spqt_sparsify",
                     "spqt_sparse_gemv", "spqt_dense_gemv", "spqt_sparse_linear_host", "spqt_set_tuning",
                     "spqt_set_debug", "spqt_workspace_status", "spqt_probe_read"):
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().spqt_status_string(int(status)).decode()


def _ok(status: int, where: str) -> None:
    if status != 0:
        raise SpqtError(status, where)


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype:
        raise TypeError("%s must be %s, got %s" % (name, dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t.data_ptr()


@dataclass
class PackedSizes:
    codes_bytes: int
    scale_zero_bytes: int
    gemv_workspace_bytes: int


def spqt_packed_sizes(m: int, n: int, bits: int = 4, group: int = 128) -> PackedSizes:
    out = [ctypes.c_size_t(0) for _ in range(3)]
    _ok(lib().spqt_packed_sizes(m, n, bits, group, *[ctypes.byref(o) for o in out]), "spqt_packed_sizes")
    return PackedSizes(*[int(o.value) for o in out])


@dataclass
class Packed:
    """Device buffers written by :func:`spqt_pack` (zigzag layout)."""
    codes: torch.Tensor        # uint8[R*n*B]
    scale_zero: torch.Tensor   # float16[2*R*n]: (scale, zero) of block (r,k) at 2*(r*n+k)
    m: int
    n: int
    bits: int
    group: int

    @property
    def scales(self) -> torch.Tensor:
        """float16[R*n], a strided view of scale_zero."""
        return self.scale_zero[0::2]

    @property
    def zeros(self) -> torch.Tensor:
        """float16[R*n], a strided view of scale_zero."""
        return self.scale_zero[1::2]

    @property
    def nbytes(self) -> int:
        return self.codes.numel() + 2 * self.scale_zero.numel()


def new_workspace(m: int, n: int, bits: int = 4, group: int = 128, device=None) -> torch.Tensor:
    """Zeroed GEMV workspace (zeroed once; every call leaves it ready for the next)."""
    sz = spqt_packed_sizes(m, n, bits, group).gemv_workspace_bytes
    return torch.zeros(sz, dtype=torch.uint8, device=device or "cuda")


def spqt_pack(W: torch.Tensor, bits: int = 4, group: int = 128, stream=None) -> Packed:
    if W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be 2-D with unit column stride")
    if not W.is_cuda or W.dtype != torch.float16:
        raise TypeError("W must be a CUDA float16 tensor")
    m, n = W.shape
    sz = spqt_packed_sizes(m, n, bits, group)
    codes = torch.empty(sz.codes_bytes, dtype=torch.uint8, device=W.device)
    scale_zero = torch.empty(sz.scale_zero_bytes // 2, dtype=torch.float16, device=W.device)
    _ok(lib().spqt_pack(W.data_ptr(), m, n, W.stride(0), bits, group, codes.data_ptr(),
                        scale_zero.data_ptr(), _stream(stream)), "spqt_pack")
    return Packed(codes, scale_zero, m, n, bits, group)


def spqt_unpack(p: Packed, stream=None) -> torch.Tensor:
    q = torch.empty((p.m, p.n), dtype=torch.uint8, device=p.codes.device)
    _ok(lib().spqt_unpack(_dev(p.codes, torch.uint8, "codes"), p.m, p.n, p.bits, p.group,
                          q.data_ptr(), _stream(stream)), "spqt_unpack")
    return q


def spqt_sparsify(x: torch.Tensor, t: float, idx: torch.Tensor = None, count: torch.Tensor = None,
                  stream=None):
    """-> (idx int32[n] of which the first count[0] entries are valid, count int32[1]), both on the device."""
    n = x.numel()
    if idx is None:
        idx = torch.empty(max(n, 1), dtype=torch.int32, device=x.device)
    if count is None:
        count = torch.empty(1, dtype=torch.int32, device=x.device)
    if idx.numel() < n:
        raise ValueError("idx must hold n entries")
    _ok(lib().spqt_sparsify(_dev(x, torch.float16, "x"), n, float(t), _dev(idx, torch.int32, "idx"),
                            _dev(count, torch.int32, "count"), _stream(stream)), "spqt_sparsify")
    return idx, count


def spqt_sparse_gemv(p: Packed, x: torch.Tensor, idx: torch.Tensor, count: torch.Tensor,
                     workspace: torch.Tensor, y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    if x.numel() != p.n or y.numel() != p.m:
        raise ValueError("x must have n entries and y m entries")
    _ok(lib().spqt_sparse_gemv(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"),
        p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), _dev(idx, torch.int32, "idx"), _dev(count, torch.int32, "count"),
        _dev(y, torch.float16, "y"), _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
        _stream(stream)), "spqt_sparse_gemv")
    return y


def spqt_sparse_gemv_static(p: Packed, x: torch.Tensor, idx: torch.Tensor, count: torch.Tensor,
                            y: torch.Tensor, stream=None) -> torch.Tensor:
    """The sparse GEMV on the library's built-in 1 MiB scratch, for callers that may not allocate
    device memory: nothing is allocated here either, so ``y`` must be passed in.  Calls on one
    device share the scratch and must not overlap on the GPU."""
    if x.numel() != p.n or y.numel() != p.m:
        raise ValueError("x must have n entries and y m entries")
    _ok(lib().spqt_sparse_gemv_static(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"),
        p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), _dev(idx, torch.int32, "idx"), _dev(count, torch.int32, "count"),
        _dev(y, torch.float16, "y"), _stream(stream)), "spqt_sparse_gemv_static")
    return y


def spqt_sparsify_gemv(p: Packed, x: torch.Tensor, t: float, workspace: torch.Tensor,
                       idx: torch.Tensor = None, count: torch.Tensor = None, y: torch.Tensor = None, stream=None):
    """Index collection and sparse GEMV in one launch -> (y, idx, count)."""
    if idx is None:
        idx = torch.empty(p.n, dtype=torch.int32, device=x.device)
    if count is None:
        count = torch.empty(1, dtype=torch.int32, device=x.device)
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    if x.numel() != p.n or y.numel() != p.m or idx.numel() < p.n:
        raise ValueError("x and idx must have n entries and y m entries")
    _ok(lib().spqt_sparsify_gemv(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"),
        p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), float(t), _dev(idx, torch.int32, "idx"), _dev(count, torch.int32, "count"),
        _dev(y, torch.float16, "y"), _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
        _stream(stream)), "spqt_sparsify_gemv")
    return y, idx, count


def spqt_dense_gemv(p: Packed, x: torch.Tensor, workspace: torch.Tensor, y: torch.Tensor = None,
                    stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    if x.numel() != p.n or y.numel() != p.m:
        raise ValueError("x must have n entries and y m entries")
    _ok(lib().spqt_dense_gemv(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"),
        p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)), "spqt_dense_gemv")
    return y


class HostLinear:
    """Staging buffers for :func:`spqt_sparse_linear_host`: pinned host x / y and
    device x, idx, count, y for one packed matrix."""

    def __init__(self, p: Packed, workspace: torch.Tensor = None):
        dev = p.codes.device
        self.p = p
        self.x_host = torch.empty(p.n, dtype=torch.float16).pin_memory()
        self.y_host = torch.empty(p.m, dtype=torch.float16).pin_memory()
        self.x_dev = torch.empty(p.n, dtype=torch.float16, device=dev)
        self.idx = torch.empty(p.n, dtype=torch.int32, device=dev)
        self.count = torch.zeros(1, dtype=torch.int32, device=dev)
        self.y_dev = torch.empty(p.m, dtype=torch.float16, device=dev)
        self.workspace = workspace if workspace is not None else new_workspace(p.m, p.n, p.bits, p.group, dev)


def spqt_sparse_linear_host(h: HostLinear, t: float, stream=None, wait: bool = True) -> torch.Tensor:
    """x in ``h.x_host`` -> y in ``h.y_host`` (copies, index collection, sparse GEMV; with ``wait`` the call
    returns when y is there, otherwise once everything is enqueued and the caller synchronises the stream)."""
    p = h.p
    fn = lib().spqt_sparse_linear_host if wait else lib().spqt_sparse_linear_host_async
    _ok(fn(
        p.codes.data_ptr(), p.scale_zero.data_ptr(), p.m, p.n, p.bits, p.group,
        h.x_host.data_ptr(), float(t), h.y_host.data_ptr(), h.x_dev.data_ptr(), h.idx.data_ptr(),
        h.count.data_ptr(), h.y_dev.data_ptr(), h.workspace.data_ptr(), h.workspace.numel(),
        _stream(stream)), "spqt_sparse_linear_host")
    return h.y_host


class _HostLinearDesc(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scale_zero", ctypes.c_void_p), ("m", ctypes.c_int), ("n", ctypes.c_int),
                ("bits", ctypes.c_int), ("group", ctypes.c_int), ("x_host", ctypes.c_void_p), ("t", ctypes.c_float),
                ("y_host", ctypes.c_void_p), ("x_dev", ctypes.c_void_p), ("idx_dev", ctypes.c_void_p),
                ("count_dev", ctypes.c_void_p), ("y_dev", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t)]


class HostStep:
    """The host-buffer linears of a token step (``HostLinear`` objects and their thresholds) recorded once by
    spqt_host_step_create; :meth:`launch` replays them with one call (asynchronous: synchronise the stream before
    reading the ``y_host`` buffers).  Keeps the ``HostLinear`` objects alive."""

    def __init__(self, hs, ts):
        self.hs = list(hs)
        arr = (_HostLinearDesc * len(self.hs))()
        for d, h, t in zip(arr, self.hs, ts):
            p = h.p
            d.codes, d.scale_zero, d.m, d.n, d.bits, d.group = p.codes.data_ptr(), p.scale_zero.data_ptr(), p.m, p.n, p.bits, p.group
            d.x_host, d.t, d.y_host = h.x_host.data_ptr(), float(t), h.y_host.data_ptr()
            d.x_dev, d.idx_dev, d.count_dev, d.y_dev = h.x_dev.data_ptr(), h.idx.data_ptr(), h.count.data_ptr(), h.y_dev.data_ptr()
            d.workspace, d.workspace_bytes = h.workspace.data_ptr(), h.workspace.numel()
        self.handle = ctypes.c_void_p(None)
        _ok(lib().spqt_host_step_create(ctypes.cast(arr, ctypes.c_void_p), len(self.hs), ctypes.byref(self.handle)), "spqt_host_step_create")

    def launch(self, stream=None) -> None:
        _ok(lib().spqt_host_step_launch(self.handle, _stream(stream)), "spqt_host_step_launch")

    def close(self) -> None:
        if self.handle:
            lib().spqt_host_step_destroy(self.handle)
            self.handle = ctypes.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def spqt_probe_read(buf: torch.Tensor, pattern: int, moved: torch.Tensor, stream=None) -> None:
    """Measurement aid: stream `buf` into shared memory in 64-byte blocks (pattern 0: all of them, 1: one random
    half of every 128-byte line); adds the bytes fetched to `moved` (int64[1] on the device)."""
    _ok(lib().spqt_probe_read(_dev(buf, torch.uint8, "buf"), buf.numel(), int(pattern),
                              _dev(moved, torch.int64, "moved"), _stream(stream)), "spqt_probe_read")


def spqt_probe_arith(chunks_per_warp: int, sink: torch.Tensor, stream=None) -> int:
    """Measurement aid: the GEMV loop's arithmetic alone on shared-memory operands (16 warps per SM, `chunks_per_warp`
    2 KB chunks each); `sink` is float32 on the device, at least 512 values per SM.  Returns the chunks processed."""
    total = ctypes.c_ulonglong(0)
    _ok(lib().spqt_probe_arith(int(chunks_per_warp), _dev(sink, torch.float32, "sink"), sink.numel(), ctypes.byref(total),
                               _stream(stream)), "spqt_probe_arith")
    return int(total.value)


def spqt_set_debug(on: bool) -> None:
    """Checked mode: validate idx/count on the device before every sparse GEMV (off by default)."""
    _ok(lib().spqt_set_debug(1 if on else 0), "spqt_set_debug")


def new_gemm_small_workspace(p: Packed) -> torch.Tensor:
    """Zeroed workspace of the small-batch calls (zeroed once; every call leaves it ready for the next)."""
    out = ctypes.c_size_t(0)
    _ok(lib().spqt_gemm_small_workspace(p.m, p.n, p.bits, p.group, ctypes.byref(out)), "spqt_gemm_small_workspace")
    return torch.zeros(int(out.value), dtype=torch.uint8, device=p.codes.device)


def _batch(p: Packed, X: torch.Tensor, Y: torch.Tensor):
    if X.dim() != 2 or X.stride(1) != 1 or X.shape[1] != p.n or not (1 <= X.shape[0] <= 8):
        raise ValueError("X must be [batch <= 8][n] with unit column stride")
    if Y is None:
        Y = torch.empty((X.shape[0], p.m), dtype=torch.float16, device=X.device)
    if Y.dtype != torch.float16 or X.dtype != torch.float16 or not X.is_cuda or not Y.is_cuda:
        raise TypeError("X and Y must be CUDA float16 tensors")
    if Y.shape != (X.shape[0], p.m) or Y.stride(1) != 1:
        raise ValueError("Y must be [batch][m] with unit column stride")
    return Y


def spqt_sparse_gemm_small(p: Packed, X: torch.Tensor, t: float, workspace: torch.Tensor, idx: torch.Tensor = None,
                           count: torch.Tensor = None, Y: torch.Tensor = None, stream=None):
    """2..8 decode rows over the union of their active sets -> (Y [batch][m], idx, count)."""
    Y = _batch(p, X, Y)
    if idx is None:
        idx = torch.empty(p.n, dtype=torch.int32, device=X.device)
    if count is None:
        count = torch.empty(1, dtype=torch.int32, device=X.device)
    _ok(lib().spqt_sparse_gemm_small(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"), p.m, p.n, p.bits, p.group,
        X.data_ptr(), X.stride(0), X.shape[0], float(t), _dev(idx, torch.int32, "idx"), _dev(count, torch.int32, "count"),
        Y.data_ptr(), Y.stride(0), _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)),
        "spqt_sparse_gemm_small")
    return Y, idx, count


def spqt_dense_gemm_small(p: Packed, X: torch.Tensor, workspace: torch.Tensor, Y: torch.Tensor = None, stream=None):
    Y = _batch(p, X, Y)
    _ok(lib().spqt_dense_gemm_small(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"), p.m, p.n, p.bits, p.group,
        X.data_ptr(), X.stride(0), X.shape[0], Y.data_ptr(), Y.stride(0),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)), "spqt_dense_gemm_small")
    return Y


@dataclass
class RowwisePacked:
    """Device buffers written by :func:`spqt_rowwise_pack` (the row-wise comparison layout)."""
    codes: torch.Tensor        # uint8[m*n/2]
    scale_zero: torch.Tensor   # float16[2*m*n/group]
    m: int
    n: int
    bits: int
    group: int

    @property
    def scales(self) -> torch.Tensor:
        return self.scale_zero[0::2]

    @property
    def zeros(self) -> torch.Tensor:
        return self.scale_zero[1::2]


def spqt_rowwise_packed_sizes(m: int, n: int, bits: int = 4, group: int = 128):
    out = [ctypes.c_size_t(0) for _ in range(2)]
    _ok(lib().spqt_rowwise_packed_sizes(m, n, bits, group, *[ctypes.byref(o) for o in out]), "spqt_rowwise_packed_sizes")
    return int(out[0].value), int(out[1].value)


def spqt_rowwise_pack(W: torch.Tensor, bits: int = 4, group: int = 128, stream=None) -> RowwisePacked:
    if W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be 2-D with unit column stride")
    if not W.is_cuda or W.dtype != torch.float16:
        raise TypeError("W must be a CUDA float16 tensor")
    m, n = W.shape
    cb, sb = spqt_rowwise_packed_sizes(m, n, bits, group)
    codes = torch.empty(cb, dtype=torch.uint8, device=W.device)
    scale_zero = torch.empty(sb // 2, dtype=torch.float16, device=W.device)
    _ok(lib().spqt_rowwise_pack(W.data_ptr(), m, n, W.stride(0), bits, group, codes.data_ptr(),
                                scale_zero.data_ptr(), _stream(stream)), "spqt_rowwise_pack")
    return RowwisePacked(codes, scale_zero, m, n, bits, group)


def spqt_rowwise_dense_gemv(p: RowwisePacked, x: torch.Tensor, y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_rowwise_dense_gemv(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"), p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"), _stream(stream)), "spqt_rowwise_dense_gemv")
    return y


@dataclass
class KqPacked:
    """Device buffer written by :func:`spqt_kq_pack` (144-byte records of the two-level format, zigzag order)."""
    records: torch.Tensor      # uint8[(m/256)*n*144]  (80, 176, 208 or 272 bytes per record with 2-, 5-, 6- or 8-bit codes)
    m: int
    n: int
    bits: int = 4


def spqt_kq_packed_sizes(m: int, n: int):
    out = [ctypes.c_size_t(0) for _ in range(2)]
    _ok(lib().spqt_kq_packed_sizes(m, n, *[ctypes.byref(o) for o in out]), "spqt_kq_packed_sizes")
    return int(out[0].value), int(out[1].value)


def spqt_kq_pack(W: torch.Tensor, stream=None) -> KqPacked:
    if W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be 2-D with unit column stride")
    if not W.is_cuda or W.dtype != torch.float16:
        raise TypeError("W must be a CUDA float16 tensor")
    m, n = W.shape
    rb, _ = spqt_kq_packed_sizes(m, n)
    records = torch.empty(rb, dtype=torch.uint8, device=W.device)
    _ok(lib().spqt_kq_pack(W.data_ptr(), m, n, W.stride(0), records.data_ptr(), _stream(stream)), "spqt_kq_pack")
    return KqPacked(records, m, n)


def spqt_kqw_packed_sizes(m: int, n: int, bits: int):
    out = [ctypes.c_size_t(0) for _ in range(2)]
    _ok(lib().spqt_kqw_packed_sizes(m, n, bits, *[ctypes.byref(o) for o in out]), "spqt_kqw_packed_sizes")
    return int(out[0].value), int(out[1].value)


def spqt_kqw_pack(W: torch.Tensor, bits: int, stream=None) -> KqPacked:
    """The two-level format with 2-, 4-, 5-, 6- or 8-bit codes."""
    if W.dim() != 2 or W.stride(1) != 1:
        raise ValueError("W must be 2-D with unit column stride")
    if not W.is_cuda or W.dtype != torch.float16:
        raise TypeError("W must be a CUDA float16 tensor")
    m, n = W.shape
    rb, _ = spqt_kqw_packed_sizes(m, n, bits)
    records = torch.empty(rb, dtype=torch.uint8, device=W.device)
    _ok(lib().spqt_kqw_pack(W.data_ptr(), m, n, W.stride(0), bits, records.data_ptr(), _stream(stream)), "spqt_kqw_pack")
    return KqPacked(records, m, n, bits)


def spqt_kqw_sparse_gemv(p: KqPacked, x: torch.Tensor, idx: torch.Tensor, count: torch.Tensor, workspace: torch.Tensor,
                         y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_kqw_sparse_gemv(
        _dev(p.records, torch.uint8, "records"), p.m, p.n, p.bits, _dev(x, torch.float16, "x"),
        _dev(idx, torch.int32, "idx"), _dev(count, torch.int32, "count"), _dev(y, torch.float16, "y"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)), "spqt_kqw_sparse_gemv")
    return y


def spqt_kqw_dense_gemv(p: KqPacked, x: torch.Tensor, workspace: torch.Tensor, y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_kqw_dense_gemv(
        _dev(p.records, torch.uint8, "records"), p.m, p.n, p.bits, _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)), "spqt_kqw_dense_gemv")
    return y


def new_kq_workspace(p: KqPacked) -> torch.Tensor:
    """Zeroed GEMV workspace for the two-level format (zeroed once; every call leaves it ready for the next)."""
    _, wb = spqt_kq_packed_sizes(p.m, p.n)
    return torch.zeros(wb, dtype=torch.uint8, device=p.records.device)


def spqt_kq_sparse_gemv(p: KqPacked, x: torch.Tensor, idx: torch.Tensor, count: torch.Tensor, workspace: torch.Tensor,
                        y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_kq_sparse_gemv(
        _dev(p.records, torch.uint8, "records"), p.m, p.n, _dev(x, torch.float16, "x"), _dev(idx, torch.int32, "idx"),
        _dev(count, torch.int32, "count"), _dev(y, torch.float16, "y"), _dev(workspace, torch.uint8, "workspace"),
        workspace.numel(), _stream(stream)), "spqt_kq_sparse_gemv")
    return y


def spqt_kq_dense_gemv(p: KqPacked, x: torch.Tensor, workspace: torch.Tensor, y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_kq_dense_gemv(
        _dev(p.records, torch.uint8, "records"), p.m, p.n, _dev(x, torch.float16, "x"), _dev(y, torch.float16, "y"),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(stream)), "spqt_kq_dense_gemv")
    return y


def spqt_rowwise_thresholded_gemv(p: RowwisePacked, x: torch.Tensor, t: float, y: torch.Tensor = None, stream=None) -> torch.Tensor:
    if y is None:
        y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    _ok(lib().spqt_rowwise_thresholded_gemv(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"), p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), float(t), _dev(y, torch.float16, "y"), _stream(stream)), "spqt_rowwise_thresholded_gemv")
    return y


def spqt_autotune(p: Packed, x: torch.Tensor, t: float, workspace: torch.Tensor, flush: torch.Tensor = None, stream=None):
    """Profile grid sizes for this shape and keep the fastest -> (ctas for the sparse calls, ctas for the dense call).
    ``flush``: an optional uint8 buffer larger than L2, rewritten before every timed launch.  Synchronises."""
    idx = torch.empty(p.n, dtype=torch.int32, device=x.device)
    count = torch.empty(1, dtype=torch.int32, device=x.device)
    y = torch.empty(p.m, dtype=torch.float16, device=x.device)
    a, b = ctypes.c_int(0), ctypes.c_int(0)
    _ok(lib().spqt_autotune(
        _dev(p.codes, torch.uint8, "codes"), _dev(p.scale_zero, torch.float16, "scale_zero"), p.m, p.n, p.bits, p.group,
        _dev(x, torch.float16, "x"), float(t), idx.data_ptr(), count.data_ptr(), y.data_ptr(),
        _dev(workspace, torch.uint8, "workspace"), workspace.numel(),
        flush.data_ptr() if flush is not None else None, flush.numel() if flush is not None else 0,
        ctypes.byref(a), ctypes.byref(b), _stream(stream)), "spqt_autotune")
    return int(a.value), int(b.value)


def new_calibration_workspace(device=None) -> torch.Tensor:
    """Zeroed histogram workspace of spqt_calibrate_threshold (zeroed once; every call leaves it zeroed)."""
    return torch.zeros(32768, dtype=torch.int32, device=device or "cuda")


def spqt_calibrate_threshold(x: torch.Tensor, sparsity: float, workspace: torch.Tensor = None,
                             threshold: torch.Tensor = None, stream=None) -> torch.Tensor:
    """Nearest-rank threshold of |x| over a pool of fp16 calibration activations -> float32[1] on the device."""
    if workspace is None:
        workspace = new_calibration_workspace(x.device)
    if threshold is None:
        threshold = torch.empty(1, dtype=torch.float32, device=x.device)
    _ok(lib().spqt_calibrate_threshold(
        _dev(x, torch.float16, "x") if x.numel() else None, x.numel(), float(sparsity),
        _dev(threshold, torch.float32, "threshold"), _dev(workspace, torch.int32, "workspace"), workspace.numel() * 4,
        _stream(stream)), "spqt_calibrate_threshold")
    return threshold


def spqt_set_tuning(gemv_ctas: int = 0, no_overlap: int = 0) -> None:
    _ok(lib().spqt_set_tuning(int(gemv_ctas), int(no_overlap)), "spqt_set_tuning")


def _status_word(rc: int, out: ctypes.c_int, where: str) -> int:
    # the call returns SPQT_ERR_TIMEOUT (6) / SPQT_ERR_INVALID_ARG (1) for a non-zero word it has read
    if out.value == -1 or rc not in (0, 1, 6):
        raise SpqtError(rc, where)
    return int(out.value)


def spqt_workspace_status(workspace: torch.Tensor, m: int, group: int = 128, stream=None) -> int:
    """The workspace's status word: 0, 1 (a bounded on-chip wait expired in a GEMV that used this workspace)
    or 2 (checked mode refused an index list).  Synchronises."""
    out = ctypes.c_int(-1)
    rc = lib().spqt_workspace_status(_dev(workspace, torch.uint8, "workspace"), m, group,
                                     ctypes.byref(out), _stream(stream))
    return _status_word(rc, out, "spqt_workspace_status")


def spqt_static_status(m: int, group: int = 128, stream=None) -> int:
    """Status word of the built-in scratch after the last spqt_sparse_gemv_static call (synchronises)."""
    out = ctypes.c_int(-1)
    rc = lib().spqt_static_status(m, group, ctypes.byref(out), _stream(stream))
    return _status_word(rc, out, "spqt_static_status")


def spqt_launch_count() -> int:
    return int(lib().spqt_launch_count())
