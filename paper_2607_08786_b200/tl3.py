"""Python binding of the C-ABI library declared in ``include/tl3.h``.

Argument marshalling only: every step of the SpMM runs in the library's CUDA kernels.  PyTorch
tensors serve as device memory and streams.  There is no CPU fallback -- if ``libtl3.so`` has not
been built, the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libtl3.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_NOT_UPLOADED, ERR_BAD_CONTAINER = -1, -2, -3, -4
ERR_CUDA, ERR_DEVICE_TIMEOUT, ERR_NO_MEMORY, ERR_SCRATCH_LIMIT = -5, -6, -7, -8
STATIC_SCRATCH_BYTES = 3 << 20

CANONICAL = ("tc_vals", "tc_meta", "chain_tau0", "chain_rho0", "chain_len", "pdd_bytes", "tile_dir",
             "res_rho", "res_val")
# the compact form of the Residual layer, derived from res_rho (numbered after the nine above)
COMPACT = ("res_dir", "res_list", "res_mask")
# the compact form of the Sparse-TC value array, derived from tc_vals (numbered after those)
COMPACT_VALUES = ("val_dir", "val_pack", "val_mask")
_CANONICAL_DTYPES = (np.uint16, np.uint8, np.uint16, np.uint16, np.uint8, np.uint8, np.uint32,
                     np.uint16, np.uint16, np.uint32, np.uint16, np.uint8, np.uint32, np.uint16, np.uint8)

# every symbol include/tl3.h declares
SYMBOLS = ("tl3_encode", "tl3_encode_device", "tl3_encode_device_only", "tl3_decode", "tl3_canonical", "tl3_stats", "tl3_serialize", "tl3_serialize_compact", "tl3_deserialize",
           "tl3_free", "tl3_device_bytes", "tl3_pack", "tl3_upload", "tl3_bind", "tl3_plan_device", "tl3_upload_device", "tl3_workspace_bytes", "tl3_workspace_init",
           "tl3_spmm", "tl3_spmm_ex", "tl3_spmm_nt", "tl3_spmm_host", "tl3_spmm_host_async", "tl3_spmm_static_scratch", "tl3_static_scratch_status", "tl3_status", "tl3_status_word", "tl3_selftest_bounded_wait", "tl3_last_launch", "tl3_strerror",
           "tl3_last_cuda_error", "tl3_get_tuning", "tl3_set_tuning")


class Tl3Error(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().tl3_strerror(code).decode()
        if code == ERR_CUDA:
            msg += f" (cudaError {lib().tl3_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


class Params(ctypes.Structure):
    _fields_ = [("tile_m", ctypes.c_int32), ("tile_k", ctypes.c_int32), ("maxd", ctypes.c_int32)]


class Tuning(ctypes.Structure):
    _fields_ = [("decode_before_x", ctypes.c_int32)]


class Epilogue(ctypes.Structure):
    _fields_ = [("bias", ctypes.c_void_p), ("activation", ctypes.c_int32)]


ACTIVATIONS = {None: 0, "none": 0, "relu": 1, "silu": 2, "gelu_tanh": 3}


class Stats(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("M", "K", "M_pad", "K_pad", "n_tiles", "nnz", "n_tc", "n_sf", "n_res", "n_dummy",
                 "n_slots_unused", "canonical_bytes", "device_bytes", "canonical_bytes_compact",
                 "dev_n_sf", "dev_n_res", "dev_n_dummy", "dev_pdd_bytes", "canonical_bytes_compact_all")]

    def as_dict(self) -> dict:
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def lib() -> ctypes.CDLL:
    """Loads ``libtl3.so``; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with "
                               "`python -m paper_2607_08786_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i64, sz, ci = ctypes.c_void_p, ctypes.c_int64, ctypes.c_size_t, ctypes.c_int
        L.tl3_encode.argtypes = [vp, i64, i64, ctypes.POINTER(Params), ctypes.POINTER(vp)]
        L.tl3_encode_device.argtypes = [vp, i64, i64, i64, vp, ctypes.POINTER(vp)]
        L.tl3_encode_device_only.argtypes = [vp, i64, i64, i64, vp, ctypes.POINTER(vp)]
        L.tl3_decode.argtypes = [vp, vp]
        L.tl3_canonical.argtypes = [vp, ci, ctypes.POINTER(vp), ctypes.POINTER(sz)]
        L.tl3_stats.argtypes = [vp, ctypes.POINTER(Stats)]
        L.tl3_serialize.argtypes = [vp, vp, ctypes.POINTER(sz)]
        L.tl3_serialize_compact.argtypes = [vp, vp, ctypes.POINTER(sz)]
        L.tl3_deserialize.argtypes = [vp, sz, ctypes.POINTER(vp)]
        L.tl3_free.argtypes = [vp]
        L.tl3_free.restype = None
        L.tl3_device_bytes.argtypes = [vp]
        L.tl3_device_bytes.restype = sz
        L.tl3_pack.argtypes = [vp, vp, sz]
        L.tl3_upload.argtypes = [vp, vp, vp]
        L.tl3_bind.argtypes = [vp, vp]
        L.tl3_plan_device.argtypes = [vp, vp]
        L.tl3_upload_device.argtypes = [vp, vp, vp]
        L.tl3_workspace_bytes.argtypes = [vp, ci]
        L.tl3_workspace_bytes.restype = sz
        L.tl3_workspace_init.argtypes = [vp, sz, vp]
        L.tl3_spmm.argtypes = [vp, vp, i64, vp, i64, ci, vp, vp]
        L.tl3_spmm_ex.argtypes = [vp, vp, i64, vp, i64, ci, ctypes.POINTER(Epilogue), vp, vp]
        L.tl3_spmm_nt.argtypes = [vp, vp, i64, vp, i64, ci, ctypes.POINTER(Epilogue), vp, vp]
        L.tl3_spmm_host.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp]
        L.tl3_spmm_host_async.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp]
        L.tl3_spmm_static_scratch.argtypes = [vp, vp, i64, vp, i64, ci, vp]
        L.tl3_static_scratch_status.argtypes = [vp]
        L.tl3_status.argtypes = [vp, vp, vp]
        L.tl3_status_word.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
        L.tl3_selftest_bounded_wait.argtypes = [vp, vp]
        L.tl3_last_launch.argtypes = [vp, ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci)]
        L.tl3_strerror.argtypes = [ci]
        L.tl3_strerror.restype = ctypes.c_char_p
        L.tl3_last_cuda_error.argtypes = []
        L.tl3_get_tuning.argtypes = [ctypes.POINTER(Tuning)]
        L.tl3_set_tuning.argtypes = [ctypes.POINTER(Tuning)]
        for name in SYMBOLS:
            fn = getattr(L, name)
            if name not in ("tl3_free", "tl3_device_bytes", "tl3_workspace_bytes", "tl3_strerror"):
                fn.restype = ci
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != OK:
        raise Tl3Error(code, where)


def _u16(a) -> np.ndarray:
    a = np.asarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    if a.dtype != np.uint16:
        raise TypeError("expected float16 or uint16 (fp16 bit patterns)")
    return np.ascontiguousarray(a)


def _stream_ptr(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return int(getattr(stream, "cuda_stream", stream))


class Matrix:
    """Handle of one encoded weight matrix (``tl3_matrix``)."""

    def __init__(self, handle: int):
        self._h = ctypes.c_void_p(handle)
        self._blob = None          # torch.uint8 tensor holding the device blob
        self._workspaces = {}

    # -- construction ------------------------------------------------------------------------
    @classmethod
    def encode(cls, W, tile_m: int = 128, tile_k: int = 128, maxd: int = 15) -> "Matrix":
        W = _u16(W)
        if W.ndim != 2:
            raise ValueError("W must be 2-D")
        h = ctypes.c_void_p()
        p = Params(tile_m, tile_k, maxd)
        _check(lib().tl3_encode(W.ctypes.data, W.shape[0], W.shape[1], ctypes.byref(p), ctypes.byref(h)),
               "tl3_encode")
        return cls(h.value)

    @classmethod
    def encode_on_device(cls, W, stream=None, device_only: bool = False) -> "Matrix":
        """The same container, built by the GPU encoder from a torch.float16 matrix on the device.
        ``device_only=True`` keeps it there (no host copy): follow with ``upload_packed_on_device``."""
        import torch
        if W.dtype != torch.float16 or W.dim() != 2 or W.stride(1) != 1 or not W.is_cuda:
            raise ValueError("W must be a 2-D float16 CUDA tensor with contiguous rows")
        h = ctypes.c_void_p()
        fn = lib().tl3_encode_device_only if device_only else lib().tl3_encode_device
        _check(fn(W.data_ptr(), W.shape[0], W.shape[1], W.stride(0), _stream_ptr(stream), ctypes.byref(h)), "tl3_encode_device")
        return cls(h.value)

    @classmethod
    def deserialize(cls, data: bytes) -> "Matrix":
        h = ctypes.c_void_p()
        buf = (ctypes.c_char * len(data)).from_buffer_copy(data)
        _check(lib().tl3_deserialize(ctypes.addressof(buf), len(data), ctypes.byref(h)), "tl3_deserialize")
        return cls(h.value)

    def close(self) -> None:
        if self._h:
            lib().tl3_free(self._h)
            self._h = ctypes.c_void_p()
        self._blob = None
        self._workspaces = {}

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- host side ---------------------------------------------------------------------------
    def stats(self) -> dict:
        s = Stats()
        _check(lib().tl3_stats(self._h, ctypes.byref(s)), "tl3_stats")
        return s.as_dict()

    @property
    def shape(self):
        s = self.stats()
        return s["M"], s["K"]

    def decode(self) -> np.ndarray:
        M, K = self.shape
        W = np.empty((M, K), dtype=np.uint16)
        _check(lib().tl3_decode(self._h, W.ctypes.data), "tl3_decode")
        return W

    def canonical(self, which) -> np.ndarray:
        idx = (CANONICAL + COMPACT + COMPACT_VALUES).index(which) if isinstance(which, str) else int(which)
        p, n = ctypes.c_void_p(), ctypes.c_size_t()
        _check(lib().tl3_canonical(self._h, idx, ctypes.byref(p), ctypes.byref(n)), "tl3_canonical")
        if n.value == 0:
            return np.zeros(0, dtype=_CANONICAL_DTYPES[idx])
        buf = (ctypes.c_uint8 * n.value).from_address(p.value)
        return np.frombuffer(buf, dtype=_CANONICAL_DTYPES[idx]).copy()

    def serialize(self, compact: bool = False) -> bytes:
        """The container as bytes; ``compact=True`` writes the Residual positions and the value
        array in their compact forms (``deserialize`` reads both)."""
        fn = lib().tl3_serialize_compact if compact else lib().tl3_serialize
        n = ctypes.c_size_t()
        _check(fn(self._h, None, ctypes.byref(n)), "tl3_serialize")
        buf = ctypes.create_string_buffer(n.value)
        _check(fn(self._h, buf, ctypes.byref(n)), "tl3_serialize")
        return buf.raw[:n.value]

    # -- device side -------------------------------------------------------------------------
    def device_bytes(self) -> int:
        return int(lib().tl3_device_bytes(self._h))

    def pack(self) -> np.ndarray:
        """The device blob as a host uint8 array (what ``upload`` copies to the GPU)."""
        buf = np.empty(self.device_bytes(), dtype=np.uint8)
        _check(lib().tl3_pack(self._h, buf.ctypes.data, buf.nbytes), "tl3_pack")
        return buf

    def upload(self, device="cuda", stream=None):
        """Allocates the blob as a torch.uint8 tensor, packs and copies the matrix into it."""
        import torch
        blob = torch.empty(self.device_bytes(), dtype=torch.uint8, device=device)
        _check(lib().tl3_upload(self._h, blob.data_ptr(), _stream_ptr(stream)), "tl3_upload")
        self._blob = blob
        return blob

    def upload_packed_on_device(self, device="cuda", stream=None):
        """As :meth:`upload`, with the device packer running on the GPU (same bytes)."""
        import torch
        _check(lib().tl3_plan_device(self._h, _stream_ptr(stream)), "tl3_plan_device")
        blob = torch.empty(self.device_bytes(), dtype=torch.uint8, device=device)
        _check(lib().tl3_upload_device(self._h, blob.data_ptr(), _stream_ptr(stream)), "tl3_upload_device")
        self._blob = blob
        return blob

    def bind(self, blob) -> None:
        """Makes a device tensor that already holds the packed blob (``pack()`` copied over, or a
        clone of what ``upload`` returned) the weights that later launches read."""
        _check(lib().tl3_bind(self._h, blob.data_ptr()), "tl3_bind")
        self._blob = blob

    def workspace_bytes(self, N: int) -> int:
        return int(lib().tl3_workspace_bytes(self._h, N))

    def new_workspace(self, N: int, stream=None):
        import torch
        n = self.workspace_bytes(N)
        if n == 0:
            raise Tl3Error(ERR_UNSUPPORTED, "tl3_workspace_bytes")
        ws = torch.empty(n, dtype=torch.uint8, device=self._blob.device if self._blob is not None else "cuda")
        _check(lib().tl3_workspace_init(ws.data_ptr(), n, _stream_ptr(stream)), "tl3_workspace_init")
        return ws

    def spmm(self, X, Y=None, workspace=None, stream=None, bias=None, activation=None):
        """``Y = W X`` on the GPU, or ``Y = act(W X + bias)`` when a bias (torch.float16, M entries, on
        the device) and / or an activation ("relu", "silu", "gelu_tanh") is given.
        X: torch.float16 (K x N, last dim contiguous) on the device."""
        import torch
        if X.dtype != torch.float16 or X.dim() != 2 or X.stride(1) != 1:
            raise ValueError("X must be a 2-D float16 tensor with contiguous rows")
        M, K = self.shape
        N = X.shape[1]
        if X.shape[0] != K:
            raise ValueError("X has the wrong number of rows")
        if Y is None:
            Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
        if workspace is None:
            key = 16 if N <= 16 else 32 if N <= 32 else 64        # wider blocks reuse the 64-column scratch
            workspace = self._workspaces.get(key)
            if workspace is None:
                workspace = self._workspaces[key] = self.new_workspace(N, stream)
        if bias is None and activation is None:
            _check(lib().tl3_spmm(self._h, X.data_ptr(), X.stride(0), Y.data_ptr(), Y.stride(0), N,
                                  workspace.data_ptr(), _stream_ptr(stream)), "tl3_spmm")
            return Y
        if bias is not None and (bias.dtype != torch.float16 or bias.numel() != M or not bias.is_contiguous()):
            raise ValueError("bias must be a contiguous float16 tensor with one entry per row of W")
        ep = Epilogue(bias.data_ptr() if bias is not None else None, ACTIVATIONS[activation])
        _check(lib().tl3_spmm_ex(self._h, X.data_ptr(), X.stride(0), Y.data_ptr(), Y.stride(0), N, ctypes.byref(ep),
                                 workspace.data_ptr(), _stream_ptr(stream)), "tl3_spmm_ex")
        return Y

    def spmm_nt(self, Xt, Yt=None, workspace=None, stream=None, bias=None, activation=None):
        """``Yt = Xt W^T`` (+ bias, activation): activations in the [batch, hidden] layout.
        Xt: torch.float16 (N x K, last dim contiguous) on the device; Yt: N x M."""
        import torch
        if Xt.dtype != torch.float16 or Xt.dim() != 2 or Xt.stride(1) != 1:
            raise ValueError("Xt must be a 2-D float16 tensor with contiguous rows")
        M, K = self.shape
        N = Xt.shape[0]
        if Xt.shape[1] != K:
            raise ValueError("Xt has the wrong number of columns")
        if Yt is None:
            Yt = torch.empty((N, M), dtype=torch.float16, device=Xt.device)
        if workspace is None:
            key = 16 if N <= 16 else 32 if N <= 32 else 64
            workspace = self._workspaces.get(key)
            if workspace is None:
                workspace = self._workspaces[key] = self.new_workspace(N, stream)
        if bias is not None and (bias.dtype != torch.float16 or bias.numel() != M or not bias.is_contiguous()):
            raise ValueError("bias must be a contiguous float16 tensor with one entry per row of W")
        ep = Epilogue(bias.data_ptr() if bias is not None else None, ACTIVATIONS[activation])
        _check(lib().tl3_spmm_nt(self._h, Xt.data_ptr(), Xt.stride(0), Yt.data_ptr(), Yt.stride(0), N, ctypes.byref(ep),
                                 workspace.data_ptr(), _stream_ptr(stream)), "tl3_spmm_nt")
        return Yt

    def spmm_static_scratch(self, X, Y=None, stream=None):
        """``Y = W X`` without a caller-supplied workspace and without any allocation inside the
        library: the scratch is a fixed 3 MiB array in the library image (see ``tl3.h``).  Raises
        ``Tl3Error(ERR_SCRATCH_LIMIT)`` when the problem needs more.  Calls must not overlap on the
        GPU.  (``Y`` is allocated here, by torch, only if the caller passes none.)"""
        import torch
        if X.dtype != torch.float16 or X.dim() != 2 or X.stride(1) != 1:
            raise ValueError("X must be a 2-D float16 tensor with contiguous rows")
        M, K = self.shape
        if X.shape[0] != K:
            raise ValueError("X has the wrong number of rows")
        N = X.shape[1]
        if Y is None:
            Y = torch.empty((M, N), dtype=torch.float16, device=X.device)
        _check(lib().tl3_spmm_static_scratch(self._h, X.data_ptr(), X.stride(0), Y.data_ptr(), Y.stride(0), N,
                                             _stream_ptr(stream)), "tl3_spmm_static_scratch")
        return Y

    def spmm_host(self, X: np.ndarray, Y: np.ndarray, dX, dY, workspace, stream=None) -> None:
        """``Y = W X`` with host arrays (fp16); device scratch dX, dY supplied by the caller."""
        X = _u16(X)
        if Y.dtype not in (np.uint16, np.float16) or not Y.flags.c_contiguous:
            raise TypeError("Y must be a contiguous fp16/uint16 array")
        _check(lib().tl3_spmm_host(self._h, X.ctypes.data, Y.ctypes.data, X.shape[1], dX.data_ptr(),
                                   dY.data_ptr(), workspace.data_ptr(), _stream_ptr(stream)), "tl3_spmm_host")

    def spmm_host_async(self, X: np.ndarray, Y: np.ndarray, dX, dY, workspace, stream=None) -> None:
        """As :meth:`spmm_host` but only enqueued on ``stream``: ``X`` must stay alive and ``Y`` is
        defined once the stream has been synchronised."""
        X = _u16(X)
        if Y.dtype not in (np.uint16, np.float16) or not Y.flags.c_contiguous:
            raise TypeError("Y must be a contiguous fp16/uint16 array")
        _check(lib().tl3_spmm_host_async(self._h, X.ctypes.data, Y.ctypes.data, X.shape[1], dX.data_ptr(),
                                         dY.data_ptr(), workspace.data_ptr(), _stream_ptr(stream)), "tl3_spmm_host_async")

    def status(self, workspace, stream=None) -> int:
        return int(lib().tl3_status(self._h, workspace.data_ptr(), _stream_ptr(stream)))

    def status_word(self, workspace, stream=None) -> int:
        w = ctypes.c_uint32()
        _check(lib().tl3_status_word(workspace.data_ptr(), _stream_ptr(stream), ctypes.byref(w)), "tl3_status_word")
        return int(w.value)

    def last_launch(self) -> dict:
        c, s, b = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        _check(lib().tl3_last_launch(self._h, ctypes.byref(c), ctypes.byref(s), ctypes.byref(b)), "tl3_last_launch")
        return {"ctas": c.value, "stages": s.value, "smem_bytes": b.value}


def encode(W, **kw) -> Matrix:
    return Matrix.encode(W, **kw)


def get_tuning() -> dict:
    """The process-wide launch tuning (``tl3_get_tuning``)."""
    t = Tuning()
    _check(lib().tl3_get_tuning(ctypes.byref(t)), "tl3_get_tuning")
    return {n: int(getattr(t, n)) for n, _ in Tuning._fields_}


def set_tuning(**kw) -> None:
    """``set_tuning()`` restores the defaults; keywords override single fields of the current tuning."""
    if not kw:
        _check(lib().tl3_set_tuning(None), "tl3_set_tuning")
        return
    cur = get_tuning()
    cur.update(kw)
    t = Tuning(**cur)
    _check(lib().tl3_set_tuning(ctypes.byref(t)), "tl3_set_tuning")
