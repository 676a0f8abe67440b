"""Python binding of the C-ABI library ``liblynx.so``: argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used for device memory and
streams.  There is no CPU fallback: if the library cannot be loaded, importing the symbols
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

COMP_NONE, COMP_ROW, COMP_TENSOR, COMP_GROUP = 0, 1, 2, 3
FUSE_AUTO, FUSE_SEPARATE, FUSE_FUSED = 0, 1, 2

EXPORTS = [
    "lynx_create", "lynx_destroy", "lynx_status_string", "lynx_last_error", "lynx_values_bytes",
    "lynx_meta_bytes", "lynx_workspace_bytes", "lynx_reserve", "lynx_prune_compress",
    "lynx_sparse_linear", "lynx_act_sparse_linear", "lynx_act_sparse_linear_host",
    "lynx_meta_to_canonical", "lynx_decompress", "lynx_launch_count", "lynx_prune_compress_static",
    "lynx_reserve_lora", "lynx_lora_down", "lynx_prune_compress_lora", "lynx_sparse_linear_lora", "lynx_act_sparse_linear_lora",
    "lynx_quantize_weights_fp8", "lynx_prune_compress_fp8", "lynx_sparse_linear_fp8",
    "lynx_act_sparse_linear_fp8", "lynx_gemm_plan", "lynx_gemm_schedule_items", "lynx_selftest_wait_timeout",
]


class _Deferred:
    """Pass as ``row_scale`` to ``Lynx.prune_compress`` (ROW mode) and to the ``Lynx.sparse_linear`` call
    that follows on the same context: the prune kernel stops at its row sums and the GEMM epilogue
    forms the scale from them (``LYNX_ROW_SCALE_DEFERRED``)."""

    def __repr__(self):
        return "ROW_SCALE_DEFERRED"


ROW_SCALE_DEFERRED = _Deferred()


class LynxError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: lynx status {status} ({status_string(status)})")
        self.status = status


class _Comp(ctypes.Structure):
    _fields_ = [("row_scale", ctypes.c_void_p), ("residual", ctypes.c_void_p), ("ldr", ctypes.c_int64)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads (building first if the sources are newer) the CUDA library.  Raises on failure."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.is_stale():
        try:
            _build.build()
        except Exception as e:  # no nvcc on this host and no prebuilt library
            if not os.path.exists(path):
                raise RuntimeError(f"liblynx.so is missing and could not be built: {e}") from e
    lib = ctypes.CDLL(path)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
    lib.lynx_create.argtypes = [ctypes.POINTER(vp), i32]
    lib.lynx_destroy.argtypes = [vp]
    lib.lynx_status_string.argtypes = [i32]
    lib.lynx_status_string.restype = ctypes.c_char_p
    lib.lynx_last_error.argtypes = [vp]
    for name in ("lynx_values_bytes", "lynx_meta_bytes"):
        getattr(lib, name).argtypes = [i64, i64]
        getattr(lib, name).restype = ctypes.c_size_t
    lib.lynx_workspace_bytes.argtypes = [i64, i64, i64]
    lib.lynx_workspace_bytes.restype = ctypes.c_size_t
    lib.lynx_reserve.argtypes = [vp, i64, i64, i64]
    lib.lynx_prune_compress.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, i32, vp]
    lib.lynx_sparse_linear.argtypes = [vp, vp, vp, i64, i64, vp, i64, i64, vp, ctypes.POINTER(_Comp), vp,
                                       i64, vp]
    lib.lynx_act_sparse_linear.argtypes = [vp, vp, i64, i64, i64, vp, i64, i64, vp, i32, vp, i64, vp, i64,
                                           i32, vp]
    lib.lynx_act_sparse_linear_host.argtypes = [vp, vp, i64, i64, vp, i64, i64, vp, i32, vp, i32, vp]
    lib.lynx_meta_to_canonical.argtypes = [vp, vp, i64, i64, vp, vp]
    lib.lynx_decompress.argtypes = [vp, vp, vp, i64, i64, vp, vp]
    lib.lynx_prune_compress_static.argtypes = [vp, i64, i64, i64, vp, vp, vp, i32, vp]
    lib.lynx_reserve_lora.argtypes = [vp, i64, i64, i64]
    lib.lynx_lora_down.argtypes = [vp, vp, i64, i64, i64, vp, i64, i64, vp, vp, i64, vp]
    lib.lynx_prune_compress_lora.argtypes = [vp, vp, i64, i64, i64, vp, i64, i64, vp, vp, ctypes.c_int, vp, i64, vp]
    lib.lynx_sparse_linear_lora.argtypes = [vp, vp, vp, i64, i64, vp, i64, i64, vp, ctypes.POINTER(_Comp), vp,
                                            i64, vp, i64, i64, vp, i64, vp]
    lib.lynx_act_sparse_linear_lora.argtypes = [vp, vp, i64, i64, i64, vp, i64, i64, vp, vp, i64, vp, i64, i64,
                                                i32, vp, i64, vp, i64, vp]
    lib.lynx_quantize_weights_fp8.argtypes = [vp, vp, i64, i64, i64, i32, vp, vp, vp]
    lib.lynx_prune_compress_fp8.argtypes = [vp, vp, i64, i64, i64, vp, vp, vp, vp, i32, vp]
    lib.lynx_sparse_linear_fp8.argtypes = [vp, vp, vp, i64, i64, vp, i64, i64, vp, vp, ctypes.POINTER(_Comp), vp,
                                           i64, vp]
    lib.lynx_act_sparse_linear_fp8.argtypes = [vp, vp, i64, i64, i64, vp, vp, i64, i64, vp, vp, i32, vp, i64, vp,
                                               i64, vp]
    lib.lynx_gemm_plan.argtypes = [i32, i64, i64, i64, i32, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.lynx_gemm_schedule_items.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(i32), i32]
    lib.lynx_selftest_wait_timeout.argtypes = [vp, i64, vp]
    lib.lynx_launch_count.argtypes = [vp]
    lib.lynx_launch_count.restype = i64
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().lynx_status_string(int(status)).decode()


def values_bytes(M: int, K: int) -> int:
    return int(load_library().lynx_values_bytes(M, K))


def meta_bytes(M: int, K: int) -> int:
    return int(load_library().lynx_meta_bytes(M, K))


def gemm_plan(num_sms: int, M: int, N: int, K: int, lora_steps: int = 0):
    """-> (uses_two_row_tile_kernel, doubles, clusters): host-only view of the GEMM's plan."""
    d, c = ctypes.c_int(0), ctypes.c_int(0)
    r = load_library().lynx_gemm_plan(num_sms, M, N, K, lora_steps, ctypes.byref(d), ctypes.byref(c))
    if r < 0:
        raise ValueError("lynx_gemm_plan: bad arguments")
    return bool(r), d.value, c.value


def gemm_schedule_items(tiles_m: int, tiles_n: int, clusters: int, doubles: int, cluster: int):
    """-> list of (first row tile, column tile, row tiles, ordinal) of one CTA pair (host only)."""
    cap = tiles_m * tiles_n + 1
    buf = (ctypes.c_int * (4 * cap))()
    n = load_library().lynx_gemm_schedule_items(tiles_m, tiles_n, clusters, doubles, cluster, buf, cap)
    if n < 0:
        raise ValueError("lynx_gemm_schedule_items: bad arguments")
    return [tuple(buf[4 * i:4 * i + 4]) for i in range(n)]


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, what: str):
    if status != 0:
        raise LynxError(status, what)


def _bf16_2d(t: torch.Tensor, name: str):
    if t.dtype != torch.bfloat16 or t.dim() != 2 or t.stride(1) != 1:
        raise TypeError(f"{name}: expected a 2-D bf16 tensor with unit inner stride")
    return t


STATIC_SCRATCH_BYTES = 8 << 20


def prune_compress_static(X: torch.Tensor, mode: int = COMP_NONE, values=None, meta=None, row_scale=None):
    """``lynx_prune_compress_static``: the prune/compress step for callers that cannot allocate
    device memory (a process whose memory pool owns the whole GPU, or a loop that must not incur
    the device synchronisation an allocation implies).  The library allocates nothing: pass
    ``values`` / ``meta`` / ``row_scale`` that you already own (they are only created here, with
    torch, when left out).  Runs on the current device and torch's current stream, uses the
    library's fixed scratch array shared by all calls -- do not overlap two calls on the GPU.
    The first call on a device performs a one-time address look-up."""
    _bf16_2d(X, "X")
    M, K = X.shape
    if values is None:
        values = torch.empty((M, K // 2), dtype=torch.bfloat16, device=X.device)
    if meta is None:
        meta = torch.empty(meta_bytes(M, K), dtype=torch.uint8, device=X.device)
    if row_scale is None and mode in (COMP_ROW, COMP_TENSOR):
        row_scale = torch.empty(M, dtype=torch.float32, device=X.device)
    _check(load_library().lynx_prune_compress_static(_ptr(X), M, K, X.stride(0), _ptr(values), _ptr(meta),
                                                     _ptr(row_scale), mode, _stream()),
           "lynx_prune_compress_static")
    return values, meta, row_scale


class Lynx:
    """One library context on one CUDA device (scratch workspace, error word)."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        self.device = torch.device("cuda", device)
        h = ctypes.c_void_p()
        _check(self._lib.lynx_create(ctypes.byref(h), device), "lynx_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.lynx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- bookkeeping -------------------------------------------------------------------------
    def reserve(self, M: int, N: int, K: int):
        _check(self._lib.lynx_reserve(self._h, M, N, K), "lynx_reserve")

    def last_error(self) -> int:
        return int(self._lib.lynx_last_error(self._h))

    def selftest_wait_timeout(self, limit_us: int = 1000):
        """Launches the one-warp kernel whose bounded wait runs out (see lynx_selftest_wait_timeout)."""
        _check(self._lib.lynx_selftest_wait_timeout(self._h, limit_us, _stream()), "lynx_selftest_wait_timeout")

    def launch_count(self) -> int:
        return int(self._lib.lynx_launch_count(self._h))

    # -- the three calls of the path ---------------------------------------------------------
    def prune_compress(self, X: torch.Tensor, mode: int = COMP_NONE, values=None, meta=None,
                       row_scale=None) -> Tuple[torch.Tensor, torch.Tensor, Optional[torch.Tensor]]:
        _bf16_2d(X, "X")
        M, K = X.shape
        if values is None:
            values = torch.empty((M, K // 2), dtype=torch.bfloat16, device=X.device)
        if meta is None:
            meta = torch.empty(meta_bytes(M, K), dtype=torch.uint8, device=X.device)
        if row_scale is None and mode in (COMP_ROW, COMP_TENSOR):
            row_scale = torch.empty(M, dtype=torch.float32, device=X.device)
        rs = ctypes.c_void_p(1) if row_scale is ROW_SCALE_DEFERRED else _ptr(row_scale)
        _check(self._lib.lynx_prune_compress(self._h, _ptr(X), M, K, X.stride(0), _ptr(values), _ptr(meta),
                                             rs, mode, _stream()), "lynx_prune_compress")
        return values, meta, row_scale

    def sparse_linear(self, values: torch.Tensor, meta: torch.Tensor, W: torch.Tensor, bias=None,
                      row_scale=None, residual=None, out=None) -> torch.Tensor:
        _bf16_2d(values, "values")
        _bf16_2d(W, "W")
        M, K = values.shape[0], values.shape[1] * 2
        N = W.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=values.device)
        comp = _Comp(1 if row_scale is ROW_SCALE_DEFERRED else (None if row_scale is None else row_scale.data_ptr()),
                     None if residual is None else residual.data_ptr(),
                     0 if residual is None else residual.stride(0))
        _check(self._lib.lynx_sparse_linear(self._h, _ptr(values), _ptr(meta), M, K, _ptr(W), N, W.stride(0),
                                            _ptr(bias), ctypes.byref(comp), _ptr(out), out.stride(0),
                                            _stream()), "lynx_sparse_linear")
        return out

    def act_sparse_linear(self, X: torch.Tensor, W: torch.Tensor, bias=None, mode: int = COMP_NONE,
                          residual=None, out=None, fuse: int = FUSE_AUTO) -> torch.Tensor:
        _bf16_2d(X, "X")
        _bf16_2d(W, "W")
        M, K = X.shape
        N = W.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
        _check(self._lib.lynx_act_sparse_linear(self._h, _ptr(X), M, K, X.stride(0), _ptr(W), N, W.stride(0),
                                                _ptr(bias), mode, _ptr(residual),
                                                0 if residual is None else residual.stride(0), _ptr(out),
                                                out.stride(0), fuse, _stream()), "lynx_act_sparse_linear")
        return out

    def act_sparse_linear_host(self, X_host: torch.Tensor, W: torch.Tensor, bias=None, mode: int = COMP_NONE,
                               Y_host=None, fuse: int = FUSE_AUTO) -> torch.Tensor:
        """X_host / Y_host are CPU (ideally pinned) bf16 tensors; W, bias are CUDA tensors."""
        assert X_host.device.type == "cpu" and X_host.is_contiguous() and X_host.dtype == torch.bfloat16
        M, K = X_host.shape
        N = W.shape[0]
        if Y_host is None:
            Y_host = torch.empty((M, N), dtype=torch.bfloat16, pin_memory=True)
        assert Y_host.device.type == "cpu" and Y_host.is_contiguous()
        _check(self._lib.lynx_act_sparse_linear_host(self._h, _ptr(X_host), M, K, _ptr(W), N, W.stride(0),
                                                     _ptr(bias), mode, _ptr(Y_host), fuse, _stream()),
               "lynx_act_sparse_linear_host")
        return Y_host

    # -- low-rank branch -----------------------------------------------------------------------
    def reserve_lora(self, M: int, K: int, R: int):
        _check(self._lib.lynx_reserve_lora(self._h, M, K, R), "lynx_reserve_lora")

    def lora_down(self, X: torch.Tensor, LB: torch.Tensor, row_scale=None, out=None) -> torch.Tensor:
        """T = bf16((X L_B^T) / s): [M, R]."""
        _bf16_2d(X, "X")
        _bf16_2d(LB, "LB")
        M, K = X.shape
        R = LB.shape[0]
        if out is None:
            out = torch.empty((M, R), dtype=torch.bfloat16, device=X.device)
        _check(self._lib.lynx_lora_down(self._h, _ptr(X), M, K, X.stride(0), _ptr(LB), R, LB.stride(0),
                                        _ptr(row_scale), _ptr(out), out.stride(0), _stream()), "lynx_lora_down")
        return out

    def prune_compress_lora(self, X: torch.Tensor, LB: torch.Tensor, mode: int = COMP_NONE, values=None, meta=None,
                            T=None):
        """One launch, X read once -> (values, meta, T = (X L_B^T) / s); under COMP_ROW the row sums stay
        on the context: pass ROW_SCALE_DEFERRED to the sparse_linear_lora call that follows."""
        _bf16_2d(X, "X")
        _bf16_2d(LB, "LB")
        M, K = X.shape
        R = LB.shape[0]
        if values is None:
            values = torch.empty((M, K // 2), dtype=torch.bfloat16, device=X.device)
        if meta is None:
            meta = torch.empty(meta_bytes(M, K), dtype=torch.uint8, device=X.device)
        if T is None:
            T = torch.empty((M, R), dtype=torch.bfloat16, device=X.device)
        _check(self._lib.lynx_prune_compress_lora(self._h, _ptr(X), M, K, X.stride(0), _ptr(LB), R, LB.stride(0),
                                                  _ptr(values), _ptr(meta), mode, _ptr(T), T.stride(0), _stream()),
               "lynx_prune_compress_lora")
        return values, meta, T

    def sparse_linear_lora(self, values: torch.Tensor, meta: torch.Tensor, W: torch.Tensor, T: torch.Tensor,
                           LA: torch.Tensor, bias=None, row_scale=None, residual=None, out=None) -> torch.Tensor:
        _bf16_2d(values, "values")
        _bf16_2d(W, "W")
        _bf16_2d(T, "T")
        _bf16_2d(LA, "LA")
        M, K = values.shape[0], values.shape[1] * 2
        N = W.shape[0]
        R = LA.shape[1]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=values.device)
        comp = _Comp(1 if row_scale is ROW_SCALE_DEFERRED else (None if row_scale is None else row_scale.data_ptr()),
                     None if residual is None else residual.data_ptr(),
                     0 if residual is None else residual.stride(0))
        _check(self._lib.lynx_sparse_linear_lora(self._h, _ptr(values), _ptr(meta), M, K, _ptr(W), N, W.stride(0),
                                                 _ptr(bias), ctypes.byref(comp), _ptr(T), T.stride(0), _ptr(LA), R,
                                                 LA.stride(0), _ptr(out), out.stride(0), _stream()),
               "lynx_sparse_linear_lora")
        return out

    def act_sparse_linear_lora(self, X: torch.Tensor, W: torch.Tensor, LA: torch.Tensor, LB: torch.Tensor,
                               bias=None, mode: int = COMP_NONE, residual=None, out=None) -> torch.Tensor:
        _bf16_2d(X, "X")
        _bf16_2d(W, "W")
        _bf16_2d(LA, "LA")
        _bf16_2d(LB, "LB")
        M, K = X.shape
        N = W.shape[0]
        R = LB.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
        _check(self._lib.lynx_act_sparse_linear_lora(self._h, _ptr(X), M, K, X.stride(0), _ptr(W), N, W.stride(0),
                                                     _ptr(bias), _ptr(LA), LA.stride(0), _ptr(LB), LB.stride(0), R,
                                                     mode, _ptr(residual),
                                                     0 if residual is None else residual.stride(0), _ptr(out),
                                                     out.stride(0), _stream()), "lynx_act_sparse_linear_lora")
        return out

    # -- FP8 composition -----------------------------------------------------------------------
    def quantize_weights_fp8(self, W: torch.Tensor, per_channel: bool = True):
        """-> (Wq uint8 [N, K] E4M3 codes, wscale float32 [N])"""
        _bf16_2d(W, "W")
        N, K = W.shape
        Wq = torch.empty((N, K), dtype=torch.uint8, device=W.device)
        ws = torch.empty(N, dtype=torch.float32, device=W.device)
        _check(self._lib.lynx_quantize_weights_fp8(self._h, _ptr(W), N, K, W.stride(0), 1 if per_channel else 0,
                                                   _ptr(Wq), _ptr(ws), _stream()), "lynx_quantize_weights_fp8")
        return Wq, ws

    def prune_compress_fp8(self, X: torch.Tensor, mode: int = COMP_NONE, values_q=None, meta=None, row_scale=None,
                           row_amax=None):
        """-> (values_q uint8 [M, K/2], meta uint8, row_scale float32 [M] = s * amax / 448);
        row_amax (float32 [M]) replaces the row maxima found in the data (X is then read once)."""
        _bf16_2d(X, "X")
        M, K = X.shape
        if values_q is None:
            values_q = torch.empty((M, K // 2), dtype=torch.uint8, device=X.device)
        if meta is None:
            meta = torch.empty(meta_bytes(M, K), dtype=torch.uint8, device=X.device)
        if row_scale is None:
            row_scale = torch.empty(M, dtype=torch.float32, device=X.device)
        _check(self._lib.lynx_prune_compress_fp8(self._h, _ptr(X), M, K, X.stride(0), _ptr(row_amax), _ptr(values_q),
                                                 _ptr(meta), _ptr(row_scale), mode, _stream()),
               "lynx_prune_compress_fp8")
        return values_q, meta, row_scale

    def sparse_linear_fp8(self, values_q: torch.Tensor, meta: torch.Tensor, Wq: torch.Tensor, wscale=None,
                          bias=None, row_scale=None, residual=None, out=None) -> torch.Tensor:
        M, K = values_q.shape[0], values_q.shape[1] * 2
        N = Wq.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=values_q.device)
        comp = _Comp(None if row_scale is None else row_scale.data_ptr(),
                     None if residual is None else residual.data_ptr(),
                     0 if residual is None else residual.stride(0))
        _check(self._lib.lynx_sparse_linear_fp8(self._h, _ptr(values_q), _ptr(meta), M, K, _ptr(Wq), N, Wq.stride(0),
                                                _ptr(wscale), _ptr(bias), ctypes.byref(comp), _ptr(out),
                                                out.stride(0), _stream()), "lynx_sparse_linear_fp8")
        return out

    def act_sparse_linear_fp8(self, X: torch.Tensor, Wq: torch.Tensor, wscale=None, bias=None,
                              mode: int = COMP_NONE, residual=None, out=None, row_amax=None) -> torch.Tensor:
        _bf16_2d(X, "X")
        M, K = X.shape
        N = Wq.shape[0]
        if out is None:
            out = torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
        _check(self._lib.lynx_act_sparse_linear_fp8(self._h, _ptr(X), M, K, X.stride(0), _ptr(row_amax), _ptr(Wq), N,
                                                    Wq.stride(0),
                                                    _ptr(wscale), _ptr(bias), mode, _ptr(residual),
                                                    0 if residual is None else residual.stride(0), _ptr(out),
                                                    out.stride(0), _stream()), "lynx_act_sparse_linear_fp8")
        return out

    # -- inspection ----------------------------------------------------------------------------
    def meta_to_canonical(self, meta: torch.Tensor, M: int, K: int) -> torch.Tensor:
        out = torch.empty((M, K // 16), dtype=torch.int16, device=meta.device)
        _check(self._lib.lynx_meta_to_canonical(self._h, _ptr(meta), M, K, _ptr(out), _stream()),
               "lynx_meta_to_canonical")
        return out

    def decompress(self, values: torch.Tensor, meta: torch.Tensor) -> torch.Tensor:
        M, K = values.shape[0], values.shape[1] * 2
        out = torch.empty((M, K), dtype=torch.bfloat16, device=values.device)
        _check(self._lib.lynx_decompress(self._h, _ptr(values), _ptr(meta), M, K, _ptr(out), _stream()),
               "lynx_decompress")
        return out
