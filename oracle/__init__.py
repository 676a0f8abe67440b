"""ctypes front end of the CPU oracle (``lynx_oracle.c``).

TEST INFRASTRUCTURE ONLY: the tests, the smoke check and the bench's cpu-baseline / reference
legs may import this package; the product (the CUDA library and its Python binding) never does,
and this package never imports the product.

All tensors cross this boundary as numpy arrays: bf16 data as ``uint16`` bit patterns,
metadata as ``uint16`` (canonical) or ``uint8`` (hardware order), results as ``float32``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lynx_oracle.c")
_LIB = os.path.join(_HERE, "liblynx_oracle.so")
_lock = threading.Lock()
_lib = None

COMP_NONE, COMP_ROW, COMP_TENSOR, COMP_GROUP = 0, 1, 2, 3


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over rows of the GEMM only)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            # no -march=native: the built file may be carried to a host with another CPU
            cmd = ["gcc", "-O3", "-fno-fast-math", "-ffp-contract=off", "-fopenmp",
                   "-fvisibility=hidden", "-shared", "-fPIC", "-std=c99", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_f32_to_bf16.restype = ctypes.c_uint16
        lib.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        lib.oracle_bf16_to_f32.restype = ctypes.c_float
        lib.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        lib.oracle_meta_hw_bytes.restype = ctypes.c_int64
        lib.oracle_meta_hw_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64]
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i64(v):
    return ctypes.c_int64(int(v))


def _u16(a, name):
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"{name}: expected uint16 bf16 bit patterns, got {a.dtype}")
    return a


def _check_x(X):
    X = _u16(X, "X")
    M, K = X.shape
    if K % 16:
        raise ValueError("K must be a multiple of 16")
    return X, M, K


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    return int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (numpy only; no oracle arithmetic)."""
    return (np.asarray(a, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def f32_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16 bit patterns, via the oracle's scalar routine."""
    flat = np.ascontiguousarray(a, dtype=np.float32).ravel()
    out = np.empty(flat.shape, dtype=np.uint16)
    _load().oracle_f32_to_bf16_array(_p(flat), _i64(flat.size), _p(out))
    return out.reshape(np.shape(a))


def topk24_mask(X: np.ndarray) -> np.ndarray:
    X, M, K = _check_x(X)
    mask = np.empty((M, K), dtype=np.uint8)
    _load().oracle_topk24_mask(_p(X), _i64(M), _i64(K), _i64(K), _p(mask))
    return mask


def compress(X: np.ndarray):
    """-> (values uint16 [M, K/2], meta_canon uint16 [M, K/16])"""
    X, M, K = _check_x(X)
    values = np.empty((M, K // 2), dtype=np.uint16)
    meta = np.empty((M, K // 16), dtype=np.uint16)
    _load().oracle_compress(_p(X), _i64(M), _i64(K), _i64(K), _p(values), _p(meta))
    return values, meta


def compress_group_scaled(X: np.ndarray):
    """Per-group norm compensation folded into the values (fp32 reading).
    -> (values uint16 [M, K/2] = bf16(s_g * kept), meta_canon uint16 [M, K/16])"""
    X, M, K = _check_x(X)
    values = np.empty((M, K // 2), dtype=np.uint16)
    meta = np.empty((M, K // 16), dtype=np.uint16)
    _load().oracle_compress_group_scaled(_p(X), _i64(M), _i64(K), _i64(K), _p(values), _p(meta))
    return values, meta


def group_scale_f64(X: np.ndarray) -> np.ndarray:
    """The per-group factors in fp64: [M, K/4]."""
    X, M, K = _check_x(X)
    s = np.empty((M, K // 4), dtype=np.float64)
    _load().oracle_group_scale_f64(_p(X), _i64(M), _i64(K), _i64(K), _p(s))
    return s


def decompress(values: np.ndarray, meta_canon: np.ndarray) -> np.ndarray:
    values = _u16(values, "values")
    meta_canon = _u16(meta_canon, "meta_canon")
    M, K2 = values.shape
    K = 2 * K2
    out = np.empty((M, K), dtype=np.uint16)
    _load().oracle_decompress(_p(values), _p(meta_canon), _i64(M), _i64(K), _p(out))
    return out


def meta_hw_bytes(M: int, K: int) -> int:
    return int(_load().oracle_meta_hw_bytes(_i64(M), _i64(K)))


def meta_canon_to_hw(meta_canon: np.ndarray, M: int, K: int) -> np.ndarray:
    if K % 128:
        raise ValueError("hardware metadata order needs K % 128 == 0")
    meta_canon = _u16(meta_canon, "meta_canon")
    out = np.zeros(meta_hw_bytes(M, K), dtype=np.uint8)
    _load().oracle_meta_canon_to_hw(_p(meta_canon), _i64(M), _i64(K), _p(out))
    return out


def meta_hw_to_canon(meta_hw: np.ndarray, M: int, K: int) -> np.ndarray:
    meta_hw = np.ascontiguousarray(meta_hw, dtype=np.uint8)
    assert meta_hw.size == meta_hw_bytes(M, K)
    out = np.empty((M, K // 16), dtype=np.uint16)
    _load().oracle_meta_hw_to_canon(_p(meta_hw), _i64(M), _i64(K), _p(out))
    return out


def row_scale(X: np.ndarray, mode: int) -> np.ndarray:
    X, M, K = _check_x(X)
    s = np.empty(M, dtype=np.float32)
    _load().oracle_row_scale(_p(X), _i64(M), _i64(K), _i64(K), ctypes.c_int(mode), _p(s))
    return s


def _rows(rows, M):
    if rows is None:
        return None, M
    r = np.ascontiguousarray(rows, dtype=np.int64)
    assert r.ndim == 1 and (r >= 0).all() and (r < M).all()
    return r, r.size


def gemm_masked_f32(Xmasked: np.ndarray, W: np.ndarray, rows=None) -> np.ndarray:
    Xmasked = _u16(Xmasked, "Xmasked")
    W = _u16(W, "W")
    M, K = Xmasked.shape
    N = W.shape[0]
    r, nr = _rows(rows, M)
    acc = np.empty((nr, N), dtype=np.float32)
    _load().oracle_gemm_masked_f32(_p(Xmasked), _i64(K), _p(W), _i64(N), _i64(W.shape[1]), _p(r),
                                   _i64(nr), _p(acc))
    return acc


def gemm_sparse_f32(values, meta_canon, W, rows=None) -> np.ndarray:
    values = _u16(values, "values")
    meta_canon = _u16(meta_canon, "meta_canon")
    W = _u16(W, "W")
    M, K2 = values.shape
    K = 2 * K2
    N = W.shape[0]
    r, nr = _rows(rows, M)
    acc = np.empty((nr, N), dtype=np.float32)
    _load().oracle_gemm_sparse_f32(_p(values), _p(meta_canon), _i64(K), _p(W), _i64(N),
                                   _i64(W.shape[1]), _p(r), _i64(nr), _p(acc))
    return acc


def gemm_masked_f64(Xmasked, W) -> np.ndarray:
    Xmasked = _u16(Xmasked, "Xmasked")
    W = _u16(W, "W")
    M, K = Xmasked.shape
    N = W.shape[0]
    acc = np.empty((M, N), dtype=np.float64)
    _load().oracle_gemm_masked_f64(_p(Xmasked), _i64(M), _i64(K), _p(W), _i64(N), _i64(W.shape[1]),
                                   _p(acc))
    return acc


def epilogue(acc, M, s=None, bias=None, Yr=None, rows=None) -> np.ndarray:
    acc = np.ascontiguousarray(acc, dtype=np.float32)
    nr, N = acc.shape
    r, nr2 = _rows(rows, M)
    assert nr2 == nr
    s = None if s is None else np.ascontiguousarray(s, dtype=np.float32)
    bias = None if bias is None else _u16(bias, "bias")
    Yr = None if Yr is None else _u16(Yr, "Yr")
    Y = np.empty((nr, N), dtype=np.float32)
    _load().oracle_epilogue(_p(acc), _i64(N), _p(r), _i64(nr), _p(s), _p(bias), _p(Yr), _i64(N),
                            _p(Y))
    return Y


def lora_residual(X, LB, LA, rows=None) -> np.ndarray:
    """Y_r = (X L_B^T) L_A^T in fp32 for `rows` (None = all rows)."""
    X, M, K = _check_x(X)
    LB = _u16(LB, "LB")
    LA = _u16(LA, "LA")
    R = LB.shape[0]
    N = LA.shape[0]
    assert LB.shape == (R, K) and LA.shape == (N, R) and R <= 512
    r, nr = _rows(rows, M)
    Yr = np.empty((nr, N), dtype=np.float32)
    _load().oracle_lora_residual_rows(_p(X), _i64(M), _i64(K), _i64(K), _p(LB), _i64(R), _p(LA), _i64(N),
                                      _p(r), _i64(nr), _p(Yr))
    return Yr


# ------------------------------------------------------------------------- FP8 composition ---

def e4m3_encode(x) -> np.ndarray:
    """fp32 -> E4M3 (FN) codes: round to nearest even, finite overflow and Inf saturate to +-448."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint8)
    _load().oracle_e4m3_encode_array(_p(x), _i64(x.size), _p(out))
    return out


def e4m3_decode(codes) -> np.ndarray:
    lib = _load()
    lib.oracle_e4m3_decode.restype = ctypes.c_float
    lib.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
    table = np.array([lib.oracle_e4m3_decode(i) for i in range(256)], dtype=np.float32)
    return table[np.asarray(codes, dtype=np.uint8)]


def quantize_weights_fp8(W, per_channel: bool):
    """-> (Wq uint8 [N, K], wscale float32 [N]); per_channel False = direct cast (scale 1)."""
    W = _u16(W, "W")
    N, K = W.shape
    Wq = np.empty((N, K), dtype=np.uint8)
    ws = np.empty(N, dtype=np.float32)
    _load().oracle_quantize_weights_fp8(_p(W), _i64(N), _i64(K), _i64(K), ctypes.c_int(1 if per_channel else 0),
                                        _p(Wq), _p(ws))
    return Wq, ws


def compress_fp8(X, row_amax=None):
    """-> (values_q uint8 [M, K/2], meta_canon uint16 [M, K/16], act_scale float32 [M]);
    row_amax (float32 [M]) replaces the row maxima taken from the data."""
    X, M, K = _check_x(X)
    row_amax = None if row_amax is None else np.ascontiguousarray(row_amax, dtype=np.float32)
    vq = np.empty((M, K // 2), dtype=np.uint8)
    meta = np.empty((M, K // 16), dtype=np.uint16)
    sc = np.empty(M, dtype=np.float32)
    _load().oracle_compress_fp8(_p(X), _i64(M), _i64(K), _i64(K), _p(row_amax), _p(vq), _p(meta), _p(sc))
    return vq, meta, sc


def meta_canon_to_hw_fp8(meta_canon, M: int, K: int) -> np.ndarray:
    meta_canon = _u16(meta_canon, "meta_canon")
    out = np.empty(((M + 127) // 128) * (K // 128) * 2048, dtype=np.uint8)
    _load().oracle_meta_canon_to_hw_fp8(_p(meta_canon), _i64(M), _i64(K), _p(out))
    return out


def act_sparse_linear_fp8(X, Wq, wscale, bias=None, comp_mode=COMP_NONE, Yr=None, rows=None, row_amax=None):
    """Whole FP8 path.  -> dict(values_q, meta_canon, row_scale (= s * act_scale), Y[fp32, rows x N])."""
    X, M, K = _check_x(X)
    Wq = np.ascontiguousarray(Wq, dtype=np.uint8)
    wscale = np.ascontiguousarray(wscale, dtype=np.float32)
    N = Wq.shape[0]
    assert Wq.shape == (N, K) and wscale.shape == (N,) and comp_mode in (COMP_NONE, COMP_ROW)
    bias = None if bias is None else _u16(bias, "bias")
    Yr = None if Yr is None else _u16(Yr, "Yr")
    r, nr = _rows(rows, M)
    vq = np.empty((M, K // 2), dtype=np.uint8)
    meta = np.empty((M, K // 16), dtype=np.uint16)
    rs = np.empty(M, dtype=np.float32)
    acc = np.empty((nr, N), dtype=np.float32)
    Y = np.empty((nr, N), dtype=np.float32)
    row_amax = None if row_amax is None else np.ascontiguousarray(row_amax, dtype=np.float32)
    _load().oracle_act_sparse_linear_fp8(_p(X), _i64(M), _i64(K), _i64(K), _p(row_amax), _p(Wq), _p(wscale), _i64(N), _p(bias),
                                         ctypes.c_int(comp_mode), _p(Yr), _i64(N), _p(r), _i64(nr), _p(vq),
                                         _p(meta), _p(rs), _p(acc), _p(Y))
    return {"values_q": vq, "meta_canon": meta, "row_scale": rs, "Y": Y}


def act_sparse_linear_lora(X, W, LA, LB, bias=None, comp_mode=COMP_NONE, Yr=None, rows=None):
    """Whole path of Algorithm 1 with the LoRA branch: Y = s * (X~ W^T) + b [+ Yr] + X (L_A L_B)^T."""
    out = act_sparse_linear(X, W, bias=bias, comp_mode=comp_mode, Yr=Yr, rows=rows)
    lora = lora_residual(X, LB, LA, rows=rows)
    Y = np.ascontiguousarray(out["Y"], dtype=np.float32)
    _load().oracle_add_lora(_p(Y), _p(lora), _i64(Y.shape[0]), _i64(Y.shape[1]))
    out["Y"] = Y
    out["lora"] = lora
    return out


def act_sparse_linear(X, W, bias=None, comp_mode=COMP_NONE, Yr=None, rows=None):
    """Whole path.  -> dict(values, meta_canon, scale, Y[fp32, rows x N])."""
    X, M, K = _check_x(X)
    W = _u16(W, "W")
    N = W.shape[0]
    assert W.shape[1] == K
    bias = None if bias is None else _u16(bias, "bias")
    Yr = None if Yr is None else _u16(Yr, "Yr")
    r, nr = _rows(rows, M)
    values = np.empty((M, K // 2), dtype=np.uint16)
    meta = np.empty((M, K // 16), dtype=np.uint16)
    scale = np.empty(M, dtype=np.float32)
    xm = np.empty((M, K), dtype=np.uint16)
    acc = np.empty((nr, N), dtype=np.float32)
    Y = np.empty((nr, N), dtype=np.float32)
    _load().oracle_act_sparse_linear(_p(X), _i64(M), _i64(K), _i64(K), _p(W), _i64(N), _i64(K),
                                     _p(bias), ctypes.c_int(comp_mode), _p(Yr), _i64(N), _p(r),
                                     _i64(nr), _p(values), _p(meta), _p(scale), _p(xm), _p(acc), _p(Y))
    return {"values": values, "meta_canon": meta, "scale": scale, "Y": Y}
