"""CPU oracle for scaled-dot-product attention -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only the test-suite, the smoke check and the benchmark's ``cpu_baseline`` / ``--impl reference``
legs may import this package.  It shares no code with the CUDA library and never imports it.

``forward`` is the paper's definition (Eq. 3 with the softmax split of Eq. 4) evaluated in
IEEE double by ``sd_attn_oracle.c``; this module only builds that C file with gcc, marshals
numpy arrays into it and hands the results back.  No arithmetic of the method lives here.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd_attn_oracle.c")
_LIB = os.path.join(_HERE, "libsd_attn_oracle.so")
_lock = threading.Lock()
_lib = None

F16, F32 = 0, 1

_GEGLU_SRC = os.path.join(_HERE, "sd_geglu_oracle.c")
_GEGLU_LIB = os.path.join(_HERE, "libsd_geglu_oracle.so")
_geglu_lib = None
_GN_SRC = os.path.join(_HERE, "sd_groupnorm_oracle.c")
_GN_LIB = os.path.join(_HERE, "libsd_groupnorm_oracle.so")
_gn_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (plain -O2, OpenMP, no fast-math, no FP contraction)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            lib.sd_attn_oracle_forward.restype = ctypes.c_int
            lib.sd_attn_oracle_forward.argtypes = [
                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,      # q k v
                ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,      # out L S
                ctypes.c_void_p,                                        # probs
                ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                ctypes.c_float, ctypes.c_int,
                ctypes.c_void_p, ctypes.c_int64]
            lib.sd_attn_oracle_max_threads.restype = ctypes.c_int
            lib.sd_attn_oracle_set_threads.argtypes = [ctypes.c_int]
            lib.sd_attn_oracle_half_to_double.argtypes = [ctypes.c_void_p, ctypes.c_void_p,
                                                          ctypes.c_int64]
            _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().sd_attn_oracle_max_threads())


def set_threads(n: int) -> None:
    _load().sd_attn_oracle_set_threads(int(n))


def half_to_double(bits: np.ndarray) -> np.ndarray:
    """Widen raw binary16 bit patterns (uint16) with the oracle's own decoder."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().sd_attn_oracle_half_to_double(bits.ctypes.data, out.ctypes.data, bits.size)
    return out


def forward(q: np.ndarray, k: np.ndarray, v: np.ndarray, scale, rows=None, want_probs=False):
    """Attention of Eq. 3 in double precision.

    q: [B,H,Nq,d], k and v: [B,H,Nk,d]; all float16 or all float32 numpy arrays.
    scale: rounded to binary32 first (the value the C-ABI of the GPU library receives).
    rows: optional 1-D int64 array of flattened row ids ``(b*H+h)*Nq+i``; then only those
          rows are evaluated and the leading axes of the results are ``[len(rows)]``.
    Returns ``(out, L, S)`` or ``(out, L, S, P)``: out float64 ``[B,H,Nq,d]`` (or [n,d]),
    L and S float64 ``[B,H,Nq]`` (or [n]) as in Eq. 4, P float64 ``[..., Nk]``.
    """
    if q.dtype != k.dtype or q.dtype != v.dtype:
        raise TypeError("q, k, v must share one dtype")
    if q.dtype == np.float16:
        dtype = F16
    elif q.dtype == np.float32:
        dtype = F32
    else:
        raise TypeError("dtype must be float16 or float32")
    if q.ndim != 4 or k.ndim != 4 or v.ndim != 4:
        raise ValueError("expected [B,H,N,d] arrays")
    B, H, Nq, d = q.shape
    if k.shape[:2] != (B, H) or k.shape[3] != d or v.shape != k.shape:
        raise ValueError("shape mismatch between q, k, v")
    Nk = k.shape[2]
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    v = np.ascontiguousarray(v)
    if rows is None:
        lead = (B, H, Nq)
        rows_ptr, n_rows = None, 0
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64).ravel()
        lead = (rows.size,)
        rows_ptr, n_rows = rows.ctypes.data, rows.size
    out = np.zeros(lead + (d,), dtype=np.float64)
    L = np.zeros(lead, dtype=np.float64)
    S = np.zeros(lead, dtype=np.float64)
    P = np.zeros(lead + (Nk,), dtype=np.float64) if want_probs else None
    rc = _load().sd_attn_oracle_forward(
        q.ctypes.data, k.ctypes.data, v.ctypes.data, out.ctypes.data, L.ctypes.data,
        S.ctypes.data, P.ctypes.data if want_probs else None,
        B, H, Nq, Nk, d, ctypes.c_float(float(np.float32(scale))), dtype, rows_ptr, n_rows)
    if rc != 0:
        raise RuntimeError("sd_attn_oracle_forward failed with code %d" % rc)
    return (out, L, S, P) if want_probs else (out, L, S)


# ---------------------------------------------------------------------------------------------------------------
# Fused GEGLU (Sec. 3.1, Eq. 2): out = x[:, :C] * GELU(x[:, C:]).  The arithmetic lives in sd_geglu_oracle.c.

def build_geglu(force: bool = False) -> str:
    stale = (not os.path.exists(_GEGLU_LIB)) or os.path.getmtime(_GEGLU_LIB) < os.path.getmtime(_GEGLU_SRC)
    if force or stale:
        tmp = _GEGLU_LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _GEGLU_SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _GEGLU_LIB)
    return _GEGLU_LIB


def _load_geglu():
    global _geglu_lib
    with _lock:
        if _geglu_lib is None:
            lib = ctypes.CDLL(build_geglu())
            lib.sd_geglu_oracle_forward.restype = ctypes.c_int
            lib.sd_geglu_oracle_forward.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64,
                                                    ctypes.c_int]
            lib.sd_geglu_oracle_gelu.restype = ctypes.c_double
            lib.sd_geglu_oracle_gelu.argtypes = [ctypes.c_double]
            _geglu_lib = lib
    return _geglu_lib


def gelu(g: float) -> float:
    """GELU of Eq. 2 for one double."""
    return float(_load_geglu().sd_geglu_oracle_gelu(float(g)))


def geglu_forward(x: np.ndarray) -> np.ndarray:
    """x: [..., 2C] float16 or float32 -> [..., C] float64, out = x[..., :C] * GELU(x[..., C:])."""
    if x.dtype == np.float16:
        dtype = F16
    elif x.dtype == np.float32:
        dtype = F32
    else:
        raise TypeError("x must be float16 or float32")
    if x.shape[-1] % 2:
        raise ValueError("the last dimension holds both halves: it must be even")
    x = np.ascontiguousarray(x)
    C = x.shape[-1] // 2
    rows = x.size // (2 * C) if C else 0
    out = np.empty(x.shape[:-1] + (C,), dtype=np.float64)
    rc = _load_geglu().sd_geglu_oracle_forward(x.ctypes.data, out.ctypes.data, rows, C, dtype)
    if rc != 0:
        raise ValueError("sd_geglu_oracle_forward rejected its arguments")
    return out


# ---------------------------------------------------------------------------------------------------------------
# Fused group normalisation (Sec. 3.1, Eq. 1).  The arithmetic lives in sd_groupnorm_oracle.c.

def build_groupnorm(force: bool = False) -> str:
    stale = (not os.path.exists(_GN_LIB)) or os.path.getmtime(_GN_LIB) < os.path.getmtime(_GN_SRC)
    if force or stale:
        tmp = _GN_LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _GN_SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _GN_LIB)
    return _GN_LIB


def _load_groupnorm():
    global _gn_lib
    with _lock:
        if _gn_lib is None:
            lib = ctypes.CDLL(build_groupnorm())
            lib.sd_groupnorm_oracle_forward.restype = ctypes.c_int
            lib.sd_groupnorm_oracle_forward.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int64] * 4 + [ctypes.c_double,
                                                                                                      ctypes.c_int]
            _gn_lib = lib
    return _gn_lib


def groupnorm_forward(x: np.ndarray, groups: int, eps: float, gamma=None, beta=None):
    """x: [N, C, ...] float16 or float32 (spatial dimensions flattened); returns (y, mean, rstd) in float64:
    y like x, mean and rstd [N, groups]."""
    if x.dtype == np.float16:
        dtype = F16
    elif x.dtype == np.float32:
        dtype = F32
    else:
        raise TypeError("x must be float16 or float32")
    if x.ndim < 2:
        raise ValueError("x must be [N, C, ...]")
    x = np.ascontiguousarray(x)
    N, C = x.shape[0], x.shape[1]
    HW = int(np.prod(x.shape[2:])) if x.ndim > 2 else 1
    for name, t in (("gamma", gamma), ("beta", beta)):
        if t is not None and (t.dtype != x.dtype or t.shape != (C,)):
            raise ValueError("%s must be [C] in x's dtype" % name)
    ga = np.ascontiguousarray(gamma) if gamma is not None else None
    be = np.ascontiguousarray(beta) if beta is not None else None
    y = np.empty(x.shape, dtype=np.float64)
    mean = np.empty((N, groups), dtype=np.float64)
    rstd = np.empty((N, groups), dtype=np.float64)
    rc = _load_groupnorm().sd_groupnorm_oracle_forward(
        x.ctypes.data, ga.ctypes.data if ga is not None else None, be.ctypes.data if be is not None else None,
        y.ctypes.data, mean.ctypes.data, rstd.ctypes.data, N, C, HW, groups, float(eps), dtype)
    if rc != 0:
        raise ValueError("sd_groupnorm_oracle_forward rejected its arguments")
    return y, mean, rstd


# ---------------------------------------------------------------------------------------------------------------
# The 3x3 convolution behind the Winograd step (Sec. 3.3).  The arithmetic lives in sd_conv_oracle.c; the cost model
# of Table 2 is three ratios, written out below.

_CONV_SRC = os.path.join(_HERE, "sd_conv_oracle.c")
_CONV_LIB = os.path.join(_HERE, "libsd_conv_oracle.so")
_conv_lib = None


def build_conv(force: bool = False) -> str:
    stale = (not os.path.exists(_CONV_LIB)) or os.path.getmtime(_CONV_LIB) < os.path.getmtime(_CONV_SRC)
    if force or stale:
        tmp = _CONV_LIB + ".tmp.%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared", "-o", tmp, _CONV_SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
        os.replace(tmp, _CONV_LIB)
    return _CONV_LIB


def _load_conv():
    global _conv_lib
    with _lock:
        if _conv_lib is None:
            lib = ctypes.CDLL(build_conv())
            lib.sd_conv3x3_oracle_forward.restype = ctypes.c_int
            lib.sd_conv3x3_oracle_forward.argtypes = [ctypes.c_void_p] * 4 + [ctypes.c_int64] * 5 + [ctypes.c_int]
            _conv_lib = lib
    return _conv_lib


def conv3x3_forward(x: np.ndarray, w: np.ndarray, bias=None) -> np.ndarray:
    """x: [N, H, W, C], w: [K, 3, 3, C], bias: [K] or None, all float16 or all float32 -> y [N, H, W, K] float64:
    stride 1, zero padding 1, the filter not flipped (Sec. 3.3's convolution, by its definition)."""
    if x.dtype == np.float16:
        dtype = F16
    elif x.dtype == np.float32:
        dtype = F32
    else:
        raise TypeError("x must be float16 or float32")
    if x.ndim != 4 or w.ndim != 4 or w.shape[1:3] != (3, 3) or w.shape[3] != x.shape[3] or w.dtype != x.dtype:
        raise ValueError("x must be [N,H,W,C] and w [K,3,3,C] in the same dtype")
    if bias is not None and (bias.dtype != x.dtype or bias.shape != (w.shape[0],)):
        raise ValueError("bias must be [K] in x's dtype")
    x, w = np.ascontiguousarray(x), np.ascontiguousarray(w)
    b = np.ascontiguousarray(bias) if bias is not None else None
    N, H, W, C = x.shape
    K = w.shape[0]
    y = np.empty((N, H, W, K), dtype=np.float64)
    rc = _load_conv().sd_conv3x3_oracle_forward(x.ctypes.data, w.ctypes.data, b.ctypes.data if b is not None else None,
                                                y.ctypes.data, N, H, W, C, K, dtype)
    if rc != 0:
        raise ValueError("sd_conv3x3_oracle_forward rejected its arguments")
    return y


def winograd_cost_model(m: int):
    """Table 2 for an m x m output tile of a 3 x 3 filter, from the definitions: a tile of m*m outputs costs 9 m^2
    multiplications directly and (m + 2)^2 in the transformed domain ("Flops Saving" = their ratio); the transformed
    input holds (m + 2)^2 values per m^2 of the tensor ("Tensor"), the transformed filter (m + 2)^2 per 9 ("Weight")."""
    t = (m + 2) ** 2
    return 9.0 * m * m / t, t / float(m * m), t / 9.0
