"""ctypes binding of the C-ABI attention library (argument marshalling only).

Function names mirror ``include/sd_attn.h``.  Tensors are passed as raw device addresses
(``tensor.data_ptr()``); PyTorch only owns the memory and the streams.  There is no fallback:
if ``libsd_attn.so`` is missing or fails to load, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libsd_attn.so")

# status codes, dtypes and modes of include/sd_attn.h
OK, ERR_INVALID_VALUE, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_DEVICE_TIMEOUT = range(8)
F16, F32, BF16 = 0, 1, 2
MODE_AUTO, MODE_FUSED, MODE_CROSS, MODE_TWOPASS, MODE_SIMT = range(5)
MODE_NAMES = {MODE_AUTO: "auto", MODE_FUSED: "fused", MODE_CROSS: "cross", MODE_TWOPASS: "twopass",
              MODE_SIMT: "simt"}
LAYOUT_BHND, LAYOUT_BNHD = 0, 1   # sd_attn_layout: head-major [B,H,N,d] / token-major [B,N,H,d]
CROSS_MAX_NK = 128
MAX_D = 160
STATIC_MAX_SCRATCH = 34 * 1024 * 1024   # SD_ATTN_STATIC_MAX_SCRATCH: built-in scratch of the no-allocation entry point

EXPORTS = ["sd_attn_create", "sd_attn_create_ex", "sd_attn_static_query_status", "sd_attn_selftest_wait_timeout", "sd_attn_ubench", "sd_attn_forward", "sd_attn_destroy", "sd_attn_set_mode",
           "sd_attn_workspace_bytes", "sd_attn_set_workspace", "sd_attn_twopass_buffers",
           "sd_attn_query_status", "sd_attn_last_mode", "sd_attn_launch_count", "sd_attn_status_string",
           "sd_attn_forward_host", "sd_attn_host_staging_bytes",
           "sd_attn_forward_twopass_static", "sd_geglu_forward", "sd_groupnorm_forward", "sd_attn_set_layout", "sd_attn_forward_batch",
           "sd_winograd_filter_elems", "sd_winograd_transform_filter", "sd_winograd_workspace_bytes",
           "sd_winograd_conv3x3_forward", "sd_winograd_query_status"]

_lib = None


class Problem(ctypes.Structure):
    """sd_attn_problem: one problem of sd_attn_forward_batch."""
    _fields_ = [("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("out", ctypes.c_void_p),
                ("B", ctypes.c_int), ("H", ctypes.c_int), ("Nq", ctypes.c_int), ("Nk", ctypes.c_int),
                ("d", ctypes.c_int), ("scale", ctypes.c_float)]


class Options(ctypes.Structure):
    """sd_attn_options: choices made when a handle is created (all zero = the defaults)."""
    _fields_ = [("struct_size", ctypes.c_size_t), ("no_pdl", ctypes.c_int), ("fused_tiles", ctypes.c_int),
                ("fused_split", ctypes.c_int), ("fused_shares", ctypes.c_int), ("cross_one_tile", ctypes.c_int),
                ("host_one_slice", ctypes.c_int), ("batch_serial", ctypes.c_int)]

    def __init__(self, **kw):
        super().__init__(**kw)
        self.struct_size = ctypes.sizeof(Options)


class SdAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: status %d (%s)" % (where, status, status_string(status)))


def load() -> ctypes.CDLL:
    """Load libsd_attn.so (built in-tree by ``build.py``).  Raises if it is absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            "%s not found: build it with `python -m paper_2304_11267_b200.build` "
            "(there is no CPU fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.sd_attn_create.restype = ci
    lib.sd_attn_create.argtypes = [ctypes.POINTER(vp)]
    lib.sd_attn_create_ex.restype = ci
    lib.sd_attn_create_ex.argtypes = [ctypes.POINTER(Options), ctypes.POINTER(vp)]
    lib.sd_attn_selftest_wait_timeout.restype = ci
    lib.sd_attn_selftest_wait_timeout.argtypes = [vp, vp]
    lib.sd_attn_ubench.restype = ci
    lib.sd_attn_ubench.argtypes = [ci, ci, vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
    lib.sd_attn_static_query_status.restype = ci
    lib.sd_attn_static_query_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.sd_attn_forward.restype = ci
    lib.sd_attn_forward.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, vp]
    lib.sd_attn_forward_host.restype = ci
    lib.sd_attn_forward_host.argtypes = [vp, vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, cf, ci, vp]
    lib.sd_attn_host_staging_bytes.restype = sz
    lib.sd_attn_host_staging_bytes.argtypes = [ci, ci, ci, ci, ci, ci]
    lib.sd_attn_destroy.restype = ci
    lib.sd_attn_destroy.argtypes = [vp]
    lib.sd_attn_set_mode.restype = ci
    lib.sd_attn_set_mode.argtypes = [vp, ci]
    lib.sd_attn_forward_batch.restype = ci
    lib.sd_attn_forward_batch.argtypes = [vp, ctypes.POINTER(Problem), ci, ci, vp]
    lib.sd_winograd_filter_elems.restype = sz
    lib.sd_winograd_filter_elems.argtypes = [ci, ci]
    lib.sd_winograd_transform_filter.restype = ci
    lib.sd_winograd_transform_filter.argtypes = [vp, vp, ci, ci, vp]
    lib.sd_winograd_workspace_bytes.restype = sz
    lib.sd_winograd_workspace_bytes.argtypes = [ci, ci, ci, ci, ci]
    lib.sd_winograd_conv3x3_forward.restype = ci
    lib.sd_winograd_conv3x3_forward.argtypes = [vp, vp, vp, vp, vp, sz, ci, ci, ci, ci, ci, vp]
    lib.sd_winograd_query_status.restype = ci
    lib.sd_winograd_query_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.sd_attn_set_layout.restype = ci
    lib.sd_attn_set_layout.argtypes = [vp, ci]
    lib.sd_attn_workspace_bytes.restype = sz
    lib.sd_attn_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci]
    lib.sd_attn_set_workspace.restype = ci
    lib.sd_attn_set_workspace.argtypes = [vp, vp, sz]
    lib.sd_attn_twopass_buffers.restype = ci
    lib.sd_attn_twopass_buffers.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(vp)]
    lib.sd_attn_query_status.restype = ci
    lib.sd_attn_query_status.argtypes = [vp, vp, ctypes.POINTER(ci)]
    lib.sd_attn_last_mode.restype = ci
    lib.sd_attn_last_mode.argtypes = [vp]
    lib.sd_attn_launch_count.restype = ctypes.c_longlong
    lib.sd_attn_launch_count.argtypes = [vp]
    lib.sd_attn_status_string.restype = ctypes.c_char_p
    lib.sd_attn_status_string.argtypes = [ci]
    lib.sd_attn_forward_twopass_static.restype = ci
    lib.sd_attn_forward_twopass_static.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, ci, cf, ci, vp]
    lib.sd_geglu_forward.restype = ci
    lib.sd_geglu_forward.argtypes = [vp, vp, ctypes.c_longlong, ci, ci, vp]
    lib.sd_groupnorm_forward.restype = ci
    lib.sd_groupnorm_forward.argtypes = [vp, vp, vp, vp, ci, ci, ctypes.c_longlong, ci, cf, ci, vp]
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().sd_attn_status_string(int(status)).decode()


# ------------------------------------------------------------------ one-to-one wrappers

def sd_attn_create() -> int:
    h = ctypes.c_void_p()
    rc = load().sd_attn_create(ctypes.byref(h))
    if rc != OK:
        raise SdAttnError(rc, "sd_attn_create")
    return h.value


def sd_attn_create_ex(options: Optional[Options]) -> int:
    """A handle with non-default choices (``Options(no_pdl=1, ...)``); None gives the defaults."""
    h = ctypes.c_void_p()
    rc = load().sd_attn_create_ex(ctypes.byref(options) if options is not None else None, ctypes.byref(h))
    if rc != OK:
        raise SdAttnError(rc, "sd_attn_create_ex")
    return h.value


def sd_attn_static_query_status(stream=0):
    """Status word of sd_attn_forward_twopass_static on the current device: (status, [code, block, site, tile])."""
    detail = (ctypes.c_int * 4)()
    rc = load().sd_attn_static_query_status(stream or None, detail)
    return rc, list(detail)


def sd_attn_destroy(handle: Optional[int]) -> int:
    return load().sd_attn_destroy(handle)


def sd_attn_forward(handle, q, k, v, out, B, H, Nq, Nk, d, scale, dtype, stream=0) -> int:
    """Raw call: q, k, v, out are device addresses (ints).  Returns the status code."""
    return load().sd_attn_forward(handle, q, k, v, out, B, H, Nq, Nk, d, ctypes.c_float(scale), dtype,
                                  stream or None)


def sd_attn_forward_host(handle, q, k, v, out, staging, staging_bytes, B, H, Nq, Nk, d, scale, dtype,
                         stream=0) -> int:
    """Raw call with HOST addresses for q, k, v, out and a device staging buffer."""
    return load().sd_attn_forward_host(handle, q, k, v, out, staging, staging_bytes, B, H, Nq, Nk, d,
                                       ctypes.c_float(scale), dtype, stream or None)


def sd_attn_host_staging_bytes(B, H, Nq, Nk, d, dtype) -> int:
    return int(load().sd_attn_host_staging_bytes(B, H, Nq, Nk, d, dtype))


def sd_attn_forward_twopass_static(q, k, v, out, B, H, Nq, Nk, d, scale, dtype, stream=0) -> int:
    """Two-pass attention on the library's built-in scratch array: no handle, no allocation anywhere.

    For callers that cannot call cudaMalloc (the device heap belongs to someone else).  q, k, v, out are
    device addresses.  Returns the status code; ERR_WORKSPACE when the call needs more scratch than
    ``STATIC_MAX_SCRATCH`` bytes.  Calls that overlap on the GPU race on the shared array.
    """
    return load().sd_attn_forward_twopass_static(q, k, v, out, B, H, Nq, Nk, d, ctypes.c_float(scale), dtype,
                                                 stream or None)


def sd_geglu_forward(x, out, rows: int, C: int, dtype: int, stream=0) -> int:
    """Fused GEGLU (Sec. 3.1, Eq. 2): out[r][c] = x[r][c] * GELU(x[r][C + c]); x is [rows][2C], out [rows][C].

    x and out are device addresses; returns the status code.  No handle: the operation has no state.
    """
    return load().sd_geglu_forward(x or None, out or None, rows, C, dtype, stream or None)


def geglu(x, out=None, stream=None):
    """Marshalling helper for torch tensors: x [..., 2C] (float16 or float32, contiguous, CUDA) -> [..., C]."""
    import torch
    if not x.is_cuda or not x.is_contiguous():
        raise ValueError("x must be a contiguous CUDA tensor")
    if x.dtype not in (torch.float16, torch.float32) or x.shape[-1] % 2:
        raise ValueError("x must be float16 or float32 with an even last dimension")
    C = x.shape[-1] // 2
    if out is None:
        out = torch.empty(x.shape[:-1] + (C,), dtype=x.dtype, device=x.device)
    rows = x.numel() // (2 * C) if C else 0
    s = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    rc = sd_geglu_forward(x.data_ptr(), out.data_ptr(), rows, C, F16 if x.dtype == torch.float16 else F32, s)
    if rc != OK:
        raise SdAttnError(rc, "sd_geglu_forward")
    return out


def sd_groupnorm_forward(x, gamma, beta, y, N: int, C: int, HW: int, G: int, eps: float, dtype: int, stream=0) -> int:
    """Fused group normalisation (Sec. 3.1, Eq. 1) of x [N][C][HW] into y; gamma and beta are [C] or 0 (none).

    All pointers are device addresses; returns the status code.  No handle: the operation has no state.
    """
    return load().sd_groupnorm_forward(x or None, gamma or None, beta or None, y or None, N, C, HW, G,
                                       ctypes.c_float(eps), dtype, stream or None)


def groupnorm(x, groups: int, eps: float = 1e-5, gamma=None, beta=None, out=None, stream=None):
    """Marshalling helper for torch tensors: x [N, C, ...] (float16 or float32, contiguous, CUDA)."""
    import torch
    if not x.is_cuda or not x.is_contiguous() or x.dim() < 2:
        raise ValueError("x must be a contiguous CUDA tensor [N, C, ...]")
    if x.dtype not in (torch.float16, torch.float32):
        raise ValueError("x must be float16 or float32")
    N, C = x.shape[0], x.shape[1]
    HW = x.numel() // (N * C) if N * C else 1
    for t in (gamma, beta):
        if t is not None and (t.dtype != x.dtype or tuple(t.shape) != (C,) or not t.is_cuda or not t.is_contiguous()):
            raise ValueError("gamma and beta must be contiguous CUDA tensors [C] of x's dtype")
    if out is None:
        out = torch.empty_like(x)
    s = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    rc = sd_groupnorm_forward(x.data_ptr(), gamma.data_ptr() if gamma is not None else 0,
                              beta.data_ptr() if beta is not None else 0, out.data_ptr(), N, C, HW, groups, eps,
                              F16 if x.dtype == torch.float16 else F32, s)
    if rc != OK:
        raise SdAttnError(rc, "sd_groupnorm_forward")
    return out


def sd_winograd_filter_elems(K: int, C: int) -> int:
    return int(load().sd_winograd_filter_elems(K, C))


def sd_winograd_transform_filter(w, U, K, C, stream) -> int:
    return load().sd_winograd_transform_filter(w or None, U or None, K, C, stream or None)


def sd_winograd_workspace_bytes(N, H, W, C, K) -> int:
    return int(load().sd_winograd_workspace_bytes(N, H, W, C, K))


def sd_winograd_conv3x3_forward(x, U, bias, y, workspace, workspace_bytes, N, H, W, C, K, stream) -> int:
    return load().sd_winograd_conv3x3_forward(x or None, U or None, bias or None, y or None, workspace or None,
                                              workspace_bytes, N, H, W, C, K, stream or None)


def sd_winograd_query_status(stream=0):
    detail = (ctypes.c_int * 4)()
    rc = load().sd_winograd_query_status(stream or None, detail)
    return rc, list(detail)


class WinogradConv3x3:
    """A layer's transformed filter plus torch-tensor marshalling: ``WinogradConv3x3(w, bias)(x)`` with
    w [K,3,3,C], bias [K] or None, x [N,H,W,C] float16 CUDA tensors (channels-last memory) -> y [N,H,W,K]."""

    def __init__(self, w, bias=None, stream: Optional[int] = None):
        import torch
        if not (w.is_cuda and w.dtype == torch.float16 and w.is_contiguous() and w.dim() == 4 and w.shape[1:3] == (3, 3)):
            raise ValueError("w must be a contiguous float16 CUDA tensor [K,3,3,C]")
        self.K, self.C = int(w.shape[0]), int(w.shape[3])
        self.bias = bias.contiguous() if bias is not None else None
        self.U = torch.empty(sd_winograd_filter_elems(self.K, self.C), dtype=torch.float16, device=w.device)
        s = stream if stream is not None else torch.cuda.current_stream(w.device).cuda_stream
        rc = sd_winograd_transform_filter(w.data_ptr(), self.U.data_ptr(), self.K, self.C, s)
        if rc != OK:
            raise SdAttnError(rc, "sd_winograd_transform_filter")
        self._workspace = None

    def __call__(self, x, out=None, stream: Optional[int] = None):
        import torch
        if not (x.is_cuda and x.dtype == torch.float16 and x.is_contiguous() and x.dim() == 4 and x.shape[3] == self.C):
            raise ValueError("x must be a contiguous float16 CUDA tensor [N,H,W,%d]" % self.C)
        N, H, W, _ = (int(v) for v in x.shape)
        need = sd_winograd_workspace_bytes(N, H, W, self.C, self.K)
        if self._workspace is None or self._workspace.numel() < need:
            self._workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
        if out is None:
            out = torch.empty(N, H, W, self.K, dtype=torch.float16, device=x.device)
        s = stream if stream is not None else torch.cuda.current_stream(x.device).cuda_stream
        rc = sd_winograd_conv3x3_forward(x.data_ptr(), self.U.data_ptr(),
                                         self.bias.data_ptr() if self.bias is not None else 0, out.data_ptr(),
                                         self._workspace.data_ptr(), self._workspace.numel(), N, H, W, self.C, self.K, s)
        if rc != OK:
            raise SdAttnError(rc, "sd_winograd_conv3x3_forward")
        return out


def sd_attn_set_mode(handle, mode: int) -> int:
    return load().sd_attn_set_mode(handle, mode)


def sd_attn_forward_batch(handle, problems, dtype: int, stream) -> int:
    """problems: a ctypes array of Problem (see make_problems) or a sequence of Problem."""
    if not isinstance(problems, ctypes.Array):
        problems = (Problem * len(problems))(*problems)
    return load().sd_attn_forward_batch(handle, problems, len(problems), dtype, stream or None)


def make_problems(items):
    """items: (q_ptr, k_ptr, v_ptr, out_ptr, B, H, Nq, Nk, d, scale) tuples -> a ctypes array of Problem."""
    arr = (Problem * len(items))()
    for p, it in zip(arr, items):
        p.q, p.k, p.v, p.out, p.B, p.H, p.Nq, p.Nk, p.d, p.scale = it
    return arr


def sd_attn_set_layout(handle, layout: int) -> int:
    return load().sd_attn_set_layout(handle, layout)


def sd_attn_workspace_bytes(mode, B, H, Nq, Nk, d, dtype) -> int:
    return int(load().sd_attn_workspace_bytes(mode, B, H, Nq, Nk, d, dtype))


def sd_attn_set_workspace(handle, ptr, nbytes) -> int:
    return load().sd_attn_set_workspace(handle, ptr or None, nbytes)


def sd_attn_twopass_buffers(handle):
    a, s = ctypes.c_void_p(), ctypes.c_void_p()
    rc = load().sd_attn_twopass_buffers(handle, ctypes.byref(a), ctypes.byref(s))
    if rc != OK:
        raise SdAttnError(rc, "sd_attn_twopass_buffers")
    return a.value, s.value


def sd_attn_query_status(handle, stream=0):
    detail = (ctypes.c_int * 4)()
    rc = load().sd_attn_query_status(handle, stream or None, detail)
    return rc, list(detail)


def sd_attn_selftest_wait_timeout(handle, stream=0) -> int:
    """Enqueue the self-test kernel whose bounded wait runs out (see include/sd_attn.h)."""
    return load().sd_attn_selftest_wait_timeout(handle, stream or None)


UBENCH_OPS = {"ex2": 0, "fma": 1, "fma_x2": 2, "softmax_sweep": 3, "softmax_sweep_poly": 4}


def sd_attn_ubench(op: int, iters: int = 4096, stream=0):
    """Instruction-rate probe (see include/sd_attn.h): (results per clock per SM, SM clock in MHz)."""
    rate, mhz = ctypes.c_double(), ctypes.c_double()
    rc = load().sd_attn_ubench(op, iters, stream or None, ctypes.byref(rate), ctypes.byref(mhz))
    if rc != OK:
        raise SdAttnError(rc, "sd_attn_ubench")
    return rate.value, mhz.value


def sd_attn_last_mode(handle) -> int:
    return load().sd_attn_last_mode(handle)


def sd_attn_launch_count(handle) -> int:
    return int(load().sd_attn_launch_count(handle))


# ------------------------------------------------------------------ convenience for torch tensors

class Attention:
    """A handle plus torch-tensor marshalling: ``Attention().forward(q, k, v)``."""

    def __init__(self, mode: int = MODE_AUTO, layout: int = LAYOUT_BHND, options: Optional[Options] = None):
        self.handle = sd_attn_create_ex(options) if options is not None else sd_attn_create()
        self._workspace = None
        self.layout = LAYOUT_BHND
        if mode != MODE_AUTO:
            self.set_mode(mode)
        if layout != LAYOUT_BHND:
            self.set_layout(layout)

    def set_layout(self, layout: int) -> None:
        """LAYOUT_BHND: q [B,H,Nq,d]; LAYOUT_BNHD: q [B,Nq,H,d] (k, v, out alike)."""
        rc = sd_attn_set_layout(self.handle, layout)
        if rc != OK:
            raise SdAttnError(rc, "sd_attn_set_layout")
        self.layout = layout

    def set_mode(self, mode: int) -> None:
        rc = sd_attn_set_mode(self.handle, mode)
        if rc != OK:
            raise SdAttnError(rc, "sd_attn_set_mode")

    def forward(self, q, k, v, scale: Optional[float] = None, out=None, stream: Optional[int] = None):
        import torch
        if not (q.is_cuda and k.is_cuda and v.is_cuda):
            raise ValueError("q, k, v must be CUDA tensors")
        if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous()):
            raise ValueError("q, k, v must be contiguous [B,H,N,d] (or, token-major, [B,N,H,d]) tensors")
        if q.dtype == torch.float16:
            dtype = F16
        elif q.dtype == torch.float32:
            dtype = F32
        elif q.dtype == torch.bfloat16:
            dtype = BF16
        else:
            raise TypeError("float16, bfloat16 or float32 only")
        if self.layout == LAYOUT_BNHD:
            B, Nq, H, d = q.shape
            Nk = k.shape[1]
        else:
            B, H, Nq, d = q.shape
            Nk = k.shape[2]
        if out is None:
            out = torch.empty_like(q)
        if scale is None:
            scale = float(d) ** -0.5
        if stream is None:
            stream = torch.cuda.current_stream(q.device).cuda_stream
        rc = sd_attn_forward(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                             B, H, Nq, Nk, d, scale, dtype, stream)
        if rc == ERR_WORKSPACE:
            need = sd_attn_workspace_bytes(MODE_TWOPASS, B, H, Nq, Nk, d, dtype)
            self._workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
            rc = sd_attn_set_workspace(self.handle, self._workspace.data_ptr(), need)
            if rc == OK:
                rc = sd_attn_forward(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                     B, H, Nq, Nk, d, scale, dtype, stream)
        if rc != OK:
            raise SdAttnError(rc, "sd_attn_forward")
        return out

    def check(self, stream: int = 0) -> None:
        """Synchronise and raise if a kernel reported an expired wait."""
        rc, detail = sd_attn_query_status(self.handle, stream)
        if rc != OK:
            raise SdAttnError(rc, "device status %s" % detail)

    @property
    def last_mode(self) -> int:
        return sd_attn_last_mode(self.handle)

    @property
    def launch_count(self) -> int:
        return sd_attn_launch_count(self.handle)

    def close(self) -> None:
        if self.handle:
            sd_attn_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
