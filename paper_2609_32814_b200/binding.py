"""Thin ctypes binding over libalgproj.so -- argument marshalling only.

Function names mirror ``include/algproj.h``.  PyTorch appears here solely as the owner of device
memory and streams: tensors are turned into raw pointers and every step of the path runs inside
the CUDA library.  There is no CPU or eager fallback; a missing library is an error.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libalgproj.so")

ALG_OK = 0
STATUS = {0: "ALG_OK", 1: "ALG_ERR_INVALID_ARG", 2: "ALG_ERR_UNSUPPORTED_SHAPE", 3: "ALG_ERR_WORKSPACE_TOO_SMALL",
          4: "ALG_ERR_CUDA", 5: "ALG_ERR_BAD_TYPE", 6: "ALG_ERR_DEVICE_TIMEOUT"}
ALG_F32, ALG_BF16 = 0, 1
ALG_TABLE_QQ, ALG_TABLE_DENSE, ALG_TABLE_CUSTOM, ALG_TABLE_Q2POW = 0, 1, 2, 3
ALG_ACT_NONE, ALG_ACT_GELU_ERF, ALG_ACT_GELU_TANH = 0, 1, 2
ALG_SCHED_EXPLICIT, ALG_SCHED_CYCLIC, ALG_SCHED_INTERVAL = 0, 1, 2
ALG_PATH_SIMT, ALG_PATH_TCGEN05, ALG_PATH_DECODE = 0, 1, 2
OPTIONS = {"gemm_kernel": 1, "tile_n": 2, "small_m_kernel": 3, "host_plan": 4, "wait_limit_cycles": 5,
           "test_stall_bytes": 6, "stage_k": 7, "interval_period": 8, "row_gather": 9, "weight_packed": 10}

_DTYPES = {"f32": ALG_F32, "bf16": ALG_BF16, torch.float32: ALG_F32, torch.bfloat16: ALG_BF16}
_TABLES = {"qq": ALG_TABLE_QQ, "dense": ALG_TABLE_DENSE, "custom": ALG_TABLE_CUSTOM, "q2pow": ALG_TABLE_Q2POW}
_ACTS = {None: ALG_ACT_NONE, "none": ALG_ACT_NONE, "gelu": ALG_ACT_GELU_ERF, "gelu_erf": ALG_ACT_GELU_ERF,
         "gelu_tanh": ALG_ACT_GELU_TANH}
_SCHEDS = {"explicit": ALG_SCHED_EXPLICIT, "cyclic": ALG_SCHED_CYCLIC, "interval": ALG_SCHED_INTERVAL}

EXPORTS = [
    "alg_proj_create", "alg_proj_destroy", "alg_proj_set_option", "alg_ffn_set_option", "alg_proj_workspace_bytes", "alg_proj_forward", "alg_proj_gemm_count",
    "alg_proj_forward_static", "alg_proj_host_workspace_bytes", "alg_proj_forward_host", "alg_proj_packed_weight_bytes", "alg_proj_pack_weight", "alg_proj_macs", "alg_proj_kernel_path", "alg_proj_last_status", "alg_ffn_create", "alg_ffn_destroy",
    "alg_ffn_workspace_bytes", "alg_ffn_forward", "alg_ffn_host_workspace_bytes", "alg_ffn_forward_host",
    "alg_ffn_gated_create", "alg_ffn_gated_forward", "alg_proj_grad_create", "alg_proj_grad_destroy",
    "alg_proj_grad_workspace_bytes", "alg_proj_grad_input", "alg_proj_grad_weight", "alg_proj_grad_last_status", "alg_ffn_macs", "alg_ffn_last_status", "alg_ffn_set_timing", "alg_ffn_get_timing", "alg_status_string", "alg_launch_count",
]

_lib = None


class AlgError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where}: {STATUS.get(code, code)}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Load libalgproj.so (built by ``python -m paper_2609_32814_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_32814_b200.build`; "
                "there is no fallback implementation")
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
        L.alg_proj_create.argtypes = [ctypes.POINTER(vp), i32, vp, vp, i32, i32, vp, i32]
        L.alg_proj_destroy.argtypes = [vp]
        L.alg_proj_set_option.argtypes = [vp, i32, i64]
        L.alg_ffn_set_option.argtypes = [vp, i32, i64]
        L.alg_proj_workspace_bytes.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_proj_forward.argtypes = [vp, vp, i64, vp, i64, vp, i64, vp, i32, vp, i64, i32, vp, ctypes.c_size_t, vp]
        L.alg_proj_forward_static.argtypes = [vp, vp, i64, vp, i64, vp, i64, vp, i32, vp, i64, i32, vp]
        L.alg_proj_host_workspace_bytes.argtypes = [vp, i64, i32, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_proj_packed_weight_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_proj_pack_weight.argtypes = [vp, vp, i64, vp, ctypes.c_size_t, vp]
        L.alg_proj_forward_host.argtypes = [vp, vp, vp, i64, vp, i64, vp, i32, vp, i32, vp, ctypes.c_size_t, vp]
        L.alg_proj_gemm_count.argtypes = [vp, ctypes.POINTER(i64)]
        L.alg_proj_macs.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.alg_proj_kernel_path.argtypes = [vp, i64, ctypes.POINTER(i32)]
        L.alg_proj_last_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.alg_ffn_create.argtypes = [ctypes.POINTER(vp), i32, vp, vp, i32, i32, vp, i32]
        L.alg_ffn_destroy.argtypes = [vp]
        L.alg_proj_grad_create.argtypes = [ctypes.POINTER(vp), i32, vp, vp, i32, vp, i32]
        L.alg_proj_grad_destroy.argtypes = [vp]
        L.alg_proj_grad_workspace_bytes.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_proj_grad_input.argtypes = [vp, vp, i64, vp, i64, vp, i64, vp, i64, i32, vp, ctypes.c_size_t, vp]
        L.alg_proj_grad_weight.argtypes = [vp, vp, i64, vp, i64, vp, i64, vp, i64, i32, vp, ctypes.c_size_t, vp]
        L.alg_proj_grad_last_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.alg_ffn_gated_create.argtypes = [ctypes.POINTER(vp), i32, vp, vp, i32, i32, vp, i32]
        L.alg_ffn_gated_forward.argtypes = [vp, vp, vp, i64, vp, vp, vp, i32, vp, ctypes.c_size_t, vp]
        L.alg_ffn_workspace_bytes.argtypes = [vp, i64, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_ffn_forward.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, i32, vp, i32, vp, ctypes.c_size_t, vp]
        L.alg_ffn_host_workspace_bytes.argtypes = [vp, i64, i32, ctypes.POINTER(ctypes.c_size_t)]
        L.alg_ffn_forward_host.argtypes = [vp, vp, vp, i64, vp, vp, vp, vp, i32, vp, i32, vp, ctypes.c_size_t, vp]
        L.alg_ffn_macs.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.alg_ffn_last_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        L.alg_ffn_set_timing.argtypes = [vp, i32]
        L.alg_ffn_get_timing.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
        L.alg_status_string.argtypes = [i32]
        L.alg_status_string.restype = ctypes.c_char_p
        L.alg_launch_count.argtypes = []
        L.alg_launch_count.restype = i64
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != ALG_OK:
        raise AlgError(code, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _widths(w):
    arr = (ctypes.c_int32 * len(w))(*[int(v) for v in w])
    return arr


def launch_count() -> int:
    return int(lib().alg_launch_count())


class _Handle:
    _destroy = None
    _set_option = None

    def __init__(self):
        self._h = ctypes.c_void_p()
        self._ws = None

    def close(self):
        if self._h:
            getattr(lib(), self._destroy)(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_option(self, name: str, value: int):
        """alg_*_set_option: per-handle switches (see OPTIONS and the header)."""
        _check(getattr(lib(), self._set_option)(self._h, OPTIONS[name], int(value)), self._set_option)

    def _workspace(self, nbytes: int, device) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes or self._ws.device != device:
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        return self._ws


def _keep_arg(table, custom_keep, q):
    if _TABLES[table] != ALG_TABLE_CUSTOM:
        return None, None
    flat = [int(bool(v)) for v in custom_keep.reshape(-1).tolist()]
    if len(flat) != q * q * q:
        raise ValueError("custom_keep must hold q*q*q entries")
    buf = (ctypes.c_uint8 * len(flat))(*flat)
    return buf, ctypes.cast(buf, ctypes.c_void_p)


class Proj(_Handle):
    """alg_proj_* : Y = act(X *_q W + bias)."""
    _destroy = "alg_proj_destroy"
    _set_option = "alg_proj_set_option"

    def __init__(self, in_widths, out_widths, dtype="bf16", table="qq", custom_keep=None, schedule="explicit"):
        super().__init__()
        self.q = len(in_widths)
        self.in_widths, self.out_widths = list(in_widths), list(out_widths)
        self.K, self.N = sum(self.in_widths), sum(self.out_widths)
        self.dtype = _DTYPES[dtype]
        self.schedule = _SCHEDS[schedule]
        buf, keep = _keep_arg(table, custom_keep, self.q)
        s, r = _widths(in_widths), _widths(out_widths)
        _check(lib().alg_proj_create(ctypes.byref(self._h), self.q, ctypes.cast(s, ctypes.c_void_p),
                                     ctypes.cast(r, ctypes.c_void_p), self.dtype, _TABLES[table], keep,
                                     self.schedule), "alg_proj_create")

    def workspace_bytes(self, max_M: int) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_proj_workspace_bytes(self._h, max_M, ctypes.byref(out)), "alg_proj_workspace_bytes")
        return out.value

    def forward(self, X, types, W, bias=None, act=None, out=None, out_dtype=None, workspace=None, stream=None):
        M = X.shape[0]
        if out is None:
            out = torch.empty((M, self.N), dtype=out_dtype or X.dtype, device=X.device)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(M), X.device)
        _check(lib().alg_proj_forward(self._h, _ptr(X), X.stride(0) if M else self.K, _ptr(types), M, _ptr(W),
                                      W.stride(0), _ptr(bias), _ACTS[act], _ptr(out),
                                      out.stride(0) if M else self.N, _DTYPES[out.dtype], _ptr(ws), ws.numel(),
                                      _stream(stream)), "alg_proj_forward")
        return out

    def forward_static(self, X, types, W, out, bias=None, act=None, stream=None):
        """alg_proj_forward_static: same result as forward(), but the scratch is the fixed array
        inside the library, so nothing is allocated -- `out` must be supplied by the caller, and
        problems needing more than the built-in scratch raise ALG_ERR_WORKSPACE_TOO_SMALL."""
        M = X.shape[0]
        _check(lib().alg_proj_forward_static(self._h, _ptr(X), X.stride(0) if M else self.K, _ptr(types), M,
                                             _ptr(W), W.stride(0), _ptr(bias), _ACTS[act], _ptr(out),
                                             out.stride(0) if M else self.N, _DTYPES[out.dtype], _stream(stream)),
               "alg_proj_forward_static")
        return out

    def packed_weight_bytes(self) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_proj_packed_weight_bytes(self._h, ctypes.byref(out)), "alg_proj_packed_weight_bytes")
        return out.value

    def pack_weight(self, W, stream=None):
        """alg_proj_pack_weight: the padded bank as a flat bf16 tensor (pass it to forward with option weight_packed = 1)."""
        out = torch.empty(self.packed_weight_bytes() // 2, dtype=torch.bfloat16, device=W.device)
        _check(lib().alg_proj_pack_weight(self._h, _ptr(W), W.stride(0), _ptr(out), out.numel() * 2, _stream(stream)),
               "alg_proj_pack_weight")
        return out

    def host_workspace_bytes(self, max_M: int, out_dtype) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_proj_host_workspace_bytes(self._h, max_M, _DTYPES[out_dtype], ctypes.byref(out)),
               "alg_proj_host_workspace_bytes")
        return out.value

    def forward_host(self, X_host, types_host, W, Y_host, bias=None, act=None, workspace=None, stream=None):
        """alg_proj_forward_host: X_host / types_host / Y_host are packed CPU tensors (pinned for asynchronous copies)."""
        M = X_host.shape[0]
        need = self.host_workspace_bytes(M, Y_host.dtype)
        ws = workspace if workspace is not None else self._workspace(need, W.device)
        _check(lib().alg_proj_forward_host(self._h, _ptr(X_host), _ptr(types_host), M, _ptr(W), W.stride(0), _ptr(bias),
                                           _ACTS[act], _ptr(Y_host), _DTYPES[Y_host.dtype], _ptr(ws), ws.numel(),
                                           _stream(stream)), "alg_proj_forward_host")
        return Y_host

    def gemm_count(self) -> int:
        n = ctypes.c_int64()
        _check(lib().alg_proj_gemm_count(self._h, ctypes.byref(n)), "alg_proj_gemm_count")
        return n.value

    def macs(self, rows_per_type) -> int:
        rows = (ctypes.c_int64 * self.q)(*[int(v) for v in rows_per_type])
        out = ctypes.c_int64()
        _check(lib().alg_proj_macs(self._h, rows, ctypes.byref(out)), "alg_proj_macs")
        return out.value

    def kernel_path(self, M: int) -> int:
        p = ctypes.c_int()
        _check(lib().alg_proj_kernel_path(self._h, M, ctypes.byref(p)), "alg_proj_kernel_path")
        return p.value

    def last_status(self, stream=None) -> int:
        s = ctypes.c_int()
        _check(lib().alg_proj_last_status(self._h, _stream(stream), ctypes.byref(s)), "alg_proj_last_status")
        return s.value


class FFN(_Handle):
    """alg_ffn_* : Y = act(X *_q W_up + b_up) *_q W_down + b_down."""
    _destroy = "alg_ffn_destroy"
    _set_option = "alg_ffn_set_option"
    _create = "alg_ffn_create"

    def __init__(self, d_widths, f_widths, dtype="bf16", table="qq", custom_keep=None, schedule="explicit"):
        super().__init__()
        self.q = len(d_widths)
        self.D, self.F = sum(d_widths), sum(f_widths)
        self.dtype = _DTYPES[dtype]
        self.schedule = _SCHEDS[schedule]
        buf, keep = _keep_arg(table, custom_keep, self.q)
        d, f = _widths(d_widths), _widths(f_widths)
        _check(getattr(lib(), self._create)(ctypes.byref(self._h), self.q, ctypes.cast(d, ctypes.c_void_p),
                                            ctypes.cast(f, ctypes.c_void_p), self.dtype, _TABLES[table], keep,
                                            self.schedule), self._create)

    def workspace_bytes(self, max_M: int) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_ffn_workspace_bytes(self._h, max_M, ctypes.byref(out)), "alg_ffn_workspace_bytes")
        return out.value

    def host_workspace_bytes(self, max_M: int, out_dtype) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_ffn_host_workspace_bytes(self._h, max_M, _DTYPES[out_dtype], ctypes.byref(out)),
               "alg_ffn_host_workspace_bytes")
        return out.value

    def forward(self, X, types, W_up, W_down, b_up=None, b_down=None, act="gelu", out=None, out_dtype=None,
                workspace=None, stream=None):
        M = X.shape[0]
        if not (X.is_contiguous() and W_up.is_contiguous() and W_down.is_contiguous()):
            raise ValueError("alg_ffn_forward takes packed row-major tensors")
        if out is None:
            out = torch.empty((M, self.D), dtype=out_dtype or X.dtype, device=X.device)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(M), X.device)
        _check(lib().alg_ffn_forward(self._h, _ptr(X), _ptr(types), M, _ptr(W_up), _ptr(b_up), _ptr(W_down),
                                     _ptr(b_down), _ACTS[act], _ptr(out), _DTYPES[out.dtype], _ptr(ws), ws.numel(),
                                     _stream(stream)), "alg_ffn_forward")
        return out

    def forward_host(self, X_host, types_host, W_up, W_down, Y_host, b_up=None, b_down=None, act="gelu",
                     workspace=None, stream=None):
        """X_host / types_host / Y_host are CPU tensors (pinned for asynchronous copies)."""
        M = X_host.shape[0]
        need = self.host_workspace_bytes(M, Y_host.dtype)
        ws = workspace if workspace is not None else self._workspace(need, W_up.device)
        _check(lib().alg_ffn_forward_host(self._h, _ptr(X_host), _ptr(types_host), M, _ptr(W_up), _ptr(b_up),
                                          _ptr(W_down), _ptr(b_down), _ACTS[act], _ptr(Y_host), _DTYPES[Y_host.dtype],
                                          _ptr(ws), ws.numel(), _stream(stream)), "alg_ffn_forward_host")
        return Y_host

    def set_timing(self, enable: bool):
        _check(lib().alg_ffn_set_timing(self._h, int(enable)), "alg_ffn_set_timing")

    def get_timing(self):
        """Milliseconds of the last forward call: (bucketing, gather, up projection, down projection)."""
        ms = (ctypes.c_float * 4)()
        _check(lib().alg_ffn_get_timing(self._h, ms), "alg_ffn_get_timing")
        return tuple(float(v) for v in ms)

    def macs(self, rows_per_type) -> int:
        rows = (ctypes.c_int64 * self.q)(*[int(v) for v in rows_per_type])
        out = ctypes.c_int64()
        _check(lib().alg_ffn_macs(self._h, rows, ctypes.byref(out)), "alg_ffn_macs")
        return out.value

    def last_status(self, stream=None) -> int:
        s = ctypes.c_int()
        _check(lib().alg_ffn_last_status(self._h, _stream(stream), ctypes.byref(s)), "alg_ffn_last_status")
        return s.value


class GatedFFN(FFN):
    """alg_ffn_gated_* : Y = (silu(X *_q W_gate) .* (X *_q W_up)) *_q W_down, W_gate_up = [W_gate | W_up] (D x 2F)."""
    _create = "alg_ffn_gated_create"

    def forward(self, X, types, W_gate_up, W_down, out=None, out_dtype=None, workspace=None, stream=None):
        M = X.shape[0]
        if not (X.is_contiguous() and W_gate_up.is_contiguous() and W_down.is_contiguous()):
            raise ValueError("alg_ffn_gated_forward takes packed row-major tensors")
        if W_gate_up.shape != (self.D, 2 * self.F):
            raise ValueError("W_gate_up must be D x 2F: [W_gate | W_up]")
        if out is None:
            out = torch.empty((M, self.D), dtype=out_dtype or X.dtype, device=X.device)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(M), X.device)
        _check(lib().alg_ffn_gated_forward(self._h, _ptr(X), _ptr(types), M, _ptr(W_gate_up), _ptr(W_down), _ptr(out),
                                           _DTYPES[out.dtype], _ptr(ws), ws.numel(), _stream(stream)),
               "alg_ffn_gated_forward")
        return out

    def forward_host(self, *a, **k):
        raise NotImplementedError("the gated FFN has no host entry point")


class ProjGrad(_Handle):
    """alg_proj_grad_* : the two gradient maps of Y = X *_q W (dX from G and W, dW from X and G)."""
    _destroy = "alg_proj_grad_destroy"

    def __init__(self, in_widths, out_widths, table="qq", custom_keep=None, schedule="explicit"):
        super().__init__()
        self.q = len(in_widths)
        self.K, self.N = sum(in_widths), sum(out_widths)
        self.schedule = _SCHEDS[schedule]
        buf, keep = _keep_arg(table, custom_keep, self.q)
        s, r = _widths(in_widths), _widths(out_widths)
        _check(lib().alg_proj_grad_create(ctypes.byref(self._h), self.q, ctypes.cast(s, ctypes.c_void_p),
                                          ctypes.cast(r, ctypes.c_void_p), _TABLES[table], keep, self.schedule),
               "alg_proj_grad_create")

    def workspace_bytes(self, max_M: int) -> int:
        out = ctypes.c_size_t()
        _check(lib().alg_proj_grad_workspace_bytes(self._h, max_M, ctypes.byref(out)), "alg_proj_grad_workspace_bytes")
        return out.value

    def grad_input(self, G, types, W, out=None, out_dtype=None, workspace=None, stream=None):
        M = G.shape[0]
        if out is None:
            out = torch.empty((M, self.K), dtype=out_dtype or G.dtype, device=G.device)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(M), G.device)
        _check(lib().alg_proj_grad_input(self._h, _ptr(G), G.stride(0) if M else self.N, _ptr(types), M, _ptr(W), W.stride(0),
                                         _ptr(out), out.stride(0) if M else self.K, _DTYPES[out.dtype], _ptr(ws), ws.numel(),
                                         _stream(stream)), "alg_proj_grad_input")
        return out

    def grad_weight(self, X, G, types, out=None, out_dtype=torch.float32, workspace=None, stream=None):
        M = X.shape[0]
        if out is None:
            out = torch.empty((self.K, self.N), dtype=out_dtype, device=X.device)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(M), X.device)
        _check(lib().alg_proj_grad_weight(self._h, _ptr(X), X.stride(0) if M else self.K, _ptr(G), G.stride(0) if M else self.N,
                                          _ptr(types), M, _ptr(out), out.stride(0), _DTYPES[out.dtype], _ptr(ws), ws.numel(),
                                          _stream(stream)), "alg_proj_grad_weight")
        return out

    def last_status(self, stream=None) -> int:
        s = ctypes.c_int()
        _check(lib().alg_proj_grad_last_status(self._h, _stream(stream), ctypes.byref(s)), "alg_proj_grad_last_status")
        return s.value
