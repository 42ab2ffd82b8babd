"""CPU oracle for the row-typed projection Y = X *_q W -- TEST INFRASTRUCTURE ONLY.

This package wraps ``star_oracle.c`` (plain fp64 loops written from the paper's definition,
Eqs. typed-diag / typed-off / recursive-row-action, Algorithm 1, Eqs. q-product-diag/off).
It is independent of the CUDA library: it imports nothing from the product package and the
product package imports nothing from here.  Only tests, the smoke check and the benchmark's
CPU-baseline leg may use it.

Parity unpinned by the paper: FFN-level choices (erf-GELU, bias before the activation).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "star_oracle.c")
_LIB = os.path.join(_HERE, "libstar_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP). Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p, f64p, u8p, i64p = (ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double),
                                 ctypes.POINTER(ctypes.c_uint8), ctypes.POINTER(ctypes.c_int64))
        i64 = ctypes.c_int64
        lib.star_oracle_threads.restype = ctypes.c_int
        for name in ("star_support_qq", "star_support_dense", "star_support_q2_power"):
            getattr(lib, name).argtypes = [ctypes.c_int, u8p]
        lib.star_gemm_count.restype = i64
        lib.star_gemm_count.argtypes = [ctypes.c_int, u8p]
        lib.star_macs.restype = i64
        lib.star_macs.argtypes = [ctypes.c_int, u8p, i32p, i32p, i64p]
        lib.star_proj_rows.argtypes = [f64p, i64, i32p, i64, f64p, i64, f64p, f64p, i64,
                                       ctypes.c_int, i32p, i32p, u8p]
        lib.star_proj_alg1.argtypes = [f64p, i64, i32p, i64, f64p, i64, f64p, i64,
                                       ctypes.c_int, i32p, i32p, u8p]
        lib.star_proj_entries.argtypes = [f64p, i64, i32p, i64, f64p, i64, f64p, ctypes.c_int, i32p, i32p, u8p,
                                          i64p, i64p, i64, f64p]
        lib.star_gelu_array.argtypes = [f64p, i64]
        lib.star_gelu_array.restype = None
        lib.star_square.argtypes = [f64p, f64p, f64p, ctypes.c_int, i32p, i32p, i32p]
        lib.star_gelu.restype = ctypes.c_double
        lib.star_gelu.argtypes = [ctypes.c_double]
        lib.star_ffn.argtypes = [f64p, i32p, i64, f64p, f64p, f64p, f64p, f64p, f64p,
                                 ctypes.c_int, i32p, i32p, u8p]
        lib.star_proj_vjp_x.argtypes = [f64p, i64, i32p, i64, f64p, i64, f64p, i64, ctypes.c_int, i32p, i32p, u8p]
        lib.star_proj_vjp_w.argtypes = [f64p, i64, f64p, i64, i32p, i64, f64p, i64, ctypes.c_int, i32p, i32p, u8p]
        lib.star_silu.restype = ctypes.c_double
        lib.star_silu.argtypes = [ctypes.c_double]
        lib.star_ffn_swiglu.argtypes = [f64p, i32p, i64, f64p, f64p, f64p, f64p, f64p, f64p, f64p,
                                        ctypes.c_int, i32p, i32p, u8p]
        _lib = lib
    return _lib


def _p(a, ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


class OracleError(ValueError):
    pass


def _check(rc):
    if rc == 2:
        raise OracleError("row type outside [0, q)")
    if rc != 0:
        raise OracleError(f"oracle rejected its arguments (code {rc})")


def threads() -> int:
    return int(_load().star_oracle_threads())


def support(q: int, law: str = "qq") -> np.ndarray:
    """keep[i, j, k] = 1 iff a type-i row adds x_k W_kj into output group j.

    law: "qq" (complete-graph Q_q, B(i,j)={i,j}), "dense", or "q2pow" (Q_2 tensor power,
    q must be a power of two)."""
    lib = _load()
    keep = np.zeros((q, q, q), dtype=np.uint8)
    if law == "qq":
        _check(lib.star_support_qq(q, _p(keep, ctypes.c_uint8)))
    elif law == "dense":
        _check(lib.star_support_dense(q, _p(keep, ctypes.c_uint8)))
    elif law == "q2pow":
        L = int(q).bit_length() - 1
        if (1 << L) != q:
            raise OracleError("q must be a power of two for the tensor-power law")
        _check(lib.star_support_q2_power(L, _p(keep, ctypes.c_uint8)))
    else:
        raise OracleError(f"unknown law {law!r}")
    return keep


def gemm_count(keep: np.ndarray) -> int:
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    return int(_load().star_gemm_count(keep.shape[0], _p(keep, ctypes.c_uint8)))


def macs(keep, s, r, rows_per_type) -> int:
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    s, r = _i32(s), _i32(r)
    rows = np.ascontiguousarray(rows_per_type, dtype=np.int64)
    return int(_load().star_macs(keep.shape[0], _p(keep, ctypes.c_uint8), _p(s, ctypes.c_int32),
                                 _p(r, ctypes.c_int32), _p(rows, ctypes.c_int64)))


def proj(X, types, W, s, r, keep=None, bias=None, form: str = "rows") -> np.ndarray:
    """Y = X *_q W for row types `types` (0-based).  form="rows" follows the per-row equation,
    form="alg1" the batched order of Algorithm 1 (no bias)."""
    lib = _load()
    X, W, types, s, r = _f64(X), _f64(W), _i32(types), _i32(s), _i32(r)
    q = len(s)
    if keep is None:
        keep = support(q, "qq")
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    M, K = X.shape
    K2, N = W.shape
    if K != K2 or int(s.sum()) != K or int(r.sum()) != N or len(r) != q or len(types) != M:
        raise OracleError("shape mismatch")
    if keep.shape != (q, q, q):
        raise OracleError("keep must be q x q x q")
    Y = np.empty((M, N), dtype=np.float64)
    f64, i32, u8 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8
    if form == "rows":
        b = None if bias is None else _f64(bias)
        _check(lib.star_proj_rows(_p(X, f64), K, _p(types, i32), M, _p(W, f64), N, _p(b, f64),
                                  _p(Y, f64), N, q, _p(s, i32), _p(r, i32), _p(keep, u8)))
    elif form == "alg1":
        if bias is not None:
            raise OracleError("Algorithm 1 has no bias")
        _check(lib.star_proj_alg1(_p(X, f64), K, _p(types, i32), M, _p(W, f64), N, _p(Y, f64), N,
                                  q, _p(s, i32), _p(r, i32), _p(keep, u8)))
    else:
        raise OracleError(f"unknown form {form!r}")
    return Y


def proj_entries(X, types, W, s, r, rows, cols, keep=None, bias=None) -> np.ndarray:
    """Single outputs Y[rows[e], cols[e]] of proj(), each summed straight from the definition."""
    lib = _load()
    X, W, types, s, r = _f64(X), _f64(W), _i32(types), _i32(s), _i32(r)
    q = len(s)
    if keep is None:
        keep = support(q, "qq")
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    M, K = X.shape
    K2, N = W.shape
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    if K != K2 or int(s.sum()) != K or int(r.sum()) != N or len(r) != q or len(types) != M or rows.shape != cols.shape:
        raise OracleError("shape mismatch")
    out = np.empty(rows.shape, dtype=np.float64)
    b = None if bias is None else _f64(bias)
    f64, i32, u8, i64 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8, ctypes.c_int64
    _check(lib.star_proj_entries(_p(X, f64), K, _p(types, i32), M, _p(W, f64), N, _p(b, f64), q, _p(s, i32),
                                 _p(r, i32), _p(keep, u8), _p(rows, i64), _p(cols, i64), rows.size, _p(out, f64)))
    return out


def gelu_array(z) -> np.ndarray:
    """Exact GELU of every element (a new fp64 array)."""
    out = np.array(z, dtype=np.float64, order="C", copy=True)
    _load().star_gelu_array(_p(out, ctypes.c_double), out.size)
    return out


def ffn_entries(X, types, W_up, W_down, dw, fw, rows, cols, keep=None, b_up=None, b_down=None) -> np.ndarray:
    """Single outputs Y[rows[e], cols[e]] of ffn(): the hidden rows the entries need are computed in
    full (fp64, never rounded), the entries of the second projection one by one."""
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    uniq, inv = np.unique(rows, return_inverse=True)
    types = _i32(types)
    H = gelu_array(proj(_f64(X)[uniq], types[uniq], W_up, dw, fw, keep=keep, bias=b_up))
    return proj_entries(H, types[uniq], W_down, fw, dw, inv, cols, keep=keep, bias=b_down)


def square(A, B, a, c, d) -> np.ndarray:
    """C = A *_q B on q x q block arrays; block (i,k) of A is a[i] x c[k], (k,j) of B c[k] x d[j]."""
    lib = _load()
    A, B, a, c, d = _f64(A), _f64(B), _i32(a), _i32(c), _i32(d)
    q = len(a)
    if A.shape != (a.sum(), c.sum()) or B.shape != (c.sum(), d.sum()) or len(c) != q or len(d) != q:
        raise OracleError("shape mismatch")
    C = np.empty((int(a.sum()), int(d.sum())), dtype=np.float64)
    f64, i32 = ctypes.c_double, ctypes.c_int32
    _check(lib.star_square(_p(A, f64), _p(B, f64), _p(C, f64), q, _p(a, i32), _p(c, i32), _p(d, i32)))
    return C


def gelu(z: float) -> float:
    return float(_load().star_gelu(float(z)))


def ffn(X, types, W_up, W_down, dw, fw, keep=None, b_up=None, b_down=None, return_hidden=False):
    """Y = gelu(X *_q W_up + b_up) *_q W_down + b_down with the hidden state kept in fp64."""
    lib = _load()
    X, W_up, W_down, types, dw, fw = _f64(X), _f64(W_up), _f64(W_down), _i32(types), _i32(dw), _i32(fw)
    q = len(dw)
    if keep is None:
        keep = support(q, "qq")
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    M, D = X.shape
    F = int(fw.sum())
    if int(dw.sum()) != D or W_up.shape != (D, F) or W_down.shape != (F, D) or len(types) != M:
        raise OracleError("shape mismatch")
    bu = None if b_up is None else _f64(b_up)
    bd = None if b_down is None else _f64(b_down)
    H = np.empty((M, F), dtype=np.float64)
    Y = np.empty((M, D), dtype=np.float64)
    f64, i32, u8 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8
    _check(lib.star_ffn(_p(X, f64), _p(types, i32), M, _p(W_up, f64), _p(bu, f64), _p(W_down, f64),
                        _p(bd, f64), _p(H, f64), _p(Y, f64), q, _p(dw, i32), _p(fw, i32), _p(keep, u8)))
    return (Y, H) if return_hidden else Y


def silu(g: float) -> float:
    return float(_load().star_silu(float(g)))


def ffn_swiglu(X, types, W_gate, W_up, W_down, dw, fw, keep=None, return_hidden=False):
    """Y = (silu(X *_q W_gate) .* (X *_q W_up)) *_q W_down, hidden state kept in fp64, no biases."""
    lib = _load()
    X, W_gate, W_up, W_down = _f64(X), _f64(W_gate), _f64(W_up), _f64(W_down)
    types, dw, fw = _i32(types), _i32(dw), _i32(fw)
    q = len(dw)
    if keep is None:
        keep = support(q, "qq")
    keep = np.ascontiguousarray(keep, dtype=np.uint8)
    M, D = X.shape
    F = int(fw.sum())
    if int(dw.sum()) != D or W_gate.shape != (D, F) or W_up.shape != (D, F) or W_down.shape != (F, D) or len(types) != M:
        raise OracleError("shape mismatch")
    G, U, H = (np.empty((M, F), dtype=np.float64) for _ in range(3))
    Y = np.empty((M, D), dtype=np.float64)
    f64, i32, u8 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8
    _check(lib.star_ffn_swiglu(_p(X, f64), _p(types, i32), M, _p(W_gate, f64), _p(W_up, f64), _p(W_down, f64),
                               _p(G, f64), _p(U, f64), _p(H, f64), _p(Y, f64), q, _p(dw, i32), _p(fw, i32), _p(keep, u8)))
    return (Y, H) if return_hidden else Y


def proj_vjp_x(G, types, W, s, r, keep=None) -> np.ndarray:
    """dX of Y = X *_q W for the output gradient G (M x N): same block support as the forward pass."""
    lib = _load()
    G, W, types, s, r = _f64(G), _f64(W), _i32(types), _i32(s), _i32(r)
    q = len(s)
    keep = np.ascontiguousarray(support(q, "qq") if keep is None else keep, dtype=np.uint8)
    M, N = G.shape
    K = int(s.sum())
    if W.shape != (K, N) or int(r.sum()) != N or len(types) != M:
        raise OracleError("shape mismatch")
    dX = np.empty((M, K), dtype=np.float64)
    f64, i32, u8 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8
    _check(lib.star_proj_vjp_x(_p(G, f64), N, _p(types, i32), M, _p(W, f64), N, _p(dX, f64), K, q, _p(s, i32),
                               _p(r, i32), _p(keep, u8)))
    return dX


def proj_vjp_w(X, G, types, s, r, keep=None) -> np.ndarray:
    """dW of Y = X *_q W for the output gradient G: blocks no row reaches are zero."""
    lib = _load()
    X, G, types, s, r = _f64(X), _f64(G), _i32(types), _i32(s), _i32(r)
    q = len(s)
    keep = np.ascontiguousarray(support(q, "qq") if keep is None else keep, dtype=np.uint8)
    M, K = X.shape
    N = int(r.sum())
    if G.shape != (M, N) or int(s.sum()) != K or len(types) != M:
        raise OracleError("shape mismatch")
    dW = np.empty((K, N), dtype=np.float64)
    f64, i32, u8 = ctypes.c_double, ctypes.c_int32, ctypes.c_uint8
    _check(lib.star_proj_vjp_w(_p(X, f64), K, _p(G, f64), N, _p(types, i32), M, _p(dW, f64), N, q, _p(s, i32),
                               _p(r, i32), _p(keep, u8)))
    return dW
