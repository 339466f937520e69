"""ctypes front-end of the fp64 CPU oracle (``conv_oracle.c``).  TEST INFRASTRUCTURE ONLY.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this module.
It knows nothing about the CUDA library and imports nothing from the product package.

The arithmetic lives entirely in ``conv_oracle.c``; this file compiles it with gcc, widens fp32
arrays to fp64 exactly (every fp32 value is representable in fp64) and marshals pointers.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "conv_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_conv.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile ``conv_oracle.c`` into a shared library next to it and return its path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-Wall", "-Wextra",
                   "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i = ctypes.c_int
        ll = ctypes.c_longlong
        lib.oracle_conv_out_dim.argtypes = [i, i, i, i]
        lib.oracle_conv_out_dim.restype = i
        lib.oracle_conv_fwd_f64.argtypes = [dp, dp, dp, dp] + [i] * 10
        lib.oracle_conv_fwd_f64.restype = i
        lib.oracle_maxpool_fwd_f64.argtypes = [dp, dp] + [i] * 6
        lib.oracle_maxpool_fwd_f64.restype = i
        lib.oracle_conv_macs.argtypes = [i] * 9
        lib.oracle_conv_macs.restype = ll
        lib.oracle_conv_min_bytes.argtypes = [i] * 9
        lib.oracle_conv_min_bytes.restype = ll
        lib.oracle_sgemm_ai.argtypes = [ll, ll, ll]
        lib.oracle_sgemm_ai.restype = ctypes.c_double
        lib.oracle_sgemm_f64.argtypes = [dp, dp, dp, i, i, i]
        lib.oracle_sgemm_f64.restype = i
        lib.oracle_softmax_f64.argtypes = [dp, dp, i, i]
        lib.oracle_softmax_f64.restype = i
        lib.oracle_num_threads.argtypes = []
        lib.oracle_num_threads.restype = i
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float64)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def conv_out_dim(in_dim: int, ksz: int, stride: int, pad: int) -> int:
    """Output extent 1 + (in + 2*pad - ksz) // stride (Section 2 of the paper); 0 if it does not fit."""
    return int(_load().oracle_conv_out_dim(in_dim, ksz, stride, pad))


def conv_fwd(x, filt, bias=None, *, stride: int = 1, pad: int = 0, relu: bool = False) -> np.ndarray:
    """fp64 direct convolution.  x [N,C,H,W], filt [K,C,R,S], bias [K] or None -> [N,K,P,Q] float64."""
    x = _f64(x)
    filt = _f64(filt)
    if x.ndim != 4 or filt.ndim != 4 or x.shape[1] != filt.shape[1]:
        raise ValueError("expected x [N,C,H,W] and filt [K,C,R,S] with equal C")
    N, C, H, W = x.shape
    K, _, R, S = filt.shape
    P = conv_out_dim(H, R, stride, pad)
    Q = conv_out_dim(W, S, stride, pad)
    if P <= 0 or Q <= 0:
        raise ValueError("window does not fit the padded input")
    b = None
    if bias is not None:
        b = _f64(bias)
        if b.shape != (K,):
            raise ValueError("bias must have shape [K]")
    out = np.empty((N, K, P, Q), dtype=np.float64)
    rc = _load().oracle_conv_fwd_f64(_ptr(x), _ptr(filt), _ptr(b) if b is not None else None,
                                     _ptr(out), N, C, H, W, K, R, S, stride, pad, int(bool(relu)))
    if rc != 0:
        raise ValueError("oracle_conv_fwd_f64 rejected the shape")
    return out


def maxpool_fwd(x, ksz: int = 3, stride: int = 2) -> np.ndarray:
    """fp64 max-pool, no padding, floor extent.  x [N,C,H,W] -> [N,C,P,Q] float64."""
    x = _f64(x)
    N, C, H, W = x.shape
    P = conv_out_dim(H, ksz, stride, 0)
    Q = conv_out_dim(W, ksz, stride, 0)
    if P <= 0 or Q <= 0:
        raise ValueError("pool window does not fit")
    out = np.empty((N, C, P, Q), dtype=np.float64)
    rc = _load().oracle_maxpool_fwd_f64(_ptr(x), _ptr(out), N, C, H, W, ksz, stride)
    if rc != 0:
        raise ValueError("oracle_maxpool_fwd_f64 rejected the shape")
    return out


def conv_macs(N, C, H, W, K, R, S, stride, pad) -> int:
    return int(_load().oracle_conv_macs(N, C, H, W, K, R, S, stride, pad))


def conv_flops(N, C, H, W, K, R, S, stride, pad) -> int:
    """Two FLOPs per multiply-accumulate (the convention of the paper's SGEMM tables)."""
    return 2 * conv_macs(N, C, H, W, K, R, S, stride, pad)


def conv_min_bytes(N, C, H, W, K, R, S, stride, pad) -> int:
    return int(_load().oracle_conv_min_bytes(N, C, H, W, K, R, S, stride, pad))


def sgemm_ai(M: int, N: int, K: int) -> float:
    return float(_load().oracle_sgemm_ai(M, N, K))


def sgemm(A, Bm) -> np.ndarray:
    """C = A @ Bm by the definition (Section 4, Table 1): row-major [M][K] x [K][N], fp64 accumulation, k ascending."""
    a, b = _f64(A), _f64(Bm)
    if a.ndim != 2 or b.ndim != 2 or a.shape[1] != b.shape[0]:
        raise ValueError("sgemm: shapes do not chain")
    M, K = a.shape
    N = b.shape[1]
    c = np.empty((M, N), dtype=np.float64)
    rc = _load().oracle_sgemm_f64(_ptr(a), _ptr(b), _ptr(c), M, N, K)
    if rc != 0:
        raise ValueError("oracle_sgemm_f64: invalid arguments")
    return c


def softmax(x) -> np.ndarray:
    """Softmax over the last dimension of a 2-D array [rows][cols] by the definition (Section 2 names the operation), fp64."""
    a = _f64(x)
    if a.ndim != 2:
        raise ValueError("softmax: expected [rows][cols]")
    out = np.empty_like(a)
    rc = _load().oracle_softmax_f64(_ptr(a), _ptr(out), a.shape[0], a.shape[1])
    if rc != 0:
        raise ValueError("oracle_softmax_f64: invalid arguments")
    return out


def num_threads() -> int:
    """Host threads the OpenMP loops of the oracle will use."""
    return int(_load().oracle_num_threads())


def rel_l2(got, ref) -> float:
    """sqrt(sum (got-ref)^2) / sqrt(sum ref^2) in fp64; 0/0 counts as 0, x/0 as inf."""
    g = np.asarray(got, dtype=np.float64)
    r = np.asarray(ref, dtype=np.float64)
    num = float(np.sqrt(np.sum((g - r) ** 2)))
    den = float(np.sqrt(np.sum(r ** 2)))
    if den == 0.0:
        return 0.0 if num == 0.0 else float("inf")
    return num / den
