"""ctypes front end of ``kquants_oracle.cpp``: Q6_K, Q8_0 and FP16 matrices on the CPU, fp64.  TEST INFRASTRUCTURE ONLY
(tests, the smoke check and the benchmark's CPU legs); it never imports the GPU package."""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kquants_oracle.cpp")
_LIB = os.path.join(_HERE, "libkquants_oracle.so")
_lock = threading.Lock()
_lib = None

Q6_K, Q8_0, F16 = 1, 2, 3      # format ids of this checker (retyped on purpose, not imported from the product)
BLOCK_WEIGHTS = {Q6_K: 256, Q8_0: 32, F16: 1}
BLOCK_BYTES = {Q6_K: 210, Q8_0: 34, F16: 2}


def build(force: bool = False) -> str:
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.run(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-ffp-contract=off", "-Wall", "-o", tmp, _SRC],
                           check=True)
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, f32p, f64p = (C.POINTER(t) for t in (C.c_uint8, C.c_float, C.c_double))
        L.orc_fmt_dequant_f64.argtypes = [C.c_int, u8p, C.c_int64, f64p]
        L.orc_fmt_dequant_f32.argtypes = [C.c_int, u8p, C.c_int64, f32p]
        L.orc_fmt_gemv.argtypes = [C.c_int, u8p, C.c_int64, C.c_int64, f32p, C.c_int, f64p, f64p, C.c_int]
        for f in (L.orc_fmt_dequant_f64, L.orc_fmt_dequant_f32, L.orc_fmt_gemv, L.orc_fmt_block_weights, L.orc_fmt_block_bytes):
            f.restype = C.c_int
        _lib = L
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def dequant(fmt: int, blocks: np.ndarray, dtype=np.float64) -> np.ndarray:
    blocks = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1)
    assert blocks.size % BLOCK_BYTES[fmt] == 0
    n = blocks.size // BLOCK_BYTES[fmt]
    if dtype == np.float64:
        out = np.empty(n * BLOCK_WEIGHTS[fmt], np.float64)
        rc = lib().orc_fmt_dequant_f64(fmt, _p(blocks, C.c_uint8), n, _p(out, C.c_double))
    else:
        out = np.empty(n * BLOCK_WEIGHTS[fmt], np.float32)
        rc = lib().orc_fmt_dequant_f32(fmt, _p(blocks, C.c_uint8), n, _p(out, C.c_float))
    if rc != 0:
        raise ValueError("unknown format")
    return out


def gemv(fmt: int, w: np.ndarray, rows: int, cols: int, x: np.ndarray, n_threads: int | None = None):
    """y[c, r] = sum_k W[r, k] x[c, k] in fp64, and sum_k |W[r, k] x[c, k]|."""
    w = np.ascontiguousarray(w, dtype=np.uint8).reshape(-1)
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1, cols)
    if cols % BLOCK_WEIGHTS[fmt] != 0 or w.size != rows * (cols // BLOCK_WEIGHTS[fmt]) * BLOCK_BYTES[fmt]:
        raise ValueError("cols must be a multiple of the block's weights and w must hold rows * cols / block weights blocks")
    n_cols = x.shape[0]
    y = np.empty((n_cols, rows), np.float64)
    s = np.empty((n_cols, rows), np.float64)
    rc = lib().orc_fmt_gemv(fmt, _p(w, C.c_uint8), rows, cols, _p(x, C.c_float), n_cols, _p(y, C.c_double), _p(s, C.c_double),
                            n_threads or max(1, len(os.sched_getaffinity(0))))
    if rc != 0:
        raise ValueError("orc_fmt_gemv: bad arguments")
    return y, s
