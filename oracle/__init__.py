"""ctypes front end of the CPU oracle (``q4k_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may import this
package.  It never imports the GPU package and the GPU package never imports it.

All arrays are numpy arrays in host memory.  Shapes follow the oracle's C interface:
activations are ``[n_tok, width]`` row-major, Q4_K tensors are ``uint8`` buffers of
``rows * (cols // 256) * 144`` bytes.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "q4k_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

BLOCK_BYTES = 144
SUPER_BLOCK = 256

# tensor ids (same numbering as the public header; retyped here on purpose)
ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, W_GATE, W_UP, W_DOWN, OUT_NORM, W_HEAD, TOK_EMBD = range(12)


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (portable x86-64 code, no fast-math, no FMA contraction)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread", "-ffp-contract=off",
                   "-Wall", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        u8p, f32p, f64p, i32p, u16p = (C.POINTER(t) for t in (C.c_uint8, C.c_float, C.c_double, C.c_int32, C.c_uint16))
        L.orc_half_to_double.restype = C.c_double
        L.orc_half_to_double.argtypes = [C.c_uint16]
        L.orc_double_to_half.restype = C.c_uint16
        L.orc_double_to_half.argtypes = [C.c_double]
        L.orc_q4k_fields.restype = None
        L.orc_q4k_fields.argtypes = [u8p, f64p, f64p, i32p, i32p]
        L.orc_q4k_pack.restype = None
        L.orc_q4k_pack.argtypes = [C.c_uint16, C.c_uint16, i32p, i32p, u8p, u8p]
        L.orc_q4k_dequant_f64.restype = None
        L.orc_q4k_dequant_f64.argtypes = [u8p, C.c_int64, f64p]
        L.orc_q4k_dequant_f32.restype = None
        L.orc_q4k_dequant_f32.argtypes = [u8p, C.c_int64, f32p]
        L.orc_gemv_q4k.restype = C.c_int
        L.orc_gemv_q4k.argtypes = [u8p, C.c_int64, C.c_int64, f32p, C.c_int, f64p, f64p, C.c_int]
        L.orc_rmsnorm.restype = None
        L.orc_rmsnorm.argtypes = [f64p, f32p, C.c_int64, C.c_double, f64p]
        L.orc_rope.restype = None
        L.orc_rope.argtypes = [f64p, C.c_int, C.c_int, C.c_int64, C.c_double, C.c_int]
        L.orc_attend.restype = None
        L.orc_attend.argtypes = [f64p, u16p, u16p, C.c_int64, C.c_int64, C.c_int, f64p]
        L.orc_silu.restype = C.c_double
        L.orc_silu.argtypes = [C.c_double]
        L.orc_ctx_create.restype = C.c_void_p
        L.orc_ctx_create.argtypes = [i32p, C.c_float, C.c_float, C.c_int]
        L.orc_ctx_destroy.restype = None
        L.orc_ctx_destroy.argtypes = [C.c_void_p]
        L.orc_load_tensor.restype = C.c_int
        L.orc_load_tensor.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_int]
        L.orc_kv_load.restype = C.c_int
        L.orc_kv_load.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, u16p, u16p]
        L.orc_kv_read.restype = C.c_int
        L.orc_kv_read.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, u16p, u16p]
        L.orc_forward_window.restype = C.c_int
        L.orc_forward_window.argtypes = [C.c_void_p, C.c_int, C.c_int, f32p, f32p, C.c_int, C.c_int, C.c_int]
        L.orc_logits.restype = C.c_int
        L.orc_logits.argtypes = [C.c_void_p, f32p, C.c_int, f32p, C.c_int]
        L.orc_embed.restype = C.c_int
        L.orc_embed.argtypes = [C.c_void_p, i32p, C.c_int, f32p]
        L.orc_argmax.restype = C.c_int
        L.orc_argmax.argtypes = [f32p, C.c_int64, f32p]
        _lib = L
    return _lib


def _p(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def default_threads() -> int:
    return max(1, len(os.sched_getaffinity(0)))


# ---------------------------------------------------------------------------------------------
# primitives
# ---------------------------------------------------------------------------------------------
def half_to_double(bits: int) -> float:
    return lib().orc_half_to_double(int(bits) & 0xFFFF)


def double_to_half(v: float) -> int:
    return int(lib().orc_double_to_half(float(v)))


def q4k_fields(block: np.ndarray):
    """(d, dmin, sc[8], m[8]) of one 144-byte super-block."""
    block = np.ascontiguousarray(block, dtype=np.uint8)
    assert block.size == BLOCK_BYTES
    d, dmin = C.c_double(), C.c_double()
    sc, m = np.zeros(8, np.int32), np.zeros(8, np.int32)
    lib().orc_q4k_fields(_p(block, C.c_uint8), C.byref(d), C.byref(dmin), _p(sc, C.c_int32), _p(m, C.c_int32))
    return d.value, dmin.value, sc, m


def q4k_pack(d_bits: int, dmin_bits: int, sc, m, q) -> np.ndarray:
    sc = np.ascontiguousarray(sc, dtype=np.int32)
    m = np.ascontiguousarray(m, dtype=np.int32)
    q = np.ascontiguousarray(q, dtype=np.uint8)
    assert sc.size == 8 and m.size == 8 and q.size == 256
    out = np.zeros(BLOCK_BYTES, np.uint8)
    lib().orc_q4k_pack(int(d_bits), int(dmin_bits), _p(sc, C.c_int32), _p(m, C.c_int32), _p(q, C.c_uint8), _p(out, C.c_uint8))
    return out


def q4k_dequant(blocks: np.ndarray, dtype=np.float64) -> np.ndarray:
    blocks = np.ascontiguousarray(blocks, dtype=np.uint8).reshape(-1)
    assert blocks.size % BLOCK_BYTES == 0
    n_sb = blocks.size // BLOCK_BYTES
    if dtype == np.float64:
        out = np.empty(n_sb * SUPER_BLOCK, np.float64)
        lib().orc_q4k_dequant_f64(_p(blocks, C.c_uint8), n_sb, _p(out, C.c_double))
    else:
        out = np.empty(n_sb * SUPER_BLOCK, np.float32)
        lib().orc_q4k_dequant_f32(_p(blocks, C.c_uint8), n_sb, _p(out, C.c_float))
    return out


def gemv_q4k(w: np.ndarray, rows: int, cols: int, x: np.ndarray, n_threads: int | None = None):
    """y[c, r] = sum_k W[r, k] x[c, k] in fp64; also returns sum_k |W[r,k] x[c,k]|."""
    w = np.ascontiguousarray(w, dtype=np.uint8).reshape(-1)
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1, cols)
    if cols % SUPER_BLOCK != 0 or w.size != rows * (cols // SUPER_BLOCK) * BLOCK_BYTES:
        raise ValueError("orc_gemv_q4k: cols must be a multiple of 256 and w must hold rows*(cols/256)*144 bytes")
    n_cols = x.shape[0]
    y = np.empty((n_cols, rows), np.float64)
    s = np.empty((n_cols, rows), np.float64)
    rc = lib().orc_gemv_q4k(_p(w, C.c_uint8), rows, cols, _p(x, C.c_float), n_cols, _p(y, C.c_double),
                            _p(s, C.c_double), n_threads or default_threads())
    if rc != 0:
        raise ValueError("orc_gemv_q4k: bad arguments")
    return y, s


def rmsnorm(h: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    h = np.ascontiguousarray(h, dtype=np.float64)
    g = np.ascontiguousarray(g, dtype=np.float32)
    out = np.empty_like(h)
    lib().orc_rmsnorm(_p(h, C.c_double), _p(g, C.c_float), h.size, float(eps), _p(out, C.c_double))
    return out


def rope(heads: np.ndarray, pos: int, theta: float, mode: int = 0) -> np.ndarray:
    """heads: [n_heads, D] fp64; returns the rotated copy."""
    out = np.array(heads, dtype=np.float64, order="C", copy=True)
    n_heads, D = out.shape
    lib().orc_rope(_p(out, C.c_double), n_heads, D, int(pos), float(theta), int(mode))
    return out


def attend(q: np.ndarray, k_bits: np.ndarray, v_bits: np.ndarray) -> np.ndarray:
    """One query (fp64, [D]) against [n_ctx, D] fp16 bit patterns of keys and values."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    n_ctx, D = k_bits.shape
    out = np.empty(D, np.float64)
    lib().orc_attend(_p(q, C.c_double), _p(k_bits, C.c_uint16), _p(v_bits, C.c_uint16), n_ctx, D, D, _p(out, C.c_double))
    return out


def silu(z: float) -> float:
    return lib().orc_silu(float(z))


def argmax(logits: np.ndarray):
    """(index of the largest logit, lowest index on ties; gap to the runner-up)."""
    logits = np.ascontiguousarray(logits, dtype=np.float32).reshape(-1)
    margin = C.c_float()
    idx = lib().orc_argmax(_p(logits, C.c_float), logits.size, C.byref(margin))
    return idx, margin.value


# ---------------------------------------------------------------------------------------------
# model
# ---------------------------------------------------------------------------------------------
class Model:
    """The oracle's model context.  ``cfg`` is a dict with the keys of the public config struct."""

    def __init__(self, cfg: dict, n_threads: int | None = None):
        self.cfg = dict(cfg)
        self.n_threads = n_threads or default_threads()
        ints = np.array([cfg["n_layers"], cfg["hidden"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"],
                         cfg["ffn"], cfg["vocab"], cfg["kv_capacity"], cfg.get("max_n_tok", 8)], np.int32)
        self._h = lib().orc_ctx_create(_p(ints, C.c_int32), float(cfg["rms_eps"]), float(cfg["rope_theta"]),
                                       int(cfg.get("rope_mode", 0)))
        self._keep = []

    def close(self):
        if self._h:
            lib().orc_ctx_destroy(self._h)
            self._h = None
            self._keep = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load(self, layer: int, tensor_id: int, data: np.ndarray, rows: int, cols: int, copy: bool = False):
        data = np.ascontiguousarray(data)
        if not copy:
            self._keep.append(data)
        rc = lib().orc_load_tensor(self._h, layer, tensor_id, data.ctypes.data_as(C.c_void_p), rows, cols,
                                   data.nbytes, 1 if copy else 0)
        if rc != 0:
            raise ValueError(f"orc_load_tensor({layer}, {tensor_id}) rejected its arguments")

    def kv_load(self, layer: int, pos_begin: int, k_bits: np.ndarray, v_bits: np.ndarray):
        k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
        v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
        n_pos = k_bits.shape[0]
        rc = lib().orc_kv_load(self._h, layer, pos_begin, n_pos, _p(k_bits, C.c_uint16), _p(v_bits, C.c_uint16))
        if rc != 0:
            raise ValueError("orc_kv_load rejected its arguments")

    def kv_read(self, layer: int, pos_begin: int, n_pos: int):
        shape = (n_pos, self.cfg["n_kv_heads"], self.cfg["head_dim"])
        k, v = np.empty(shape, np.uint16), np.empty(shape, np.uint16)
        rc = lib().orc_kv_read(self._h, layer, pos_begin, n_pos, _p(k, C.c_uint16), _p(v, C.c_uint16))
        if rc != 0:
            raise ValueError("orc_kv_read rejected its arguments")
        return k, v

    def forward_window(self, layer_begin: int, layer_end: int, hidden: np.ndarray, pos: int) -> np.ndarray:
        hidden = np.ascontiguousarray(hidden, dtype=np.float32).reshape(-1, self.cfg["hidden"])
        out = np.empty_like(hidden)
        rc = lib().orc_forward_window(self._h, layer_begin, layer_end, _p(hidden, C.c_float), _p(out, C.c_float),
                                      int(pos), hidden.shape[0], self.n_threads)
        if rc != 0:
            raise ValueError(f"orc_forward_window failed ({rc})")
        return out

    def logits(self, hidden: np.ndarray) -> np.ndarray:
        hidden = np.ascontiguousarray(hidden, dtype=np.float32).reshape(-1, self.cfg["hidden"])
        out = np.empty((hidden.shape[0], self.cfg["vocab"]), np.float32)
        rc = lib().orc_logits(self._h, _p(hidden, C.c_float), hidden.shape[0], _p(out, C.c_float), self.n_threads)
        if rc != 0:
            raise ValueError(f"orc_logits failed ({rc})")
        return out

    def embed(self, tokens) -> np.ndarray:
        tokens = np.ascontiguousarray(tokens, dtype=np.int32).reshape(-1)
        out = np.empty((tokens.size, self.cfg["hidden"]), np.float32)
        rc = lib().orc_embed(self._h, _p(tokens, C.c_int32), tokens.size, _p(out, C.c_float))
        if rc != 0:
            raise ValueError(f"orc_embed failed ({rc})")
        return out
