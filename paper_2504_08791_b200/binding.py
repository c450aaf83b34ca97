"""Thin ctypes binding of ``libprima.so`` (argument marshalling only; every step runs in the library).

Function names mirror ``include/prima.h``.  Device buffers are torch CUDA tensors (torch is used
for device memory and streams only); host buffers are numpy arrays.  Loading fails loudly when
the library has not been built: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# PRIMA_LIB=bounds selects the range-checked build of the same sources (tests)
LIB_PATH = os.path.join(_HERE, "libprima_bounds.so" if os.environ.get("PRIMA_LIB") == "bounds" else "libprima.so")

OK, ERR_ARG, ERR_STATE, ERR_CUDA, ERR_NOMEM, ERR_DEVICE = 0, -1, -2, -3, -4, -5
ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, W_GATE, W_UP, W_DOWN, OUT_NORM, W_HEAD, TOK_EMBD = range(12)
MAX_N_TOK = 8      # tokens of one sequence per step
MAX_N_SEQ = 16     # requests per step / columns of a product
PROF_GEMV, PROF_ATTENTION = 0, 1
PROF_GEMV_QKV, PROF_GEMV_O, PROF_GEMV_GATE_UP, PROF_GEMV_DOWN, PROF_GEMV_HEAD = 16, 17, 18, 19, 20
OPT_FIRST_WAIT_POLLS = 1
OPT_FAIL_AFTER_LAUNCHES = 2
OPT_RESIDENT_LAYERS = 3
OPT_STREAM_SLOTS = 4
OPT_L2_AHEAD_BYTES = 5
OPT_L2_AHEAD_O_BYTES = 6

EXPORTS = [
    "prima_ctx_create", "prima_ctx_destroy", "prima_load_q4k_weights", "prima_forward_window", "prima_logits",
    "prima_embed", "prima_argmax", "prima_kv_load", "prima_kv_read", "prima_sync", "prima_last_error",
    "prima_launch_count", "prima_profile_enable", "prima_profile_read", "prima_dequant_q4k", "prima_gemv_q4k", "prima_gemv_plan_create", "prima_gemv_plan_run",
    "prima_gemv_plan_destroy", "prima_gemv_q4k_noalloc", "prima_gemv_q4k_noalloc_error",
    "prima_forward_window_seqs", "prima_kv_load_seq", "prima_kv_read_seq", "prima_ctx_set_option", "prima_stream_stats",
    "prima_fmt_block_weights", "prima_fmt_block_bytes", "prima_dequant_fmt", "prima_gemv_fmt", "prima_fmt_last_error",
]


class ModelConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab",
                                         "kv_capacity", "max_n_tok")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float), ("rope_mode", C.c_int32), ("device", C.c_int32)]


class PrimaError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"prima error {code}: {msg}")
        self.code = code


_lib = None


def lib():
    """Load the C-ABI library; raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2504_08791_b200.build` (`--bounds` for the range-checked one) "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i64, i32 = C.c_void_p, C.c_int64, C.c_int
        L.prima_ctx_create.argtypes = [C.POINTER(ModelConfig), vp, C.POINTER(vp)]
        L.prima_ctx_destroy.argtypes = [vp]
        L.prima_load_q4k_weights.argtypes = [vp, i32, i32, vp, i64, i64, i64]
        L.prima_forward_window.argtypes = [vp, i32, i32, vp, vp, i32, i32]
        L.prima_logits.argtypes = [vp, vp, i32, vp]
        L.prima_embed.argtypes = [vp, vp, i32, vp]
        L.prima_argmax.argtypes = [vp, vp, i32, vp]
        L.prima_kv_load.argtypes = [vp, i32, i32, i32, vp, vp]
        L.prima_kv_read.argtypes = [vp, i32, i32, i32, vp, vp]
        L.prima_forward_window_seqs.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32]
        L.prima_kv_load_seq.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.prima_kv_read_seq.argtypes = [vp, i32, i32, i32, i32, vp, vp]
        L.prima_sync.argtypes = [vp]
        L.prima_ctx_set_option.argtypes = [vp, i32, i64]
        L.prima_stream_stats.argtypes = [vp, C.POINTER(i64), C.POINTER(C.c_double)]
        L.prima_last_error.argtypes = [vp]
        L.prima_last_error.restype = C.c_char_p
        L.prima_launch_count.argtypes = [vp]
        L.prima_launch_count.restype = i64
        L.prima_profile_enable.argtypes = [vp, i32]
        L.prima_profile_read.argtypes = [vp, i32, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(i64)]
        L.prima_dequant_q4k.argtypes = [vp, i64, vp, vp]
        L.prima_gemv_q4k.argtypes = [vp, i64, i64, vp, i32, vp, vp]
        L.prima_gemv_plan_create.argtypes = [vp, i64, i64, i32, C.POINTER(vp)]
        L.prima_gemv_plan_run.argtypes = [vp, vp, i32, vp, vp]
        L.prima_gemv_plan_destroy.argtypes = [vp]
        L.prima_fmt_block_weights.argtypes = [i32]
        L.prima_fmt_block_bytes.argtypes = [i32]
        L.prima_dequant_fmt.argtypes = [i32, vp, i64, vp, vp]
        L.prima_gemv_fmt.argtypes = [i32, vp, i64, i64, vp, i32, vp, vp]
        L.prima_fmt_last_error.argtypes = []
        L.prima_fmt_last_error.restype = C.c_char_p
        L.prima_gemv_q4k_noalloc.argtypes = [vp, i64, i64, vp, i32, vp, vp]
        L.prima_gemv_q4k_noalloc_error.argtypes = []
        L.prima_gemv_q4k_noalloc_error.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("prima_last_error", "prima_launch_count", "prima_gemv_q4k_noalloc_error", "prima_fmt_last_error"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def _check(rc: int, ctx=None):
    if rc != OK:
        msg = lib().prima_last_error(ctx)
        raise PrimaError(rc, msg.decode() if msg else "")


def _dev_ptr(t):
    """Raw device pointer of a contiguous torch CUDA tensor."""
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def _stream_ptr(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _host_ptr(a: np.ndarray):
    return C.c_void_p(a.ctypes.data)


# -------------------------------------------------------------------------------------------------
def prima_dequant_q4k(dev_blocks, n_superblocks: int, dev_out, stream=None):
    _check(lib().prima_dequant_q4k(_dev_ptr(dev_blocks), n_superblocks, _dev_ptr(dev_out), _stream_ptr(stream)))


def prima_gemv_q4k(dev_w, rows: int, cols: int, dev_x, n_cols: int, dev_y, stream=None):
    _check(lib().prima_gemv_q4k(_dev_ptr(dev_w), rows, cols, _dev_ptr(dev_x), n_cols, _dev_ptr(dev_y), _stream_ptr(stream)))


FMT_Q4_K, FMT_Q6_K, FMT_Q8_0, FMT_F16 = 0, 1, 2, 3


def _check_fmt(rc: int):
    if rc != OK:
        msg = lib().prima_fmt_last_error() or lib().prima_last_error(None)
        raise PrimaError(rc, msg.decode() if msg else "")


def prima_dequant_fmt(fmt: int, dev_blocks, n_blocks: int, dev_out, stream=None):
    _check_fmt(lib().prima_dequant_fmt(fmt, _dev_ptr(dev_blocks), n_blocks, _dev_ptr(dev_out), _stream_ptr(stream)))


def prima_gemv_fmt(fmt: int, dev_w, rows: int, cols: int, dev_x, n_cols: int, dev_y, stream=None):
    _check_fmt(lib().prima_gemv_fmt(fmt, _dev_ptr(dev_w), rows, cols, _dev_ptr(dev_x), n_cols, _dev_ptr(dev_y), _stream_ptr(stream)))


def prima_gemv_q4k_noalloc(dev_w, rows: int, cols: int, dev_x, n_cols: int, dev_y, stream=None):
    """Matrix-vector product that allocates nothing (for callers that own all device memory themselves).

    Same arguments as ``prima_gemv_q4k``; limited to rows*(cols/256)*n_cols <= 4,194,304; queues its
    kernels on the stream and returns without waiting.  Calls on one device must not overlap."""
    rc = lib().prima_gemv_q4k_noalloc(_dev_ptr(dev_w), rows, cols, _dev_ptr(dev_x), n_cols, _dev_ptr(dev_y), _stream_ptr(stream))
    if rc != OK:
        raise PrimaError(rc, lib().prima_gemv_q4k_noalloc_error().decode())


class GemvPlan:
    """prima_gemv_plan_create / _run / _destroy."""

    def __init__(self, dev_w, rows: int, cols: int, max_n_cols: int = 1):
        self._h = C.c_void_p()
        self.rows, self.cols = rows, cols
        _check(lib().prima_gemv_plan_create(_dev_ptr(dev_w), rows, cols, max_n_cols, C.byref(self._h)))

    def run(self, dev_x, n_cols: int, dev_y, stream=None):
        _check(lib().prima_gemv_plan_run(self._h, _dev_ptr(dev_x), n_cols, _dev_ptr(dev_y), _stream_ptr(stream)))

    def close(self):
        if self._h:
            lib().prima_gemv_plan_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Context:
    """prima_ctx_* : one model (or one window's worth of layers) resident on one GPU."""

    def __init__(self, cfg: dict, device: int = 0, stream=None):
        self.cfg = dict(cfg)
        mc = ModelConfig(cfg["n_layers"], cfg["hidden"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["ffn"],
                         cfg["vocab"], cfg["kv_capacity"], cfg.get("max_n_tok", MAX_N_TOK), cfg["rms_eps"], cfg["rope_theta"],
                         cfg.get("rope_mode", 0), device)
        self._h = C.c_void_p()
        self._stream = stream
        _check(lib().prima_ctx_create(C.byref(mc), _stream_ptr(stream), C.byref(self._h)))

    def close(self):
        if self._h:
            lib().prima_ctx_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def load(self, layer: int, tensor_id: int, data, rows: int, cols: int):
        """prima_load_q4k_weights; ``data`` is a numpy array (host) or a torch CUDA tensor."""
        if isinstance(data, np.ndarray):
            data = np.ascontiguousarray(data)
            ptr, nbytes = _host_ptr(data), data.nbytes
        else:
            ptr, nbytes = _dev_ptr(data), data.numel() * data.element_size()
        _check(lib().prima_load_q4k_weights(self._h, layer, tensor_id, ptr, rows, cols, nbytes), self._h)

    def forward_window(self, layer_begin: int, layer_end: int, hidden_in, hidden_out, pos: int, n_tok: int):
        _check(lib().prima_forward_window(self._h, layer_begin, layer_end, _dev_ptr(hidden_in), _dev_ptr(hidden_out), pos, n_tok),
               self._h)

    def logits(self, hidden, n_tok: int, logits_out):
        _check(lib().prima_logits(self._h, _dev_ptr(hidden), n_tok, _dev_ptr(logits_out)), self._h)

    def embed(self, tokens, hidden_out):
        tokens = np.ascontiguousarray(tokens, dtype=np.int32).reshape(-1)
        _check(lib().prima_embed(self._h, _host_ptr(tokens), tokens.size, _dev_ptr(hidden_out)), self._h)

    def argmax(self, logits, n_tok: int) -> np.ndarray:
        out = np.zeros(n_tok, np.int32)
        _check(lib().prima_argmax(self._h, _dev_ptr(logits), n_tok, _host_ptr(out)), self._h)
        return out

    def kv_load(self, layer: int, pos_begin: int, k_bits: np.ndarray, v_bits: np.ndarray, seq: int = 0):
        k_bits = np.ascontiguousarray(k_bits, dtype=np.uint16)
        v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
        _check(lib().prima_kv_load_seq(self._h, seq, layer, pos_begin, k_bits.shape[0], _host_ptr(k_bits), _host_ptr(v_bits)), self._h)

    def kv_read(self, layer: int, pos_begin: int, n_pos: int, seq: int = 0):
        shape = (n_pos, self.cfg["n_kv_heads"], self.cfg["head_dim"])
        k, v = np.empty(shape, np.uint16), np.empty(shape, np.uint16)
        _check(lib().prima_kv_read_seq(self._h, seq, layer, pos_begin, n_pos, _host_ptr(k), _host_ptr(v)), self._h)
        return k, v

    def forward_window_seqs(self, layer_begin: int, layer_end: int, hidden_in, hidden_out, seqs, positions):
        """prima_forward_window_seqs: one token of each of several independent requests."""
        seqs = np.ascontiguousarray(seqs, dtype=np.int32).reshape(-1)
        positions = np.ascontiguousarray(positions, dtype=np.int32).reshape(-1)
        if seqs.size != positions.size:
            raise ValueError("one position per sequence")
        _check(lib().prima_forward_window_seqs(self._h, layer_begin, layer_end, _dev_ptr(hidden_in), _dev_ptr(hidden_out),
                                               _host_ptr(seqs), _host_ptr(positions), seqs.size), self._h)

    def sync(self):
        _check(lib().prima_sync(self._h), self._h)

    def set_option(self, option: int, value: int):
        _check(lib().prima_ctx_set_option(self._h, option, value), self._h)

    def stream_stats(self):
        """(bytes copied host-to-device for streamed layers, summed copy time in ms)."""
        b, ms = C.c_int64(), C.c_double()
        _check(lib().prima_stream_stats(self._h, C.byref(b), C.byref(ms)), self._h)
        return b.value, ms.value

    def profile_enable(self, mode):
        """0 / False: off; 1 / True: events around every launch (isolated kernels); 2: in-situ stamps."""
        _check(lib().prima_profile_enable(self._h, int(mode)), self._h)

    def profile_read(self, klass: int):
        """(milliseconds, launches, algorithmic bytes) recorded for one kernel class."""
        ms, n, b = C.c_double(), C.c_int64(), C.c_int64()
        _check(lib().prima_profile_read(self._h, klass, C.byref(ms), C.byref(n), C.byref(b)), self._h)
        return ms.value, n.value, b.value

    def launch_count(self) -> int:
        return int(lib().prima_launch_count(self._h))

    def last_error(self) -> str:
        return lib().prima_last_error(self._h).decode()
