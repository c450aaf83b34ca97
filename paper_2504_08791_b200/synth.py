"""Seeded synthetic inputs: Q4_K tensors, norm gains, activations, KV prefill, model shapes.

This module only *produces bytes and numbers*.  It contains none of the forward pass: no
dequantisation, no dot product, no normalisation.  Both the GPU tests/benchmark and the CPU
checker are fed from here, so that the two sides always see the same inputs while sharing no
arithmetic.  numpy only; it imports neither the GPU binding nor the checker.

Two weight distributions are provided.

* ``gemv_case``: the literal single-GEMV distribution -- nibbles uniform 0..15, every 6-bit scale
  and min uniform 0..63, d and dmin = |N(0, sigma=0.01)| rounded to fp16, x ~ N(0, 1) fp32.
* ``model_tensor``: a zero-mean "random-init" distribution for whole models.  Per super-block:
  nibbles uniform; sc_j uniform in 32..63 for even-numbered blocks and 0..63 for odd ones (so both
  halves of the split 6-bit fields are exercised); m_j = round(7.5*sc_j/8) and dmin = 8*d, which
  centres each sub-block on zero; d = fp16(sigma * (0.5+u) / (4.61 * 39.5)) with u uniform [0,1)
  and sigma = gain / sqrt(cols), so a row has roughly unit-gain.  (4.61 is the standard deviation
  of a uniform nibble, 39.5 the mean scale.)  The literal distribution is not used for models
  because its weights have mean +1.6 and drive 80-layer activations far outside fp32 resolution of
  the logit tolerance.

Random streams: one SFC64 generator per (seed, tensor key, row chunk), so a tensor can be produced
in parallel and in pieces, always with the same bytes.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

BLOCK_BYTES = 144
SUPER_BLOCK = 256

# tensor ids of the public header
ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, W_GATE, W_UP, W_DOWN, OUT_NORM, W_HEAD, TOK_EMBD = range(12)
LAYER_TENSORS = (ATTN_NORM, WQ, WK, WV, WO, FFN_NORM, W_GATE, W_UP, W_DOWN)
GLOBAL_TENSORS = (OUT_NORM, W_HEAD, TOK_EMBD)

_CHUNK_BLOCKS = 1 << 16  # super-blocks per generation chunk (9.4 MB)


def _rng(seed: int, *key: int) -> np.random.Generator:
    return np.random.Generator(np.random.SFC64([int(seed) & 0xFFFFFFFF] + [int(k) & 0xFFFFFFFF for k in key]))


def _threads() -> int:
    return max(1, min(32, len(os.sched_getaffinity(0))))


def _random_bytes(rng: np.random.Generator, n: int) -> np.ndarray:
    words = rng.integers(0, 2**64, (n + 7) // 8, dtype=np.uint64, endpoint=False)
    return words.view(np.uint8)[:n]


def pack_scales(sc: np.ndarray, m: np.ndarray) -> np.ndarray:
    """[n, 8] scales and [n, 8] mins (values 0..63) -> [n, 12] packed bytes of the block header."""
    sc = sc.astype(np.uint8)
    m = m.astype(np.uint8)
    out = np.empty((sc.shape[0], 12), np.uint8)
    out[:, 0:4] = (sc[:, 0:4] & 63) | ((sc[:, 4:8] >> 4) << 6)
    out[:, 4:8] = (m[:, 0:4] & 63) | ((m[:, 4:8] >> 4) << 6)
    out[:, 8:12] = (sc[:, 4:8] & 15) | ((m[:, 4:8] & 15) << 4)
    return out


def pack_nibbles(q: np.ndarray) -> np.ndarray:
    """[n, 256] values 0..15 -> [n, 128] bytes: byte 32p+i = q[64p+i] | q[64p+32+i] << 4."""
    q = q.astype(np.uint8).reshape(-1, 4, 2, 32)
    return (q[:, :, 0, :] | (q[:, :, 1, :] << 4)).reshape(-1, 128)


def build_blocks(d_bits, dmin_bits, sc, m, q) -> np.ndarray:
    """Assemble super-blocks from explicit fields (used for hand-made test cases)."""
    d_bits = np.asarray(d_bits, dtype=np.uint16).reshape(-1)
    dmin_bits = np.asarray(dmin_bits, dtype=np.uint16).reshape(-1)
    n = d_bits.size
    out = np.empty((n, BLOCK_BYTES), np.uint8)
    out[:, 0:2] = d_bits.view(np.uint8).reshape(n, 2)
    out[:, 2:4] = dmin_bits.view(np.uint8).reshape(n, 2)
    out[:, 4:16] = pack_scales(np.asarray(sc).reshape(n, 8), np.asarray(m).reshape(n, 8))
    out[:, 16:] = pack_nibbles(np.asarray(q).reshape(n, 256))
    return out


# ---------------------------------------------------------------------------------------------
# the other block formats: Q8_0 (34 bytes per 32 weights), Q6_K (210 bytes per 256 weights), FP16
# ---------------------------------------------------------------------------------------------
FMT_Q4_K, FMT_Q6_K, FMT_Q8_0, FMT_F16 = 0, 1, 2, 3
FMT_BLOCK_WEIGHTS = {FMT_Q4_K: 256, FMT_Q6_K: 256, FMT_Q8_0: 32, FMT_F16: 1}
FMT_BLOCK_BYTES = {FMT_Q4_K: 144, FMT_Q6_K: 210, FMT_Q8_0: 34, FMT_F16: 2}


def build_q8_0_blocks(d_bits, q) -> np.ndarray:
    """[n] binary16 bit patterns and [n, 32] signed values -128..127 -> [n, 34] bytes."""
    d_bits = np.asarray(d_bits, dtype=np.uint16).reshape(-1)
    n = d_bits.size
    out = np.empty((n, 34), np.uint8)
    out[:, 0:2] = d_bits.view(np.uint8).reshape(n, 2)
    out[:, 2:] = np.asarray(q).reshape(n, 32).astype(np.int8).view(np.uint8)
    return out


def build_q6k_blocks(d_bits, scales, v) -> np.ndarray:
    """[n] binary16 bit patterns, [n, 16] signed scales and [n, 256] six-bit values 0..63 -> [n, 210] bytes.
    Weight k = 128 h + 32 i + l keeps its low nibble in byte 64 h + 32 (i & 1) + l of the first 128 bytes (low half
    of the byte for i < 2, high half otherwise) and its two high bits in bits 2i, 2i+1 of byte 128 + 32 h + l."""
    d_bits = np.asarray(d_bits, dtype=np.uint16).reshape(-1)
    n = d_bits.size
    v = np.asarray(v).reshape(n, 2, 4, 32).astype(np.uint8)
    out = np.zeros((n, 210), np.uint8)
    lo, hi = v & 15, v >> 4
    for h in range(2):
        for i in range(4):
            seg = out[:, 64 * h + 32 * (i & 1):64 * h + 32 * (i & 1) + 32]
            seg |= lo[:, h, i] << (0 if i < 2 else 4)
            out[:, 128 + 32 * h:128 + 32 * h + 32] |= hi[:, h, i] << (2 * i)
    out[:, 192:208] = np.asarray(scales).reshape(n, 16).astype(np.int8).view(np.uint8)
    out[:, 208:210] = d_bits.view(np.uint8).reshape(n, 2)
    return out


def fmt_tensor(seed: int, fmt: int, rows: int, cols: int, gain: float = 1.0) -> np.ndarray:
    """Random-init matrix in one of the other formats, roughly unit gain per row (weights ~ N(0, gain^2 / cols))."""
    rng = _rng(seed, 606, fmt, rows, cols)
    sigma = gain / np.sqrt(cols)
    if fmt == FMT_F16:
        return rng.normal(0.0, sigma, (rows, cols)).astype(np.float16).view(np.uint8).reshape(-1)
    n = rows * cols // FMT_BLOCK_WEIGHTS[fmt]
    blocks = _random_bytes(rng, n * FMT_BLOCK_BYTES[fmt]).reshape(n, FMT_BLOCK_BYTES[fmt]).copy()
    if fmt == FMT_Q8_0:
        d = (sigma * (0.5 + rng.random(n)) / 73.9).astype(np.float16)          # uniform signed bytes have sigma 73.9
        blocks[:, 0:2] = d.view(np.uint8).reshape(n, 2)
    else:
        d = (sigma * (0.5 + rng.random(n)) / (18.5 * 73.9)).astype(np.float16)   # uniform 6-bit values: sigma 18.5
        blocks[:, 208:210] = d.view(np.uint8).reshape(n, 2)
    return blocks.reshape(-1)


# ---------------------------------------------------------------------------------------------
# the literal single-GEMV distribution
# ---------------------------------------------------------------------------------------------
def gemv_weights(seed: int, rows: int, cols: int) -> np.ndarray:
    assert cols % SUPER_BLOCK == 0
    n_sb = rows * (cols // SUPER_BLOCK)
    rng = _rng(seed, 101)
    blocks = _random_bytes(rng, n_sb * BLOCK_BYTES).reshape(n_sb, BLOCK_BYTES).copy()
    dd = np.abs(rng.normal(0.0, 0.01, (n_sb, 2))).astype(np.float16)
    blocks[:, 0:4] = dd.view(np.uint8).reshape(n_sb, 4)
    return blocks.reshape(-1)


def activations(seed: int, n_tok: int, width: int, scale: float = 1.0) -> np.ndarray:
    return (_rng(seed, 202, n_tok, width).normal(0.0, 1.0, (n_tok, width)) * scale).astype(np.float32)


def gemv_case(seed: int = 0, rows: int = 4096, cols: int = 4096, n_cols: int = 1):
    """(w bytes, x[n_cols, cols] fp32) of the single-GEMV workload."""
    return gemv_weights(seed, rows, cols), activations(seed, n_cols, cols)


# ---------------------------------------------------------------------------------------------
# zero-mean model tensors
# ---------------------------------------------------------------------------------------------
def _model_chunk(seed: int, key: tuple, chunk: int, n_blocks: int, first_block: int, sigma: float) -> np.ndarray:
    rng = _rng(seed, 303, *key, chunk)
    blocks = _random_bytes(rng, n_blocks * BLOCK_BYTES).reshape(n_blocks, BLOCK_BYTES).copy()
    sc = rng.integers(0, 64, (n_blocks, 8), dtype=np.uint8)
    even = ((first_block + np.arange(n_blocks)) % 2) == 0
    sc[even] |= 32
    m = np.floor(7.5 * sc.astype(np.float64) / 8.0 + 0.5).astype(np.uint8)
    u = rng.random(n_blocks)
    d = (sigma * (0.5 + u) / (4.61 * 39.5)).astype(np.float16)
    dmin = (d.astype(np.float32) * 8.0).astype(np.float16)
    blocks[:, 0:2] = d.view(np.uint8).reshape(n_blocks, 2)
    blocks[:, 2:4] = dmin.view(np.uint8).reshape(n_blocks, 2)
    blocks[:, 4:16] = pack_scales(sc, m)
    return blocks


def model_tensor(seed: int, layer: int, tensor_id: int, rows: int, cols: int, gain: float = 1.0,
                 out: np.ndarray | None = None) -> np.ndarray:
    """Q4_K bytes of one weight matrix, rows*(cols/256)*144 of them."""
    assert cols % SUPER_BLOCK == 0
    n_sb = rows * (cols // SUPER_BLOCK)
    sigma = gain / np.sqrt(cols)
    if out is None:
        out = np.empty(n_sb * BLOCK_BYTES, np.uint8)
    view = out.reshape(n_sb, BLOCK_BYTES)
    jobs = [(c, min(_CHUNK_BLOCKS, n_sb - c * _CHUNK_BLOCKS)) for c in range((n_sb + _CHUNK_BLOCKS - 1) // _CHUNK_BLOCKS)]

    def run(job):
        c, n = job
        view[c * _CHUNK_BLOCKS:c * _CHUNK_BLOCKS + n] = _model_chunk(seed, (layer + 1, tensor_id), c, n, c * _CHUNK_BLOCKS, sigma)

    if len(jobs) > 1 and _threads() > 1:
        with ThreadPoolExecutor(_threads()) as ex:
            list(ex.map(run, jobs))
    else:
        for j in jobs:
            run(j)
    return out


def norm_gain(seed: int, layer: int, tensor_id: int, width: int) -> np.ndarray:
    return (1.0 + 0.1 * _rng(seed, 404, layer + 1, tensor_id).normal(0.0, 1.0, width)).astype(np.float32)


def kv_prefill(seed: int, layer: int, n_pos: int, n_kv_heads: int, head_dim: int):
    """fp16 N(0,1) keys and values as uint16 bit patterns, [n_pos, n_kv_heads, head_dim] each."""
    rng = _rng(seed, 505, layer + 1)
    k = rng.normal(0.0, 1.0, (n_pos, n_kv_heads, head_dim)).astype(np.float16).view(np.uint16)
    v = rng.normal(0.0, 1.0, (n_pos, n_kv_heads, head_dim)).astype(np.float16).view(np.uint16)
    return k, v


# ---------------------------------------------------------------------------------------------
# model shapes
# ---------------------------------------------------------------------------------------------
def model_config(name: str, **over) -> dict:
    """Shapes of the workloads: 'tiny' (tests), '8b' (Llama-3-8B), '32b' (Qwen2.5-32B), '70b' (Llama-3-70B)."""
    shapes = {
        "tiny": dict(n_layers=3, hidden=512, n_q_heads=4, n_kv_heads=2, head_dim=128, ffn=1024, vocab=768,
                     kv_capacity=96, rms_eps=1e-5, rope_theta=1e4),
        "small": dict(n_layers=4, hidden=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=2816, vocab=2048,
                      kv_capacity=320, rms_eps=1e-5, rope_theta=5e5),
        "8b": dict(n_layers=32, hidden=4096, n_q_heads=32, n_kv_heads=8, head_dim=128, ffn=14336, vocab=128256,
                   kv_capacity=1024 + 64, rms_eps=1e-5, rope_theta=5e5),
        "32b": dict(n_layers=64, hidden=5120, n_q_heads=40, n_kv_heads=8, head_dim=128, ffn=27648, vocab=152064,
                    kv_capacity=4096 + 64, rms_eps=1e-6, rope_theta=1e6),
        "70b": dict(n_layers=80, hidden=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, ffn=28672, vocab=128256,
                    kv_capacity=4096 + 64, rms_eps=1e-5, rope_theta=5e5),
    }
    cfg = dict(shapes[name])
    cfg.update(max_n_tok=8, rope_mode=0)
    cfg.update(over)
    return cfg


def tensor_shape(cfg: dict, tensor_id: int):
    e, H, G, D, F, V = cfg["hidden"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"], cfg["ffn"], cfg["vocab"]
    return {
        ATTN_NORM: (1, e), FFN_NORM: (1, e), OUT_NORM: (1, e),
        WQ: (H * D, e), WK: (G * D, e), WV: (G * D, e), WO: (e, H * D),
        W_GATE: (F, e), W_UP: (F, e), W_DOWN: (e, F), W_HEAD: (V, e), TOK_EMBD: (V, e),
    }[tensor_id]


def tensor_gain(tensor_id: int) -> float:
    # head scaled x8 so that greedy decoding has clear winners; embedding rows have unit RMS
    return {W_HEAD: 8.0}.get(tensor_id, 1.0)


def make_tensor(seed: int, cfg: dict, layer: int, tensor_id: int) -> np.ndarray:
    rows, cols = tensor_shape(cfg, tensor_id)
    if tensor_id in (ATTN_NORM, FFN_NORM, OUT_NORM):
        return norm_gain(seed, layer, tensor_id, cols)
    gain = tensor_gain(tensor_id)
    if tensor_id == TOK_EMBD:
        gain = float(np.sqrt(cols))
    return model_tensor(seed, layer, tensor_id, rows, cols, gain)


def iter_model_tensors(seed: int, cfg: dict, layers=None, with_globals: bool = True):
    """Yield (layer, tensor_id, rows, cols, data) for every tensor of the model, layer by layer."""
    for layer in (range(cfg["n_layers"]) if layers is None else layers):
        for tid in LAYER_TENSORS:
            rows, cols = tensor_shape(cfg, tid)
            yield layer, tid, rows, cols, make_tensor(seed, cfg, layer, tid)
    if with_globals:
        for tid in GLOBAL_TENSORS:
            rows, cols = tensor_shape(cfg, tid)
            yield -1, tid, rows, cols, make_tensor(seed, cfg, -1, tid)


def weight_bytes(cfg: dict, tensor_ids) -> int:
    total = 0
    for tid in tensor_ids:
        rows, cols = tensor_shape(cfg, tid)
        if tid not in (ATTN_NORM, FFN_NORM, OUT_NORM):
            total += rows * (cols // SUPER_BLOCK) * BLOCK_BYTES
    return total
