"""Pins for the CPU checker's Q6_K / Q8_0 / FP16 decoding and products.  Every expected value comes from somewhere
other than the checker: the hand-worked fixture, dense numpy built from fields that were chosen (not decoded),
one-bit toggles with the expected effect written out, and the gguf package's decoder where it is installed."""
import numpy as np
import pytest

import oracle.kquants as kq
from paper_2504_08791_b200 import synth
from tests.golden._read import kquants_blocks

FMT = {"q6_k": kq.Q6_K, "q8_0": kq.Q8_0}


@pytest.mark.parametrize("name", ["q8_0.A", "q8_0.B", "q6_k.A", "q6_k.B"])
def test_handbuilt_blocks(name):
    b = kquants_blocks()[name]
    got = kq.dequant(FMT[b["fmt"]], b["bytes"])
    got32 = kq.dequant(FMT[b["fmt"]], b["bytes"], np.float32)
    for k, v in b["w"].items():
        assert got[k] == v, (name, k, got[k], v)
        assert float(got32[k]) == v                      # exact in binary32 as well


def test_q8_0_every_payload_byte_is_one_weight_and_the_scale_applies_to_all():
    rng = np.random.default_rng(1)
    base = synth.build_q8_0_blocks([0x3C00], rng.integers(-128, 128, (1, 32)))[0]      # d = 1
    w0 = kq.dequant(kq.Q8_0, base)
    assert np.array_equal(w0, base[2:].view(np.int8).astype(np.float64))
    for k in range(32):
        for bit in range(8):
            t = base.copy()
            t[2 + k] ^= 1 << bit
            diff = kq.dequant(kq.Q8_0, t) - w0
            assert np.count_nonzero(diff) == 1 and abs(diff[k]) == (1 << bit)            # two's complement: bit 7 weighs -128
            assert (diff[k] < 0) == (bool(base[2 + k] >> bit & 1) != (bit == 7))
    t = base.copy()
    t[1] = 0x40                                                                           # d = 2
    assert np.array_equal(kq.dequant(kq.Q8_0, t), 2 * w0)


def test_q6k_every_payload_bit_moves_one_weight_and_every_scale_sixteen():
    rng = np.random.default_rng(2)
    v = rng.integers(0, 64, (1, 256))
    sc = rng.integers(-128, 128, (1, 16))
    sc[sc == 0] = 5
    base = synth.build_q6k_blocks([0x3C00], sc, v)[0]                                     # d = 1
    w0 = kq.dequant(kq.Q6_K, base)
    assert np.array_equal(w0, (np.repeat(sc[0], 16) * (v[0] - 32)).astype(np.float64))
    seen = set()
    for byte in range(192):
        for bit in range(8):
            t = base.copy()
            t[byte] ^= 1 << bit
            diff = kq.dequant(kq.Q6_K, t) - w0
            (idx,) = np.nonzero(diff)
            assert idx.size == 1
            k = int(idx[0])
            # which of the six bits of v_k this is: the low four live in the first 128 bytes, the high two in the next 64
            vbit = bit % 4 if byte < 128 else 4 + bit % 2
            assert abs(diff[k]) == abs(int(sc[0, k // 16])) * (1 << vbit)
            seen.add((k, vbit))
    assert len(seen) == 256 * 6                                                          # every bit of every value is reachable
    for i in range(16):
        t = base.copy()
        t[192 + i] ^= 1
        (idx,) = np.nonzero(kq.dequant(kq.Q6_K, t) - w0)
        assert set(idx) <= set(range(16 * i, 16 * i + 16)) and idx.size >= 14             # (v = 32 gives 0 either way)


@pytest.mark.parametrize("fmt,rows,cols,n_cols", [(kq.Q6_K, 9, 512, 2), (kq.Q8_0, 7, 96, 3), (kq.F16, 5, 40, 1), (kq.Q6_K, 1, 256, 1)])
def test_gemv_equals_dense_numpy_from_chosen_fields(fmt, rows, cols, n_cols):
    rng = np.random.default_rng(3)
    x = rng.normal(0, 1, (n_cols, cols)).astype(np.float32)
    if fmt == kq.Q6_K:
        n = rows * cols // 256
        v, sc = rng.integers(0, 64, (n, 256)), rng.integers(-128, 128, (n, 16))
        d = rng.normal(0, 0.01, n).astype(np.float16)
        w = synth.build_q6k_blocks(d.view(np.uint16), sc, v).reshape(-1)
        dense = (d.astype(np.float64)[:, None] * np.repeat(sc, 16, axis=1) * (v - 32)).reshape(rows, cols)
    elif fmt == kq.Q8_0:
        n = rows * cols // 32
        q = rng.integers(-128, 128, (n, 32))
        d = rng.normal(0, 0.01, n).astype(np.float16)
        w = synth.build_q8_0_blocks(d.view(np.uint16), q).reshape(-1)
        dense = (d.astype(np.float64)[:, None] * q).reshape(rows, cols)
    else:
        h = rng.normal(0, 1, (rows, cols)).astype(np.float16)
        w = h.view(np.uint8).reshape(-1)
        dense = h.astype(np.float64)
    assert np.array_equal(kq.dequant(fmt, w).reshape(rows, cols), dense)
    y, s = kq.gemv(fmt, w, rows, cols, x)
    want = x.astype(np.float64) @ dense.T
    np.testing.assert_allclose(y, want, rtol=0, atol=1e-12 * np.abs(want).max() + 1e-300)
    np.testing.assert_allclose(s, np.abs(x.astype(np.float64))[:, None, :].__mul__(np.abs(dense)[None]).sum(-1), rtol=1e-12)
    # rows and columns the right way round: a unit vector picks a column of W
    e = np.zeros((1, cols), np.float32)
    e[0, cols // 3] = 1.0
    assert np.array_equal(kq.gemv(fmt, w, rows, cols, e)[0][0], dense[:, cols // 3])
    assert np.array_equal(kq.gemv(fmt, w, rows, cols, x, n_threads=1)[0], kq.gemv(fmt, w, rows, cols, x, n_threads=3)[0])


@pytest.mark.parametrize("fmt,name", [(kq.Q6_K, "Q6_K"), (kq.Q8_0, "Q8_0")])
def test_decoding_agrees_with_the_gguf_package(fmt, name):
    gguf = pytest.importorskip("gguf")
    from gguf import quants
    rng = np.random.default_rng(4)
    n = 200
    blocks = rng.integers(0, 256, (n, kq.BLOCK_BYTES[fmt]), dtype=np.uint8)
    d_at = 209 if fmt == kq.Q6_K else 1
    blocks[:, d_at] &= 0xBF                                  # keep d finite
    want = quants.dequantize(blocks.reshape(-1), getattr(gguf.GGMLQuantizationType, name)).reshape(-1).astype(np.float64)
    got = kq.dequant(fmt, blocks)
    # the package rounds intermediate products to fp32; the exact value is representable, so at most a few ulps apart
    assert np.all(np.abs(want - got) <= 4 * 2.0 ** -24 * np.abs(got) + 1e-45)


def test_generators_give_roughly_unit_gain_rows():
    for fmt in (synth.FMT_Q6_K, synth.FMT_Q8_0, synth.FMT_F16):
        w = synth.fmt_tensor(5, fmt, 64, 1024)
        assert w.size == 64 * 1024 // synth.FMT_BLOCK_WEIGHTS[fmt] * synth.FMT_BLOCK_BYTES[fmt]
        dense = kq.dequant({synth.FMT_Q6_K: kq.Q6_K, synth.FMT_Q8_0: kq.Q8_0, synth.FMT_F16: kq.F16}[fmt], w).reshape(64, 1024)
        norms = np.sqrt((dense ** 2).sum(1))
        assert 0.6 < norms.mean() < 1.6 and abs(dense.mean()) < 0.01
