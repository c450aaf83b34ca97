"""Pins for the CPU checker's Q4_K decoding, fp16 conversion and GEMV.

Every expected value here comes from somewhere other than the checker: hand-worked fixtures,
numpy's own float16, dense numpy products built from fields that were chosen (not decoded), or
closed forms.
"""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth
from tests.golden._read import handbuilt_blocks


# ------------------------------------------------------------------------------------------- fp16
def test_half_to_double_all_patterns_match_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.half_to_double(int(b)) for b in bits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    # signed zeros keep their sign
    assert np.signbit(oracle.half_to_double(0x8000)) and not np.signbit(oracle.half_to_double(0x0000))


def test_double_to_half_round_trip_and_ties():
    bits = np.arange(65536, dtype=np.uint16)
    vals = bits.view(np.float16).astype(np.float64)
    finite = np.isfinite(vals)
    for b in bits[finite][::7]:
        assert oracle.double_to_half(float(np.uint16(b).view(np.float16))) == int(b)
    # midpoints between neighbouring positive halves go to the even one
    pos = np.arange(0, 0x7BFF, 37, dtype=np.uint16)
    for b in pos:
        lo = float(np.uint16(b).view(np.float16))
        hi = float(np.uint16(b + 1).view(np.float16))
        mid = 0.5 * (lo + hi)
        even = int(b) if b % 2 == 0 else int(b) + 1
        assert oracle.double_to_half(mid) == even
        assert oracle.double_to_half(np.nextafter(mid, 0.0)) == int(b)
        assert oracle.double_to_half(np.nextafter(mid, 1e9)) == int(b) + 1
    # overflow threshold: 65504 is the largest half; 65520 and above round to infinity
    assert oracle.double_to_half(65504.0) == 0x7BFF
    assert oracle.double_to_half(65519.99) == 0x7BFF
    assert oracle.double_to_half(65520.0) == 0x7C00
    assert oracle.double_to_half(-1e9) == 0xFC00
    # smallest subnormal: 2^-25 is a tie between 0 and 2^-24 -> even (0)
    assert oracle.double_to_half(2.0 ** -25) == 0
    assert oracle.double_to_half(np.nextafter(2.0 ** -25, 1.0)) == 1


def test_double_to_half_random_against_numpy():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-5, 2000), rng.normal(0, 3e4, 2000),
                        rng.normal(0, 1e-7, 1000)])
    want = x.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


# ------------------------------------------------------------------------------ hand-built blocks
@pytest.mark.parametrize("name", ["A", "B"])
def test_handbuilt_block_fields_and_weights(name):
    blk = handbuilt_blocks()[name]
    d, dmin, sc, m = oracle.q4k_fields(blk["bytes"])
    assert d == blk["d"] and dmin == blk["dmin"]
    assert list(sc) == blk["sc"] and list(m) == blk["m"]
    w = oracle.q4k_dequant(blk["bytes"])
    for idx, val in blk["w"].items():
        assert w[idx] == val, (idx, w[idx], val)
    w32 = oracle.q4k_dequant(blk["bytes"], np.float32)
    assert np.array_equal(w32, w.astype(np.float32))


def test_zero_nibbles_give_minus_dmin_m_and_full_nibbles_give_15_d_sc():
    sc = [3, 9, 27, 63, 1, 40, 33, 17]
    m = [0, 1, 2, 62, 63, 31, 32, 16]
    d_bits, dmin_bits = 0x2E66, 0x3555          # 0.1 and 0.333 as halves (whatever they round to)
    d = float(np.uint16(d_bits).view(np.float16))
    dmin = float(np.uint16(dmin_bits).view(np.float16))
    zero = synth.build_blocks([d_bits], [dmin_bits], sc, m, np.zeros(256, np.uint8))
    w = oracle.q4k_dequant(zero).reshape(8, 32)
    for j in range(8):
        assert np.all(w[j] == -dmin * m[j])
    full = synth.build_blocks([d_bits], [dmin_bits], sc, [0] * 8, np.full(256, 15, np.uint8))
    w = oracle.q4k_dequant(full).reshape(8, 32)
    for j in range(8):
        assert np.all(w[j] == 15.0 * d * sc[j])


def _expected_field_of_bit(byte, bit):
    """The packing of the 12 header bytes, written as a table: (kind, j, bit of the 6-bit field)."""
    if byte < 4:
        return ("sc", byte, bit) if bit < 6 else ("sc", byte + 4, bit - 2)
    if byte < 8:
        return ("m", byte - 4, bit) if bit < 6 else ("m", byte, bit - 2)
    return ("sc", byte - 4, bit) if bit < 4 else ("m", byte - 4, bit - 4)


def test_each_header_bit_moves_exactly_one_field_by_a_power_of_two():
    base = np.zeros(144, np.uint8)
    base[0:4] = [0x00, 0x3C, 0x00, 0x3C]
    _, _, sc0, m0 = oracle.q4k_fields(base)
    assert not sc0.any() and not m0.any()
    seen = set()
    for byte in range(12):
        for bit in range(8):
            blk = base.copy()
            blk[4 + byte] = 1 << bit
            _, _, sc, m = oracle.q4k_fields(blk)
            kind, j, fbit = _expected_field_of_bit(byte, bit)
            want_sc, want_m = np.zeros(8, np.int32), np.zeros(8, np.int32)
            (want_sc if kind == "sc" else want_m)[j] = 1 << fbit
            assert np.array_equal(sc, want_sc) and np.array_equal(m, want_m), (byte, bit)
            seen.add((kind, j, fbit))
    assert len(seen) == 96          # every bit of the sixteen 6-bit fields is reachable exactly once


def test_each_nibble_position_maps_to_one_weight():
    # a single nibble set to 1 with d = sc = 1 and no mins lights exactly one weight
    for byte in range(0, 128, 5):
        for hi in (0, 1):
            q = np.zeros(256, np.uint8)
            p, i = byte // 32, byte % 32
            k = 64 * p + 32 * hi + i
            blk = synth.build_blocks([0x3C00], [0], [1] * 8, [0] * 8, q)[0]
            blk[16 + byte] = 1 << (4 * hi)
            w = oracle.q4k_dequant(blk)
            assert w[k] == 1.0 and np.count_nonzero(w) == 1


def test_pack_is_inverse_of_decode_and_matches_the_generator_packer():
    rng = np.random.default_rng(11)
    for _ in range(50):
        sc = rng.integers(0, 64, 8)
        m = rng.integers(0, 64, 8)
        q = rng.integers(0, 16, 256).astype(np.uint8)
        d_bits, dmin_bits = int(rng.integers(0, 0x7C00)), int(rng.integers(0, 0x7C00))
        a = oracle.q4k_pack(d_bits, dmin_bits, sc, m, q)
        b = synth.build_blocks([d_bits], [dmin_bits], sc, m, q)[0]
        assert np.array_equal(a, b)
        d, dmin, sc2, m2 = oracle.q4k_fields(a)
        assert np.array_equal(sc2, sc) and np.array_equal(m2, m)
        assert d == float(np.uint16(d_bits).view(np.float16)) and dmin == float(np.uint16(dmin_bits).view(np.float16))


# ------------------------------------------------------------------- dequant and GEMV, brute force
def _dense_from_fields(rng, rows, cols):
    """Random fields -> (packed bytes, dense fp64 matrix computed from the fields directly)."""
    n_sb = rows * cols // 256
    sc = rng.integers(0, 64, (n_sb, 8))
    m = rng.integers(0, 64, (n_sb, 8))
    q = rng.integers(0, 16, (n_sb, 256))
    d16 = np.abs(rng.normal(0, 0.01, n_sb)).astype(np.float16)
    dmin16 = np.abs(rng.normal(0, 0.01, n_sb)).astype(np.float16)
    blocks = synth.build_blocks(d16.view(np.uint16), dmin16.view(np.uint16), sc, m, q)
    d = d16.astype(np.float64)[:, None]
    dmin = dmin16.astype(np.float64)[:, None]
    dense = d * np.repeat(sc, 32, axis=1) * q - dmin * np.repeat(m, 32, axis=1)
    return blocks.reshape(-1), dense.reshape(rows, cols)


@pytest.mark.parametrize("rows,cols", [(8, 256), (4, 512), (5, 768)])
def test_dequant_equals_dense_matrix_from_fields(rows, cols):
    blocks, dense = _dense_from_fields(np.random.default_rng(rows * cols), rows, cols)
    got = oracle.q4k_dequant(blocks).reshape(rows, cols)
    assert np.array_equal(got, dense)             # every product is exact in fp64
    got32 = oracle.q4k_dequant(blocks, np.float32).reshape(rows, cols)
    assert np.array_equal(got32, dense.astype(np.float32))


@pytest.mark.parametrize("rows,cols,n_cols", [(8, 256, 1), (4, 512, 3), (7, 1024, 5)])
def test_gemv_equals_dense_dot(rows, cols, n_cols):
    rng = np.random.default_rng(rows + cols + n_cols)
    blocks, dense = _dense_from_fields(rng, rows, cols)
    x = rng.normal(0, 1, (n_cols, cols)).astype(np.float32)
    y, s = oracle.gemv_q4k(blocks, rows, cols, x, n_threads=3)
    want = x.astype(np.float64) @ dense.T          # [n_cols, rows]
    want_abs = np.abs(x.astype(np.float64))[:, None, :] * np.abs(dense)[None, :, :]
    assert y.shape == (n_cols, rows)
    np.testing.assert_allclose(y, want, rtol=0, atol=1e-12 * want_abs.sum(-1).max())
    np.testing.assert_allclose(s, want_abs.sum(-1), rtol=1e-13)


def test_gemv_picks_rows_and_columns_the_right_way_round():
    # W has a single non-zero weight at (row 2, column 300); x is a one-hot at 300.
    rows, cols = 4, 512
    q = np.zeros((rows * 2, 256), np.uint8)
    q[2 * 2 + 1, 300 - 256] = 9                    # row 2, second super-block, column 44 inside it
    blocks = synth.build_blocks([0x3C00] * 8, [0] * 8, np.ones((8, 8)), np.zeros((8, 8)), q).reshape(-1)
    x = np.zeros((1, cols), np.float32)
    x[0, 300] = 2.0
    y, _ = oracle.gemv_q4k(blocks, rows, cols, x)
    assert np.array_equal(y[0], [0, 0, 18.0, 0])
    x[:] = 0
    x[0, 299] = 2.0
    y, _ = oracle.gemv_q4k(blocks, rows, cols, x)
    assert not y.any()


def test_gemv_thread_count_does_not_change_bits():
    w, x = synth.gemv_case(seed=3, rows=64, cols=512, n_cols=2)
    y1, s1 = oracle.gemv_q4k(w, 64, 512, x, n_threads=1)
    y8, s8 = oracle.gemv_q4k(w, 64, 512, x, n_threads=8)
    assert np.array_equal(y1, y8) and np.array_equal(s1, s8)


def test_generator_distributions():
    # the literal GEMV workload: fields uniform, d and dmin half-normal with sigma 0.01
    w, x = synth.gemv_case(seed=0, rows=256, cols=1024)
    blocks = w.reshape(-1, 144)
    f = [oracle.q4k_fields(b) for b in blocks[:400]]
    sc = np.array([t[2] for t in f]).ravel()
    m = np.array([t[3] for t in f]).ravel()
    d = np.array([t[0] for t in f])
    assert sc.min() == 0 and sc.max() == 63 and abs(sc.mean() - 31.5) < 1.5
    assert m.min() == 0 and m.max() == 63 and abs(m.mean() - 31.5) < 1.5
    assert abs(d.mean() - 0.01 * np.sqrt(2 / np.pi)) < 1e-3
    nib = np.concatenate([blocks[:, 16:] & 15, blocks[:, 16:] >> 4]).ravel()
    assert abs(nib.mean() - 7.5) < 0.05
    assert x.dtype == np.float32 and abs(float(x.std()) - 1.0) < 0.05
    # the model recipe: rows are zero-mean with standard deviation close to 1/sqrt(cols)
    wm = synth.model_tensor(1, 0, synth.WQ, 128, 1024)
    dense = oracle.q4k_dequant(wm).reshape(128, 1024)
    assert abs(dense.mean()) < 0.02 / np.sqrt(1024) * 4
    assert 0.8 / np.sqrt(1024) < dense.std() < 1.25 / np.sqrt(1024)
    # deterministic, and different tensors differ
    assert np.array_equal(wm, synth.model_tensor(1, 0, synth.WQ, 128, 1024))
    assert not np.array_equal(wm, synth.model_tensor(1, 1, synth.WQ, 128, 1024))


def test_dequant_agrees_with_the_gguf_package_decoder_on_random_blocks():
    """An extra, not a pin: the gguf Python package (when it is installed) decodes the same bytes to the
    same values, which shows that the layout defined here is the public Q4_K arrangement."""
    gguf = pytest.importorskip("gguf")
    from gguf import quants
    rng = np.random.default_rng(77)
    n = 300
    blocks = rng.integers(0, 256, (n, oracle.BLOCK_BYTES), dtype=np.uint8)
    # keep d and dmin finite: clear the top exponent bit of both halves
    blocks[:, 1] &= 0xBF
    blocks[:, 3] &= 0xBF
    want = quants.dequantize(blocks.reshape(-1), gguf.GGMLQuantizationType.Q4_K).reshape(-1).astype(np.float64)
    got32 = oracle.q4k_dequant(blocks, np.float32).astype(np.float64)
    got64 = oracle.q4k_dequant(blocks, np.float64)
    # the package computes in fp32 with a rounding per operation; this checker rounds the exact value once:
    # allow 3 units of fp32 rounding on the two terms' magnitudes (they may cancel)
    mag = np.empty((n, 256))
    for i in range(n):
        d, dmin, sc, m = oracle.q4k_fields(blocks[i])
        mag[i] = (abs(d) * np.repeat(sc, 32) * 15.0 + abs(dmin) * np.repeat(m, 32))
    tol = 3 * 2.0 ** -24 * mag.reshape(-1) + 1e-40
    assert np.all(np.abs(want - got64) <= tol)
    assert np.all(np.abs(want - got32) <= tol)
