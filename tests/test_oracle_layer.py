"""Pins for the CPU checker's layer arithmetic: closed forms, invariants, library special cases and
a dense numpy re-computation of a tiny model built from explicitly chosen weights."""
import numpy as np
import pytest
import scipy.special

import oracle
from paper_2504_08791_b200 import synth


def _f16(a):
    return np.asarray(a, np.float64).astype(np.float16)


# ---------------------------------------------------------------------------------------- RMSNorm
def test_rmsnorm_constant_vector_closed_form():
    for c, eps in [(2.0, 1e-5), (-0.5, 1e-6), (1e-3, 1e-5)]:
        h = np.full(64, c)
        out = oracle.rmsnorm(h, np.ones(64, np.float32), eps)
        np.testing.assert_allclose(out, c / np.sqrt(c * c + eps), rtol=1e-15)


def test_rmsnorm_unit_rms_gain_and_scale_invariance():
    rng = np.random.default_rng(0)
    h = rng.normal(0, 3, 512)
    g = rng.normal(1, 0.1, 512).astype(np.float32)
    out1 = oracle.rmsnorm(h, np.ones(512, np.float32), 0.0)
    assert abs(np.sqrt(np.mean(out1 ** 2)) - 1.0) < 1e-14
    np.testing.assert_allclose(oracle.rmsnorm(7.0 * h, g, 0.0), oracle.rmsnorm(h, g, 0.0), rtol=1e-14)
    np.testing.assert_allclose(oracle.rmsnorm(h, g, 0.0), out1 * g.astype(np.float64), rtol=1e-15)
    # eps enters under the root, added to the MEAN of squares (not the sum)
    h2 = np.array([3.0, 4.0])
    np.testing.assert_allclose(oracle.rmsnorm(h2, np.ones(2, np.float32), 0.5), h2 / np.sqrt(12.5 + 0.5), rtol=1e-15)


# ------------------------------------------------------------------------------------------- RoPE
def test_rope_unit_vectors_give_cos_and_sin_at_the_paired_index():
    D, theta = 128, 1e4
    for pos in (0, 1, 17, 4095):
        e0 = np.zeros((1, D))
        e0[0, 0] = 1.0
        out = oracle.rope(e0, pos, theta, 0)[0]
        assert abs(out[0] - np.cos(pos)) < 1e-12 and abs(out[D // 2] - np.sin(pos)) < 1e-12
        assert np.count_nonzero(np.abs(out) > 1e-15) <= 2
        out1 = oracle.rope(e0, pos, theta, 1)[0]
        assert abs(out1[0] - np.cos(pos)) < 1e-12 and abs(out1[1] - np.sin(pos)) < 1e-12
        # pair i = D/4 turns at frequency theta^(-1/2) = 0.01
        ei = np.zeros((1, D))
        ei[0, D // 4] = 1.0
        out = oracle.rope(ei, pos, theta, 0)[0]
        assert abs(out[D // 4] - np.cos(0.01 * pos)) < 1e-12 and abs(out[D // 4 + D // 2] - np.sin(0.01 * pos)) < 1e-12
        # the partner of the pair turns the other way round: (0,1) -> (-sin, cos)
        ej = np.zeros((1, D))
        ej[0, D // 2] = 1.0
        out = oracle.rope(ej, pos, theta, 0)[0]
        assert abs(out[0] + np.sin(pos)) < 1e-12 and abs(out[D // 2] - np.cos(pos)) < 1e-12


def test_rope_interleaved_mode_uses_pair_index_not_element_index_for_the_frequency():
    """Mode 1 pairs (2i, 2i+1); pair i turns at theta^(-2i/D).  Pair D/4 (elements D/2, D/2+1) at
    theta = 1e4 turns at exactly 0.01 rad per position, pair 1 (elements 2, 3) at 1e4^(-1/64)."""
    D, theta = 128, 1e4
    for pos in (1, 17, 4095):
        e = np.zeros((2, D))
        e[0, D // 2] = 1.0           # first element of pair D/4
        e[1, D // 2 + 1] = 1.0       # its partner
        out = oracle.rope(e, pos, theta, 1)
        assert abs(out[0, D // 2] - np.cos(0.01 * pos)) < 1e-12 and abs(out[0, D // 2 + 1] - np.sin(0.01 * pos)) < 1e-12
        assert abs(out[1, D // 2] + np.sin(0.01 * pos)) < 1e-12 and abs(out[1, D // 2 + 1] - np.cos(0.01 * pos)) < 1e-12
        assert np.count_nonzero(np.abs(out) > 1e-15) <= 4
        f1 = theta ** (-2.0 / D)
        e = np.zeros((1, D))
        e[0, 2] = 1.0
        out = oracle.rope(e, pos, theta, 1)[0]
        assert abs(out[2] - np.cos(f1 * pos)) < 1e-12 and abs(out[3] - np.sin(f1 * pos)) < 1e-12
        # the last pair is the slowest one
        fl = theta ** (-2.0 * (D // 2 - 1) / D)
        e = np.zeros((1, D))
        e[0, D - 2] = 1.0
        out = oracle.rope(e, pos, theta, 1)[0]
        assert abs(out[D - 2] - np.cos(fl * pos)) < 1e-12 and abs(out[D - 1] - np.sin(fl * pos)) < 1e-12


def test_rope_modes_are_the_same_rotation_up_to_the_fixed_permutation_of_elements():
    rng = np.random.default_rng(5)
    D, theta = 128, 5e5
    x = rng.normal(0, 1, (4, D))
    perm = np.empty(D, np.int64)            # element of the interleaved layout that holds split-layout element k
    perm[:D // 2] = 2 * np.arange(D // 2)
    perm[D // 2:] = 2 * np.arange(D // 2) + 1
    y = np.empty_like(x)
    y[:, perm] = x                           # y in interleaved layout = x in split layout
    a = oracle.rope(x, 321, theta, 0)
    b = oracle.rope(y, 321, theta, 1)
    np.testing.assert_allclose(b[:, perm], a, rtol=0, atol=1e-13)


def test_rope_is_identity_at_zero_preserves_norms_and_is_relative():
    rng = np.random.default_rng(1)
    D, theta = 128, 5e5
    q = rng.normal(0, 1, (3, D))
    k = rng.normal(0, 1, (3, D))
    assert np.array_equal(oracle.rope(q, 0, theta, 0), q)
    r = oracle.rope(q, 777, theta, 0)
    np.testing.assert_allclose(r[:, :64] ** 2 + r[:, 64:] ** 2, q[:, :64] ** 2 + q[:, 64:] ** 2, rtol=1e-12)
    for mode in (0, 1):
        a = np.sum(oracle.rope(q, 1000, theta, mode) * oracle.rope(k, 990, theta, mode), axis=1)
        b = np.sum(oracle.rope(q, 25, theta, mode) * oracle.rope(k, 15, theta, mode), axis=1)
        np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-9)
    # composition: rotating by p then by r equals rotating by p + r (angles add)
    np.testing.assert_allclose(oracle.rope(oracle.rope(q, 40, theta, 0), 2, theta, 0), oracle.rope(q, 42, theta, 0), atol=1e-12)


# -------------------------------------------------------------------------------------- attention
def test_attention_single_position_returns_v0_and_uniform_keys_return_the_mean():
    rng = np.random.default_rng(2)
    D = 128
    q = rng.normal(0, 1, D)
    k = _f16(rng.normal(0, 1, (1, D)))
    v = _f16(rng.normal(0, 1, (1, D)))
    out = oracle.attend(q, k.view(np.uint16), v.view(np.uint16))
    assert np.array_equal(out, v[0].astype(np.float64))
    n = 37
    k = np.repeat(_f16(rng.normal(0, 1, (1, D))), n, axis=0)
    v = _f16(rng.normal(0, 1, (n, D)))
    out = oracle.attend(q, k.view(np.uint16), v.view(np.uint16))
    np.testing.assert_allclose(out, v.astype(np.float64).mean(0), rtol=1e-12, atol=1e-14)


def test_attention_matches_library_softmax_and_is_permutation_invariant():
    rng = np.random.default_rng(3)
    D, n = 128, 200
    q = rng.normal(0, 1, D)
    k = _f16(rng.normal(0, 1, (n, D)))
    v = _f16(rng.normal(0, 1, (n, D)))
    p = scipy.special.softmax(k.astype(np.float64) @ q / np.sqrt(D))
    want = p @ v.astype(np.float64)
    out = oracle.attend(q, k.view(np.uint16), v.view(np.uint16))
    np.testing.assert_allclose(out, want, rtol=1e-11, atol=1e-13)
    perm = rng.permutation(n)
    out2 = oracle.attend(q, k[perm].view(np.uint16), v[perm].view(np.uint16))
    np.testing.assert_allclose(out2, out, rtol=1e-11, atol=1e-13)


def test_attention_large_scores_do_not_overflow():
    D = 128
    q = np.full(D, 100.0)
    k = _f16(np.stack([np.full(D, 60000.0), np.full(D, -60000.0), np.full(D, 59000.0)]))
    v = _f16(np.stack([np.full(D, 1.0), np.full(D, 2.0), np.full(D, 3.0)]))
    out = oracle.attend(q, k.view(np.uint16), v.view(np.uint16))
    assert np.all(np.isfinite(out))
    np.testing.assert_allclose(out, 1.0, rtol=1e-12)     # the first key wins by e^(huge)


def test_silu():
    assert oracle.silu(0.0) == 0.0
    for z in (0.3, 1.0, 5.0, 30.0):
        assert abs(oracle.silu(z) - oracle.silu(-z) - z) < 1e-12 * max(1, z)     # silu(z) - silu(-z) = z
        assert abs(oracle.silu(z) - z * scipy.special.expit(z)) < 1e-15 * max(1, z)
    assert abs(oracle.silu(50.0) - 50.0) < 1e-12 and abs(oracle.silu(-50.0)) < 1e-12


# ------------------------------------------------------------------------------- model-level pins
def _explicit_matrix(rng, rows, cols, scale):
    """Weights chosen field by field -> (bytes, dense fp64 matrix from the fields)."""
    n_sb = rows * cols // 256
    sc = rng.integers(16, 64, (n_sb, 8))
    m = np.floor(7.5 * sc / 8 + 0.5).astype(np.int64)
    q = rng.integers(0, 16, (n_sb, 256))
    d16 = (scale * (0.5 + rng.random(n_sb)) / (4.61 * 40.0)).astype(np.float16)
    dmin16 = (d16.astype(np.float32) * 8).astype(np.float16)
    blocks = synth.build_blocks(d16.view(np.uint16), dmin16.view(np.uint16), sc, m, q)
    dense = (d16.astype(np.float64)[:, None] * np.repeat(sc, 32, 1) * q
             - dmin16.astype(np.float64)[:, None] * np.repeat(m, 32, 1))
    return blocks.reshape(-1), dense.reshape(rows, cols)


def _build_explicit_model(cfg, seed):
    rng = np.random.default_rng(seed)
    mdl = oracle.Model(cfg, n_threads=4)
    dense = {}
    for layer in range(cfg["n_layers"]):
        for tid in synth.LAYER_TENSORS:
            rows, cols = synth.tensor_shape(cfg, tid)
            if tid in (synth.ATTN_NORM, synth.FFN_NORM):
                g = (1 + 0.1 * rng.normal(0, 1, cols)).astype(np.float32)
                mdl.load(layer, tid, g, 1, cols, copy=True)
                dense[(layer, tid)] = g.astype(np.float64)
            else:
                b, w = _explicit_matrix(rng, rows, cols, 1 / np.sqrt(cols))
                mdl.load(layer, tid, b, rows, cols, copy=True)
                dense[(layer, tid)] = w
    for tid in synth.GLOBAL_TENSORS:
        rows, cols = synth.tensor_shape(cfg, tid)
        if tid == synth.OUT_NORM:
            g = (1 + 0.1 * rng.normal(0, 1, cols)).astype(np.float32)
            mdl.load(-1, tid, g, 1, cols, copy=True)
            dense[(-1, tid)] = g.astype(np.float64)
        else:
            b, w = _explicit_matrix(rng, rows, cols, 4 / np.sqrt(cols) if tid == synth.W_HEAD else 1.0)
            mdl.load(-1, tid, b, rows, cols, copy=True)
            dense[(-1, tid)] = w
    return mdl, dense


def _np_rms(h, g, eps):
    return h / np.sqrt(np.mean(h * h) + eps) * g


def _np_rope(x, pos, theta, mode=0):  # x: [heads, D]; mode 0 pairs (i, i + D/2), mode 1 pairs (2i, 2i + 1)
    D = x.shape[1]
    ang = pos * theta ** (-2.0 * np.arange(D // 2) / D)
    c, s = np.cos(ang), np.sin(ang)
    if mode == 0:
        a, b = x[:, :D // 2], x[:, D // 2:]
        return np.concatenate([a * c - b * s, b * c + a * s], axis=1)
    a, b = x[:, 0::2], x[:, 1::2]
    out = np.empty_like(x)
    out[:, 0::2] = a * c - b * s
    out[:, 1::2] = b * c + a * s
    return out


def _np_forward(cfg, dense, h, pos, kv):
    """Dense numpy forward of all layers for ONE token; kv[l] = (K[list of G x D], V[...])."""
    e, H, G, D = cfg["hidden"], cfg["n_q_heads"], cfg["n_kv_heads"], cfg["head_dim"]
    h = h.astype(np.float32)
    for l in range(cfg["n_layers"]):
        hd = h.astype(np.float64)
        a = _np_rms(hd, dense[(l, synth.ATTN_NORM)], cfg["rms_eps"])
        q = _np_rope((dense[(l, synth.WQ)] @ a).reshape(H, D), pos, cfg["rope_theta"], cfg.get("rope_mode", 0))
        k = _np_rope((dense[(l, synth.WK)] @ a).reshape(G, D), pos, cfg["rope_theta"], cfg.get("rope_mode", 0))
        v = (dense[(l, synth.WV)] @ a).reshape(G, D)
        K, V = kv[l]
        K[pos] = k.astype(np.float16).astype(np.float64)
        V[pos] = v.astype(np.float16).astype(np.float64)
        o = np.zeros((H, D))
        for hh in range(H):
            g = hh // (H // G)
            s = np.array([K[j][g] @ q[hh] for j in range(pos + 1)]) / np.sqrt(D)
            p = scipy.special.softmax(s)
            o[hh] = sum(p[j] * V[j][g] for j in range(pos + 1))
        h = (hd + dense[(l, synth.WO)] @ o.reshape(-1)).astype(np.float32)
        hd = h.astype(np.float64)
        b = _np_rms(hd, dense[(l, synth.FFN_NORM)], cfg["rms_eps"])
        gate, up = dense[(l, synth.W_GATE)] @ b, dense[(l, synth.W_UP)] @ b
        act = gate * scipy.special.expit(gate) * up
        h = (hd + dense[(l, synth.W_DOWN)] @ act).astype(np.float32)
    return h


TINY = synth.model_config("tiny")


@pytest.mark.parametrize("rope_mode", [0, 1])
def test_tiny_model_matches_dense_numpy_forward_over_several_tokens(rope_mode):
    cfg = dict(TINY, rope_mode=rope_mode)
    mdl, dense = _build_explicit_model(cfg, seed=21)
    kv = [({}, {}) for _ in range(cfg["n_layers"])]
    tokens = [3, 700, 41, 5]
    for pos, tok in enumerate(tokens):
        h0 = mdl.embed([tok])
        assert np.array_equal(h0[0], dense[(-1, synth.TOK_EMBD)][tok].astype(np.float32))
        got = mdl.forward_window(0, cfg["n_layers"], h0, pos)
        want = _np_forward(cfg, dense, h0[0], pos, kv)
        np.testing.assert_allclose(got[0], want, rtol=0, atol=2e-6 * np.abs(want).max())
        logits = mdl.logits(got)
        want_logits = dense[(-1, synth.W_HEAD)] @ _np_rms(got[0].astype(np.float64), dense[(-1, synth.OUT_NORM)], cfg["rms_eps"])
        np.testing.assert_allclose(logits[0], want_logits, rtol=0, atol=1e-5)
        assert logits.dtype == np.float32
    # the cache holds fp16 roundings of the rotated keys: 2 (h_k e_k + h_v e_v) bytes per token and layer
    k, v = mdl.kv_read(1, 0, len(tokens))
    assert k.nbytes + v.nbytes == len(tokens) * 2 * (cfg["n_kv_heads"] * cfg["head_dim"] * 2)
    for pos in range(len(tokens)):
        assert np.array_equal(k[pos].view(np.float16).astype(np.float64), kv[1][0][pos])
        assert np.array_equal(v[pos].view(np.float16).astype(np.float64), kv[1][1][pos])


def _synthetic_model(cfg, seed, n_prefill):
    mdl = oracle.Model(cfg, n_threads=4)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg):
        mdl.load(layer, tid, data, rows, cols)
    for l in range(cfg["n_layers"]):
        k, v = synth.kv_prefill(seed, l, n_prefill, cfg["n_kv_heads"], cfg["head_dim"])
        mdl.kv_load(l, 0, k, v)
    return mdl


@pytest.mark.parametrize("splits", [[(0, 1), (1, 2), (2, 3)], [(0, 2), (2, 3)], [(0, 1), (1, 3)]])
def test_any_split_into_windows_reproduces_the_full_pass_bit_for_bit(splits):
    cfg, seed, pos = TINY, 7, 40
    h0 = synth.activations(seed, 2, cfg["hidden"])
    full = _synthetic_model(cfg, seed, pos)
    want = full.forward_window(0, cfg["n_layers"], h0, pos)
    part = _synthetic_model(cfg, seed, pos)
    h = h0
    for lb, le in splits:
        h = part.forward_window(lb, le, h, pos)
    assert np.array_equal(h, want)
    for l in range(cfg["n_layers"]):
        for a, b in zip(full.kv_read(l, 0, pos + 2), part.kv_read(l, 0, pos + 2)):
            assert np.array_equal(a, b)
    # the boundary message is e fp32 values per token
    assert h.dtype == np.float32 and h.shape == (2, cfg["hidden"]) and h[0].nbytes == 4 * cfg["hidden"]


def test_a_step_of_five_tokens_equals_five_single_token_steps():
    cfg, seed, pos = TINY, 9, 30
    h0 = synth.activations(seed, 5, cfg["hidden"])
    a = _synthetic_model(cfg, seed, pos)
    batch = a.forward_window(0, cfg["n_layers"], h0, pos)
    b = _synthetic_model(cfg, seed, pos)
    single = np.stack([b.forward_window(0, cfg["n_layers"], h0[t:t + 1], pos + t)[0] for t in range(5)])
    assert np.array_equal(batch, single)
    assert np.array_equal(a.logits(batch), b.logits(single))
    for l in range(cfg["n_layers"]):
        for x, y in zip(a.kv_read(l, 0, pos + 5), b.kv_read(l, 0, pos + 5)):
            assert np.array_equal(x, y)


def test_step_is_causal_later_tokens_do_not_change_earlier_outputs():
    cfg, seed, pos = TINY, 10, 20
    h0 = synth.activations(seed, 4, cfg["hidden"])
    h1 = h0.copy()
    h1[3] += 1.0
    a = _synthetic_model(cfg, seed, pos).forward_window(0, cfg["n_layers"], h0, pos)
    b = _synthetic_model(cfg, seed, pos).forward_window(0, cfg["n_layers"], h1, pos)
    assert np.array_equal(a[:3], b[:3]) and not np.array_equal(a[3], b[3])


def test_query_heads_read_their_own_kv_group():
    # values of KV head g are the constant g+1 everywhere; with W_o = "sum over each head's lanes"
    # this cannot be seen directly, so check through attend(): head h must use group h // (H/G).
    cfg = dict(TINY, n_layers=1)
    seed, pos = 12, 16
    mdl = _synthetic_model(cfg, seed, pos)
    G, D, H = cfg["n_kv_heads"], cfg["head_dim"], cfg["n_q_heads"]
    k, v = synth.kv_prefill(seed, 0, pos, G, D)
    # swapping the two KV heads' contents must change the output; swapping back restores it
    h0 = synth.activations(seed, 1, cfg["hidden"])
    base = mdl.forward_window(0, 1, h0, pos)
    mdl.kv_load(0, 0, k[:, ::-1], v[:, ::-1])
    swapped = mdl.forward_window(0, 1, h0, pos)
    assert not np.array_equal(base, swapped)
    mdl.kv_load(0, 0, k, v)
    assert np.array_equal(mdl.forward_window(0, 1, h0, pos), base)


def test_argmax_takes_lowest_index_on_ties_and_reports_margin():
    idx, margin = oracle.argmax(np.array([0.5, 2.0, 2.0, -1.0], np.float32))
    assert idx == 1 and margin == 0.0
    idx, margin = oracle.argmax(np.array([0.5, 2.0, 3.5, -1.0], np.float32))
    assert idx == 2 and margin == 1.5


def test_bad_arguments_are_rejected():
    mdl = _synthetic_model(TINY, 1, 4)
    h = synth.activations(1, 1, TINY["hidden"])
    with pytest.raises(ValueError):
        mdl.forward_window(0, 4, h, 0)                      # layer range outside the model
    with pytest.raises(ValueError):
        mdl.forward_window(0, 1, h, TINY["kv_capacity"])    # position beyond the cache
    with pytest.raises(ValueError):
        oracle.gemv_q4k(np.zeros(144, np.uint8), 1, 200, np.zeros((1, 200), np.float32))
