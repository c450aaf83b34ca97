"""Per-row bound |y - y_ref| <= 1e-3 * sum |w x| on the two fused input paths every layer runs.

The plain input path is covered by the single-product tests.  Here:
* the output layer is a product whose staging step applies the RMSNorm gain and defers the scalar
  factor: every logit is compared with the checker's product of the head matrix with the checker's
  normalised vector, row by row, at hidden widths 8192 and 5120, for one token and for five;
* the down projection takes SwiGLU of the gate/up accumulators in its staging step: in a one-layer
  model whose output projection W_o is all zero blocks the attention block adds nothing, so
  hidden_out - hidden_in is the down projection alone, and each of its rows is bounded against the
  checker's product with the checker's own SwiGLU vector.
"""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu

ROW_TOL = 1e-3


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


@pytest.mark.parametrize("shape,vocab,n_tok", [("70b", 20011, 1), ("70b", 9000, 5), ("32b", 20011, 1), ("32b", 9000, 8)])
def test_every_logit_is_within_the_row_bound(gpu, shape, vocab, n_tok):
    torch, binding = gpu
    seed = 61
    cfg = synth.model_config(shape, n_layers=1, vocab=vocab)          # vocab not a multiple of 8: ragged last row tile
    e = cfg["hidden"]
    g_out = synth.make_tensor(seed, cfg, -1, synth.OUT_NORM)
    w_head = synth.make_tensor(seed, cfg, -1, synth.W_HEAD)
    ctx = binding.Context(cfg)
    ctx.load(-1, synth.OUT_NORM, g_out, 1, e)
    ctx.load(-1, synth.W_HEAD, w_head, vocab, e)
    h = synth.activations(seed, n_tok, e, scale=3.0)
    hin = torch.from_numpy(h).cuda()
    out = torch.empty((n_tok, vocab), dtype=torch.float32, device="cuda")
    ctx.logits(hin, n_tok, out)
    ctx.sync()
    got = out.cpu().numpy().astype(np.float64)
    a = np.stack([oracle.rmsnorm(h[t].astype(np.float64), g_out, cfg["rms_eps"]) for t in range(n_tok)])
    want, s_abs = oracle.gemv_q4k(w_head, vocab, e, a.astype(np.float32))
    ratio = np.abs(got - want) / s_abs
    print(f"{shape} head, {n_tok} token(s): worst row error {ratio.max():.2e} of sum|w x|")
    assert np.all(np.abs(got - want) <= ROW_TOL * s_abs)
    ctx.close()


@pytest.mark.parametrize("shape,n_tok,pos", [("8b", 1, 17), ("32b", 1, 130), ("32b", 6, 64)])
def test_every_row_of_the_down_projection_is_within_the_row_bound(gpu, shape, n_tok, pos):
    torch, binding = gpu
    seed = 67
    cfg = synth.model_config(shape, n_layers=1, vocab=512, kv_capacity=256)
    e, F = cfg["hidden"], cfg["ffn"]
    ctx = binding.Context(cfg)
    tensors = {}
    for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg, with_globals=False):
        if tid == synth.WO:
            data = np.zeros_like(data)            # d = dmin = 0 in every block: the matrix is zero
        tensors[tid] = data
        ctx.load(layer, tid, data, rows, cols)
    k, v = synth.kv_prefill(seed, 0, pos, cfg["n_kv_heads"], cfg["head_dim"])
    ctx.kv_load(0, 0, k, v)
    h = synth.activations(seed, n_tok, e)
    hin = torch.from_numpy(h).cuda()
    hout = torch.empty_like(hin)
    ctx.forward_window(0, 1, hin, hout, pos, n_tok)
    ctx.sync()
    got = hout.cpu().numpy().astype(np.float64) - h.astype(np.float64)
    # the checker's feed-forward block on the unchanged residual stream
    b = np.stack([oracle.rmsnorm(h[t].astype(np.float64), tensors[synth.FFN_NORM], cfg["rms_eps"]) for t in range(n_tok)]).astype(np.float32)
    gate, _ = oracle.gemv_q4k(tensors[synth.W_GATE], F, e, b)
    up, _ = oracle.gemv_q4k(tensors[synth.W_UP], F, e, b)
    act = np.vectorize(oracle.silu)(gate) * up
    want, s_abs = oracle.gemv_q4k(tensors[synth.W_DOWN], e, F, act.astype(np.float32))
    # hidden_out is rounded to fp32 after the addition: half an ulp of |h + y| on top of the row bound
    slack = 2.0 ** -23 * (np.abs(h.astype(np.float64)) + np.abs(want))
    ratio = (np.abs(got - want) - slack) / s_abs
    print(f"{shape} down projection, {n_tok} token(s): worst row error {ratio.max():.2e} of sum|w x|")
    assert np.all(np.abs(got - want) <= ROW_TOL * s_abs + slack)
    ctx.close()
