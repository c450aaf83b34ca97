"""Several independent requests per step (one token each, own KV cache and position): the GPU step against the
CPU checker run once per request, and against the GPU's own single-request path."""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu

HIDDEN_TOL = 2e-3
LOGIT_TOL = 2e-2


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def _rel(got, want):
    rms = np.sqrt(np.mean(want.astype(np.float64) ** 2, axis=-1, keepdims=True))
    return float((np.abs(got.astype(np.float64) - want) / rms).max())


@pytest.mark.parametrize("name,seqs,lengths", [
    ("tiny", [0, 1, 2], [5, 0, 33]),
    ("small", [3, 0, 7, 1, 2, 9], [130, 17, 255, 1, 64, 128]),      # 6 requests: the multi-token product kernel
    ("small", [3, 0, 7, 1, 2, 9, 11, 5, 4], [130, 17, 255, 1, 64, 128, 0, 300, 77]),      # 9: two column blocks, the second nearly empty
    ("small", list(range(12)), [13 * i + 1 for i in range(12)]),
    ("small", list(range(15, -1, -1)), [19 * i for i in range(16)]),                    # 16 requests: both column blocks full
])
def test_requests_step_matches_checker_per_request(gpu, name, seqs, lengths):
    torch, binding = gpu
    cfg = synth.model_config(name, max_n_tok=16)
    L, n = cfg["n_layers"], len(seqs)
    ctx = binding.Context(cfg)
    refs = [oracle.Model(cfg) for _ in seqs]                       # the checker has one cache per model: one model per request
    for layer, tid, rows, cols, data in synth.iter_model_tensors(31, cfg):
        ctx.load(layer, tid, data, rows, cols)
        for r in refs:
            r.load(layer, tid, data, rows, cols)
    for i, (sq, ln) in enumerate(zip(seqs, lengths)):
        for l in range(L):
            if ln:
                k, v = synth.kv_prefill(100 + sq, l, ln, cfg["n_kv_heads"], cfg["head_dim"])
                ctx.kv_load(l, 0, k, v, seq=sq)
                refs[i].kv_load(l, 0, k, v)
    h0 = synth.activations(31, n, cfg["hidden"])
    want = np.concatenate([refs[i].forward_window(0, L, h0[i:i + 1], lengths[i]) for i in range(n)])
    hin = torch.from_numpy(h0).cuda()
    hout = torch.empty_like(hin)
    ctx.forward_window_seqs(0, 2, hin, hout, seqs, lengths)        # two windows
    ctx.forward_window_seqs(2, L, hout, hout, seqs, lengths)
    ctx.sync()
    got = hout.cpu().numpy()
    assert _rel(got, want) <= HIDDEN_TOL
    logits = torch.empty((n, cfg["vocab"]), dtype=torch.float32, device="cuda")
    ctx.logits(hout, n, logits)
    ctx.sync()
    want_logits = np.concatenate([refs[i].logits(want[i:i + 1]) for i in range(n)])
    assert np.abs(logits.cpu().numpy().astype(np.float64) - want_logits).max() <= LOGIT_TOL
    # the appended cache entries went to each request's own cache, at its own position
    for i, (sq, ln) in enumerate(zip(seqs, lengths)):
        for l in range(L):
            kr, vr = refs[i].kv_read(l, ln, 1)
            kg, vg = ctx.kv_read(l, ln, 1, seq=sq)
            for a, b in ((kr, kg), (vr, vg)):
                fa, fb = a.view(np.float16).astype(np.float64), b.view(np.float16).astype(np.float64)
                assert np.abs(fa - fb).max() <= 4e-3 * max(1.0, np.abs(fa).max())
    # each request alone through the single-request call (sequence 0 of a fresh context) agrees too
    solo = binding.Context(cfg)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(31, cfg):
        solo.load(layer, tid, data, rows, cols)
    i = n - 1
    for l in range(L):
        if lengths[i]:
            k, v = synth.kv_prefill(100 + seqs[i], l, lengths[i], cfg["n_kv_heads"], cfg["head_dim"])
            solo.kv_load(l, 0, k, v)
    one_in = torch.from_numpy(h0[i:i + 1]).cuda()
    one_out = torch.empty_like(one_in)
    solo.forward_window(0, L, one_in, one_out, lengths[i], 1)
    solo.sync()
    assert _rel(one_out.cpu().numpy(), got[i:i + 1]) <= HIDDEN_TOL
    for r in refs:
        r.close()
    ctx.close()
    solo.close()


def test_requests_step_rejects_bad_arguments(gpu):
    torch, binding = gpu
    cfg = synth.model_config("tiny")
    ctx = binding.Context(cfg)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(31, cfg):
        ctx.load(layer, tid, data, rows, cols)
    h = torch.zeros((2, cfg["hidden"]), dtype=torch.float32, device="cuda")
    for seqs, pos in (([0, 0], [1, 2]), ([0, 64], [1, 2]), ([0, -1], [1, 2]), ([0, 1], [1, cfg["kv_capacity"]]), ([0, 1], [-1, 0])):
        with pytest.raises(binding.PrimaError) as err:
            ctx.forward_window_seqs(0, cfg["n_layers"], h, h, seqs, pos)
        assert err.value.code == binding.ERR_ARG
    ctx.forward_window_seqs(0, cfg["n_layers"], h, h, [0, 1], [0, 0])      # still usable
    ctx.sync()
    ctx.close()
