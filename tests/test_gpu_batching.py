"""Continuous batching on the GPU (Appendix A.11 / A.12): requests that join and leave between steps get the tokens
that the CPU checker's greedy decoding gives each of them alone."""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth
from paper_2504_08791_b200.batching import ContextExecutor, JobQueue

pytestmark = pytest.mark.gpu

MARGIN = 4e-2


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def checker_greedy(ref, cfg, prompt, n_new):
    """The checker alone on one request: its tokens and the smallest top-2 gap before each of them."""
    L = cfg["n_layers"]
    out, gaps, pos, tok = [], [], 0, None
    feed = list(prompt)
    while len(out) < n_new:
        t = feed.pop(0) if feed else out[-1]
        h = ref.forward_window(0, L, ref.embed([t]), pos)
        pos += 1
        if not feed:
            tok, gap = oracle.argmax(ref.logits(h)[0])
            out.append(int(tok))
            gaps.append(float(gap))
    return out, gaps


@pytest.mark.parametrize("max_batch,windows", [(4, None), (9, [0, 1, 4])])
def test_queue_gives_every_request_the_checkers_greedy_tokens(gpu, max_batch, windows):
    torch, binding = gpu
    cfg = synth.model_config("small", max_n_tok=16)
    ctx = binding.Context(cfg)
    tensors = list(synth.iter_model_tensors(59, cfg))
    for layer, tid, rows, cols, data in tensors:
        ctx.load(layer, tid, data, rows, cols)
    rng = np.random.default_rng(59)
    jobs = [(list(map(int, rng.integers(0, cfg["vocab"], size=int(rng.integers(1, 7))))), int(rng.integers(2, 9))) for _ in range(12)]
    q = JobQueue(ContextExecutor(ctx, windows=windows, max_batch=max_batch))
    ids = [q.submit(p, n) for p, n in jobs[:7]]
    for _ in range(4):
        q.step()
    ids += [q.submit(p, n) for p, n in jobs[7:]]
    got = q.run()
    assert max(q.batch_sizes) == max_batch if max_batch <= 7 else max(q.batch_sizes) >= 5
    compared = 0
    for jid, (prompt, n_new) in zip(ids, jobs):
        ref = oracle.Model(cfg)                      # a fresh cache per request
        for layer, tid, rows, cols, data in tensors:
            ref.load(layer, tid, data, rows, cols)
        want, gaps = checker_greedy(ref, cfg, prompt, n_new)
        ref.close()
        assert len(got[jid]) == n_new
        for i in range(n_new):                       # equal up to the first choice the checker itself calls close
            if gaps[i] <= MARGIN:
                break
            assert got[jid][i] == want[i], (jid, i, gaps[i])
            compared += 1
    assert compared >= 40, compared
    ctx.close()
