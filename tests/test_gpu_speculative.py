"""Speculative decoding (draft proposes, target verifies in one multi-token step) gives the target's own
greedy output; checked against the CPU checker's greedy decoding of the target."""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu

MARGIN = 4e-2      # twice the logit tolerance: below this top-2 gap the two sides may legitimately differ
N_PREFILL, N_NEW = 40, 30


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def _load(binding, cfg, seed, model=None):
    ctx = binding.Context(cfg)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg):
        ctx.load(layer, tid, data, rows, cols)
        if model is not None:
            model.load(layer, tid, data, rows, cols)
    return ctx


def _prefill(ctx, cfg, seed, model=None):
    for l in range(cfg["n_layers"]):
        k, v = synth.kv_prefill(seed, l, N_PREFILL, cfg["n_kv_heads"], cfg["head_dim"])
        ctx.kv_load(l, 0, k, v)
        if model is not None:
            model.kv_load(l, 0, k, v)


@pytest.fixture(scope="module")
def reference():
    """Greedy decoding of the target by the CPU checker: tokens and top-2 gaps."""
    cfg = synth.model_config("small")
    ref = oracle.Model(cfg)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(19, cfg):
        ref.load(layer, tid, data, rows, cols)
    for l in range(cfg["n_layers"]):
        k, v = synth.kv_prefill(19, l, N_PREFILL, cfg["n_kv_heads"], cfg["head_dim"])
        ref.kv_load(l, 0, k, v)
    tok, toks, margins = 0, [], []
    for step in range(N_NEW):
        h = ref.forward_window(0, cfg["n_layers"], ref.embed([tok]), N_PREFILL + step)
        tok, margin = oracle.argmax(ref.logits(h)[0])
        toks.append(int(tok))
        margins.append(float(margin))
    ref.close()
    return toks, margins


def _agreeing_prefix(margins):
    """Number of leading steps whose choice is unambiguous."""
    n = 0
    while n < len(margins) and margins[n] > MARGIN:
        n += 1
    return n


@pytest.mark.parametrize("draft_kind", ["same_model", "other_model", "every_third_wrong", "split_windows"])
def test_speculative_output_is_the_targets_greedy_output(gpu, reference, draft_kind):
    torch, binding = gpu
    from paper_2504_08791_b200.speculative import SpeculativeDecoder
    want, margins = reference
    n_sure = _agreeing_prefix(margins)
    assert n_sure >= 8, "the reference run has an ambiguous choice too early to test anything"
    cfg = synth.model_config("small")
    target = _load(binding, cfg, 19)
    _prefill(target, cfg, 19)
    draft_seed = 23 if draft_kind == "other_model" else 19
    draft = _load(binding, cfg, draft_seed)
    _prefill(draft, cfg, 19)            # same context positions; the draft's own K/V values do not matter for the property
    counter = [0]

    def spoil(tokens):
        out = list(tokens)
        for i in range(len(out)):
            counter[0] += 1
            if counter[0] % 3 == 0:
                out[i] = (out[i] + 1) % cfg["vocab"]
        return out

    dec = SpeculativeDecoder(target, draft, n_draft=4,
                             target_windows=[0, 1, 3, 4] if draft_kind == "split_windows" else None,
                             draft_filter=spoil if draft_kind == "every_third_wrong" else None)
    got, stats = dec.generate(first_token=0, pos=N_PREFILL, n_new=N_NEW)
    assert len(got) == N_NEW
    assert got[:n_sure] == want[:n_sure], f"{draft_kind}: first difference at {[a == b for a, b in zip(got, want)].index(False)}"
    assert sum(stats.per_cycle) >= N_NEW and all(1 <= n <= 5 for n in stats.per_cycle)
    if draft_kind in ("same_model", "split_windows") and n_sure == N_NEW:
        assert stats.acceptance > 0.7          # the draft is the target: nearly everything is confirmed
    if draft_kind == "other_model":
        assert stats.acceptance < 0.3          # an unrelated random model agrees almost never
    if draft_kind == "every_third_wrong":
        assert 0.0 < stats.acceptance < 1.0
    target.close()
    draft.close()
