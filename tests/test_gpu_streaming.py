"""Layers streamed from pinned host memory (a model larger than what stays on the device): the results must be the
bits of a fully resident context, however many layers are resident, however many buffers there are, and however
the layer range is cut into windows; the copy statistics must account for every streamed layer."""
import numpy as np
import pytest

from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def _context(binding, cfg, seed, n_prefill, resident=None, slots=None):
    ctx = binding.Context(cfg)
    if resident is not None:
        ctx.set_option(binding.OPT_RESIDENT_LAYERS, resident)
    if slots is not None:
        ctx.set_option(binding.OPT_STREAM_SLOTS, slots)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg):
        ctx.load(layer, tid, data, rows, cols)
    for l in range(cfg["n_layers"]):
        if n_prefill:
            k, v = synth.kv_prefill(seed, l, n_prefill, cfg["n_kv_heads"], cfg["head_dim"])
            ctx.kv_load(l, 0, k, v)
    return ctx


def _decode(torch, ctx, cfg, h0, pos, steps, windows):
    """`steps` tokens, each through the given windows; returns the hidden states after every token."""
    out = []
    hin = torch.from_numpy(h0).cuda()
    hid = torch.empty_like(hin)
    for s in range(steps):
        src = hin
        for lb, le in windows:
            ctx.forward_window(lb, le, src, hid, pos + s, h0.shape[0] if s == 0 else h0.shape[0])
            src = hid
        ctx.sync()
        out.append(hid.cpu().numpy().copy())
    return out


@pytest.mark.parametrize("resident,slots,windows", [
    (0, 2, [(0, 4)]),                       # nothing resident, double buffering, one window
    (1, 2, [(0, 1), (1, 2), (2, 3), (3, 4)]),      # a budget of one layer per window
    (2, 3, [(0, 3), (3, 4)]),               # windows that cut through the streamed range
    (3, 2, [(0, 2), (2, 4)]),               # a single streamed layer: copied once, then it stays in its buffer
    (0, 4, [(0, 4)]),                       # as many buffers as layers: every layer is copied once
])
def test_streamed_layers_give_the_bits_of_a_resident_context(gpu, resident, slots, windows):
    torch, binding = gpu
    cfg = synth.model_config("small")
    seed, pos, steps = 71, 50, 3
    h0 = synth.activations(seed, 2, cfg["hidden"])
    full = _context(binding, cfg, seed, pos)
    want = _decode(torch, full, cfg, h0, pos, steps, [(0, cfg["n_layers"])])
    full.close()
    ctx = _context(binding, cfg, seed, pos, resident=resident, slots=slots)
    got = _decode(torch, ctx, cfg, h0, pos, steps, windows)
    for a, b in zip(got, want):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    copied, ms = ctx.stream_stats()
    layer_bytes = synth.weight_bytes(cfg, (synth.WQ, synth.WK, synth.WV, synth.WO, synth.W_GATE, synth.W_UP, synth.W_DOWN))
    n_streamed = cfg["n_layers"] - resident
    assert copied % layer_bytes == 0 and ms > 0
    n_copies = copied // layer_bytes
    if n_streamed <= slots and n_streamed <= 1 or slots >= n_streamed:
        assert n_copies == n_streamed                    # everything fits: one copy each
    else:
        assert n_streamed * steps <= n_copies <= n_streamed * (steps + 1)      # every use is a copy; the last prefetches go unused
    ctx.close()


def test_residency_options_are_checked(gpu):
    torch, binding = gpu
    cfg = synth.model_config("tiny")
    ctx = binding.Context(cfg)
    with pytest.raises(binding.PrimaError):
        ctx.set_option(binding.OPT_RESIDENT_LAYERS, cfg["n_layers"] + 1)
    with pytest.raises(binding.PrimaError):
        ctx.set_option(binding.OPT_STREAM_SLOTS, 1)
    ctx.set_option(binding.OPT_RESIDENT_LAYERS, 1)
    w = {}
    for layer, tid, rows, cols, data in synth.iter_model_tensors(3, cfg, with_globals=False):
        w[(layer, tid)] = (rows, cols, data)
    # a streamed layer must be completed before the next one is begun
    ctx.load(1, synth.WQ, w[(1, synth.WQ)][2], *w[(1, synth.WQ)][:2])
    with pytest.raises(binding.PrimaError) as e:
        ctx.load(2, synth.WQ, w[(2, synth.WQ)][2], *w[(2, synth.WQ)][:2])
    assert e.value.code == binding.ERR_STATE
    with pytest.raises(binding.PrimaError) as e:
        ctx.set_option(binding.OPT_RESIDENT_LAYERS, 2)          # too late: a matrix has been loaded
    assert e.value.code == binding.ERR_STATE
    h = torch.zeros((1, cfg["hidden"]), dtype=torch.float32, device="cuda")
    for (layer, tid), (rows, cols, data) in w.items():
        if layer == 1:
            ctx.load(layer, tid, data, rows, cols)
    with pytest.raises(binding.PrimaError):
        ctx.forward_window(0, 2, h, h, 0, 1)                    # layer 0 not loaded yet
    for (layer, tid), (rows, cols, data) in w.items():
        if layer != 1:
            ctx.load(layer, tid, data, rows, cols)
    ctx.forward_window(0, cfg["n_layers"], h, h, 0, 1)
    ctx.sync()
    ctx.close()


def test_70b_widths_half_the_layers_streamed_in_windows_of_two(gpu):
    """Llama-3-70B widths (481 MB per layer), 8 layers of which 4 stay resident, windows of 2 layers as in a ring of
    four devices, two tokens: the bits of a resident context, and 8 to 12 layer copies (4 per token + prefetches)."""
    torch, binding = gpu
    cfg = synth.model_config("70b", n_layers=8, vocab=1024)
    seed, pos, steps = 73, 4096, 2
    h0 = synth.activations(seed, 1, cfg["hidden"])
    windows = [(0, 2), (2, 4), (4, 6), (6, 8)]
    full = _context(binding, cfg, seed, pos)
    want = _decode(torch, full, cfg, h0, pos, steps, windows)
    full.close()
    ctx = _context(binding, cfg, seed, pos, resident=4, slots=2)
    got = _decode(torch, ctx, cfg, h0, pos, steps, windows)
    for a, b in zip(got, want):
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    copied, ms = ctx.stream_stats()
    layer_bytes = synth.weight_bytes(cfg, (synth.WQ, synth.WK, synth.WV, synth.WO, synth.W_GATE, synth.W_UP, synth.W_DOWN))
    assert 8 <= copied // layer_bytes <= 12
    print(f"streamed {copied / 1e9:.2f} GB at {copied / ms / 1e6:.1f} GB/s while copying")
    ctx.close()
