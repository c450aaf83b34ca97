"""GPU parity of layer windows, logits and greedy decoding against the CPU checker, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2          # absolute, on the final logits
HIDDEN_TOL = 2e-3         # of the vector's RMS, per element, after a window
MARGIN = 2 * LOGIT_TOL    # greedy tokens must agree wherever the checker's top-2 gap exceeds this


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


class Pair:
    """The same synthetic model loaded into the checker and into a GPU context."""

    def __init__(self, gpu, cfg, seed, n_prefill, layers=None, with_globals=True):
        self.torch, self.binding = gpu
        self.cfg, self.seed = cfg, seed
        self.ref = oracle.Model(cfg)
        self.ctx = self.binding.Context(cfg)
        for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg, layers=layers, with_globals=with_globals):
            self.ref.load(layer, tid, data, rows, cols)
            self.ctx.load(layer, tid, data, rows, cols)
        for l in (range(cfg["n_layers"]) if layers is None else layers):
            if n_prefill:
                k, v = synth.kv_prefill(seed, l, n_prefill, cfg["n_kv_heads"], cfg["head_dim"])
                self.ref.kv_load(l, 0, k, v)
                self.ctx.kv_load(l, 0, k, v)

    def gpu_window(self, lb, le, h, pos):
        t = self.torch
        n_tok = h.shape[0]
        hin = t.from_numpy(np.ascontiguousarray(h, np.float32)).cuda()
        hout = t.empty_like(hin)
        self.ctx.forward_window(lb, le, hin, hout, pos, n_tok)
        self.ctx.sync()
        return hout.cpu().numpy()

    def gpu_logits(self, h):
        t = self.torch
        hin = t.from_numpy(np.ascontiguousarray(h, np.float32)).cuda()
        out = t.empty((h.shape[0], self.cfg["vocab"]), dtype=t.float32, device="cuda")
        self.ctx.logits(hin, h.shape[0], out)
        self.ctx.sync()
        return out.cpu().numpy()

    def close(self):
        self.ctx.close()
        self.ref.close()


def _hidden_close(got, want, tol=HIDDEN_TOL):
    rms = np.sqrt(np.mean(want.astype(np.float64) ** 2, axis=-1, keepdims=True))
    err = np.abs(got.astype(np.float64) - want) / rms
    assert err.max() <= tol, f"hidden differs by {err.max():.2e} of its RMS (allowed {tol:.0e})"
    return float(err.max())


@pytest.mark.parametrize("name,pos,n_tok", [("tiny", 0, 1), ("tiny", 37, 1), ("tiny", 63, 2), ("small", 130, 1), ("small", 255, 5),
                                            ("small", 64, 8), ("small", 0, 3)])
def test_full_depth_window_matches_checker(gpu, name, pos, n_tok):
    cfg = synth.model_config(name)
    p = Pair(gpu, cfg, seed=11, n_prefill=pos)
    h0 = synth.activations(11, n_tok, cfg["hidden"])
    want = p.ref.forward_window(0, cfg["n_layers"], h0, pos)
    got = p.gpu_window(0, cfg["n_layers"], h0, pos)
    _hidden_close(got, want)
    # appended cache entries: binary16 roundings of nearly equal numbers, at most a few ulps apart
    for l in range(cfg["n_layers"]):
        kr, vr = p.ref.kv_read(l, pos, n_tok)
        kg, vg = p.ctx.kv_read(l, pos, n_tok)
        for a, b in ((kr, kg), (vr, vg)):
            fa, fb = a.view(np.float16).astype(np.float64), b.view(np.float16).astype(np.float64)
            assert np.abs(fa - fb).max() <= 4e-3 * max(1.0, np.abs(fa).max())
        if pos:
            # prefilled entries are untouched
            k0, v0 = synth.kv_prefill(11, l, pos, cfg["n_kv_heads"], cfg["head_dim"])
            kg, vg = p.ctx.kv_read(l, 0, pos)
            assert np.array_equal(kg, k0) and np.array_equal(vg, v0)
    logits_ref = p.ref.logits(want)
    logits_gpu = p.gpu_logits(got)
    assert np.abs(logits_gpu.astype(np.float64) - logits_ref).max() <= LOGIT_TOL
    p.close()


@pytest.mark.parametrize("splits", [[(0, 1), (1, 2), (2, 3), (3, 4)], [(0, 2), (2, 4)], [(0, 1), (1, 4)], [(0, 3), (3, 4)]])
@pytest.mark.parametrize("n_tok", [1, 5])
def test_window_splits_are_bit_identical_on_the_gpu(gpu, splits, n_tok):
    cfg = synth.model_config("small")
    pos = 100
    h0 = synth.activations(13, n_tok, cfg["hidden"])
    full = Pair(gpu, cfg, seed=13, n_prefill=pos, with_globals=False)
    want = full.gpu_window(0, cfg["n_layers"], h0, pos)
    part = Pair(gpu, cfg, seed=13, n_prefill=pos, with_globals=False)
    h = h0
    for lb, le in splits:
        h = part.gpu_window(lb, le, h, pos)
    assert np.array_equal(h.view(np.uint32), want.view(np.uint32))
    for l in range(cfg["n_layers"]):
        for a, b in zip(full.ctx.kv_read(l, 0, pos + n_tok), part.ctx.kv_read(l, 0, pos + n_tok)):
            assert np.array_equal(a, b)
    full.close()
    part.close()


@pytest.mark.parametrize("over,pos,n_tok", [
    (dict(rope_mode=1), 70, 1),                                             # interleaved rotation pairs
    (dict(rope_mode=1), 129, 6),                                            # ... on the multi-token kernels
    (dict(n_q_heads=2, n_kv_heads=2, hidden=256), 33, 1),                   # no grouping, one super-block column
    (dict(n_q_heads=8, n_kv_heads=1, hidden=1024), 200, 3),                 # one KV head for eight query heads
    (dict(n_q_heads=8, n_kv_heads=1, hidden=1024), 250, 8),                 # ... 64 query rows: four tiles in one CTA
    (dict(n_q_heads=8, n_kv_heads=1, hidden=1024), 256, 4),                 # the step's positions open a new chunk
    (dict(n_q_heads=10, n_kv_heads=2, hidden=1280, ffn=1280), 127, 1),      # five query heads per KV head, column groups of 5
    (dict(n_q_heads=10, n_kv_heads=2, hidden=1280, ffn=1280), 128, 7),
    (dict(n_q_heads=4, n_kv_heads=4, hidden=512, ffn=3328, vocab=1000), 0, 2),   # 13 super-block columns (prime), vocab not a multiple of 8
])
def test_unusual_shapes_match_checker(gpu, over, pos, n_tok):
    cfg = synth.model_config("small", **over)
    p = Pair(gpu, cfg, seed=37, n_prefill=pos)
    h0 = synth.activations(37, n_tok, cfg["hidden"])
    want = p.ref.forward_window(0, cfg["n_layers"], h0, pos)
    got = p.gpu_window(0, cfg["n_layers"], h0, pos)
    _hidden_close(got, want)
    assert np.abs(p.gpu_logits(got).astype(np.float64) - p.ref.logits(want)).max() <= LOGIT_TOL
    p.close()


@pytest.mark.parametrize("sizes", [[1, 2], [2, 1], [1, 1, 1]])
def test_ring_schedule_with_uneven_windows_is_bit_identical_to_one_pass(gpu, sizes):
    """The paper's ring schedule (devices take w_m layers per turn, several rounds) executed window by
    window gives the bits of a single full-depth pass."""
    from paper_2504_08791_b200 import schedule
    torch, binding = gpu
    cfg = synth.model_config("small")
    L = cfg["n_layers"]
    p = Pair(gpu, cfg, seed=29, n_prefill=50)
    h0 = synth.activations(29, 2, cfg["hidden"])
    one = p.gpu_window(0, L, h0, 50)
    ws = schedule.windows(L, sizes)
    assert schedule.rounds(L, sizes) >= 2
    hin = torch.from_numpy(h0).cuda()
    hout = torch.empty_like(hin)
    schedule.run_schedule(p.ctx, ws, hin, hout, 50, 2)
    p.ctx.sync()
    assert np.array_equal(hout.cpu().numpy().view(np.uint32), one.view(np.uint32))
    p.close()


def test_five_token_step_agrees_with_five_single_steps_on_the_gpu(gpu):
    cfg = synth.model_config("small")
    pos = 77
    h0 = synth.activations(17, 5, cfg["hidden"])
    a = Pair(gpu, cfg, seed=17, n_prefill=pos, with_globals=False)
    batch = a.gpu_window(0, cfg["n_layers"], h0, pos)
    single = np.concatenate([a.gpu_window(0, cfg["n_layers"], h0[t:t + 1], pos + t) for t in range(5)])
    _hidden_close(batch, single)
    a.close()


def test_llama8b_shaped_layer_with_1024_cached_positions(gpu):
    cfg = synth.model_config("8b", n_layers=1, vocab=1024)
    pos = 1024
    p = Pair(gpu, cfg, seed=1, n_prefill=pos, with_globals=False)
    h0 = synth.activations(1, 1, cfg["hidden"])
    want = p.ref.forward_window(0, 1, h0, pos)
    got = p.gpu_window(0, 1, h0, pos)
    _hidden_close(got, want)
    p.close()


def test_greedy_decode_64_tokens_matches_checker(gpu):
    torch, binding = gpu
    cfg = synth.model_config("small")
    n_prefill, steps = 40, 64
    p = Pair(gpu, cfg, seed=19, n_prefill=n_prefill)
    hid = torch.empty((1, cfg["hidden"]), dtype=torch.float32, device="cuda")
    logits = torch.empty((1, cfg["vocab"]), dtype=torch.float32, device="cuda")
    tok = 0
    low_margin = 0
    for step in range(steps):
        pos = n_prefill + step
        # checker
        h_ref = p.ref.forward_window(0, cfg["n_layers"], p.ref.embed([tok]), pos)
        l_ref = p.ref.logits(h_ref)[0]
        want_tok, margin = oracle.argmax(l_ref)
        # GPU, all through the ABI
        p.ctx.embed([tok], hid)
        p.ctx.forward_window(0, cfg["n_layers"], hid, hid, pos, 1)
        p.ctx.logits(hid, 1, logits)
        got_tok = int(p.ctx.argmax(logits, 1)[0])
        l_gpu = logits.cpu().numpy()[0]
        assert np.abs(l_gpu.astype(np.float64) - l_ref).max() <= LOGIT_TOL, f"step {step}"
        assert got_tok == int(np.argmax(l_gpu))           # the device argmax is the argmax of the device logits
        if margin > MARGIN:
            assert got_tok == want_tok, f"step {step}: margin {margin}"
        else:
            low_margin += 1
        tok = want_tok                                    # both sides continue from the checker's token
    assert low_margin <= 8, f"{low_margin} of {steps} steps had a top-2 gap below {MARGIN}"
    p.close()


def test_errors_leave_the_context_usable(gpu):
    torch, binding = gpu
    cfg = synth.model_config("tiny")
    ctx = binding.Context(cfg)
    h = torch.zeros((1, cfg["hidden"]), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PrimaError) as e:
        ctx.forward_window(0, 1, h, h, 0, 1)              # nothing loaded yet
    assert e.value.code == binding.ERR_STATE
    for layer, tid, rows, cols, data in synth.iter_model_tensors(3, cfg, layers=[0], with_globals=False):
        ctx.load(layer, tid, data, rows, cols)
    for bad in [dict(lb=0, le=2, pos=0, n=1), dict(lb=0, le=1, pos=cfg["kv_capacity"], n=1), dict(lb=0, le=1, pos=0, n=9),
                dict(lb=1, le=0, pos=0, n=1), dict(lb=0, le=1, pos=-1, n=1)]:
        with pytest.raises(binding.PrimaError):
            ctx.forward_window(bad["lb"], bad["le"], h, h, bad["pos"], bad["n"])
    w = synth.model_tensor(3, 0, synth.WQ, 512, 512)
    with pytest.raises(binding.PrimaError):
        ctx.load(0, synth.WQ, w, 512, 256)                # wrong shape
    with pytest.raises(binding.PrimaError):
        ctx.load(5, synth.WQ, w, 512, 512)                # layer out of range
    with pytest.raises(binding.PrimaError):
        ctx.load(0, 99, w, 512, 512)
    ctx.forward_window(0, 1, h, h, 0, 1)                  # still works
    ctx.sync()
    assert ctx.launch_count() > 0
    ctx.close()


def test_sums_outside_the_accumulator_range_are_reported_once(gpu):
    torch, binding = gpu
    cfg = synth.model_config("tiny")
    p = Pair(gpu, cfg, seed=41, n_prefill=10)
    h0 = synth.activations(41, 1, cfg["hidden"])
    good = p.gpu_window(0, cfg["n_layers"], h0, 10)
    hin = torch.from_numpy(h0 * 1e12).cuda()            # products of the first projection far beyond 2^27
    hout = torch.empty_like(hin)
    p.ctx.forward_window(0, cfg["n_layers"], hin, hout, 10, 1)
    with pytest.raises(binding.PrimaError) as err:
        p.ctx.sync()
    assert err.value.code == binding.ERR_DEVICE
    p.ctx.sync()                                        # reported once
    again = p.gpu_window(0, cfg["n_layers"], h0, 10)    # and the context computes the same bits as before
    assert np.array_equal(again.view(np.uint32), good.view(np.uint32))
    p.close()


@pytest.mark.parametrize("n_tok,pos,over", [
    (1, 39000, {}),                                                  # streaming kernel, 305 chunks on 74 CTAs per KV head
    (3, 19100, dict(n_kv_heads=1)),                                  # ... 150 chunks on 148 CTAs: more partial results than the merge has threads
    (1, 9500, dict(n_q_heads=8, n_kv_heads=8, hidden=1024)),         # one-token kernel, 75 chunks on 37 CTAs per KV head: two or three per CTA
])
def test_long_context_with_more_chunks_than_resident_ctas(gpu, n_tok, pos, over):
    """More chunks of cached positions than CTAs per KV head, so that a CTA takes further chunks and carries its
    running state from one to the next, in both attention kernels, and a merge over more partial results than it has
    threads."""
    cfg = synth.model_config("tiny", kv_capacity=40000, **over)
    p = Pair(gpu, cfg, seed=43, n_prefill=pos)
    h0 = synth.activations(43, n_tok, cfg["hidden"])
    want = p.ref.forward_window(0, cfg["n_layers"], h0, pos)
    got = p.gpu_window(0, cfg["n_layers"], h0, pos)
    _hidden_close(got, want)
    p.close()


@pytest.mark.parametrize("n_tok", [1, 6])
def test_a_wait_that_gives_up_is_reported_once_and_the_next_step_is_clean(gpu, n_tok):
    """The bounded waits of the streaming kernels: with the poll limit of every warp's first wait set to 0 the wait
    runs out at once; the kernels must still wait (with the ordinary limit) for every copy they requested, return
    normally and raise the status word.  prima_sync reports it once and clears the accumulators, after which the
    context gives exactly the bits of a context that never failed."""
    torch, binding = gpu
    cfg = synth.model_config("small")
    pos = 90
    h0 = synth.activations(47, n_tok, cfg["hidden"])
    p = Pair(gpu, cfg, seed=47, n_prefill=pos)
    good = p.gpu_window(0, cfg["n_layers"], h0, pos)
    good_logits = p.gpu_logits(good)
    p.ctx.set_option(binding.OPT_FIRST_WAIT_POLLS, 0)
    hin = torch.from_numpy(h0).cuda()
    hout = torch.empty_like(hin)
    p.ctx.forward_window(0, cfg["n_layers"], hin, hout, pos, n_tok)
    with pytest.raises(binding.PrimaError) as err:
        p.ctx.sync()
    assert err.value.code == binding.ERR_DEVICE and "wait" in str(err.value)
    p.ctx.sync()                                         # reported once
    p.ctx.set_option(binding.OPT_FIRST_WAIT_POLLS, -1)   # the ordinary limit again
    again = p.gpu_window(0, cfg["n_layers"], h0, pos)
    assert np.array_equal(again.view(np.uint32), good.view(np.uint32))
    assert np.array_equal(p.gpu_logits(again).view(np.uint32), good_logits.view(np.uint32))
    with pytest.raises(binding.PrimaError):
        p.ctx.set_option(99, 0)
    p.close()


def test_weights_asked_into_l2_ahead_of_time_change_no_bit(gpu):
    """The requests that bring the head of the gate/up matrix into L2 while attention and the O product run are
    hints: switched off, at their defaults, larger than the matrix or cut at odd places, the step gives the same bits."""
    torch, binding = gpu
    cfg = synth.model_config("small")
    pos = 77
    h0 = synth.activations(61, 1, cfg["hidden"])
    p = Pair(gpu, cfg, seed=61, n_prefill=pos, with_globals=False)
    base = p.gpu_window(0, cfg["n_layers"], h0, pos)
    for ahead, ahead_o in ((0, 0), (16, 0), (0, 1 << 30), (1 << 30, 1 << 30), (16 * 1000 + 16, 48), (-1, -1)):
        p.ctx.set_option(binding.OPT_L2_AHEAD_BYTES, ahead)
        p.ctx.set_option(binding.OPT_L2_AHEAD_O_BYTES, ahead_o)
        again = p.gpu_window(0, cfg["n_layers"], h0, pos)      # same position again: the cache entry is rewritten with the same bits
        assert np.array_equal(again.view(np.uint32), base.view(np.uint32)), (ahead, ahead_o)
    for bad in (-2, 24, (1 << 30) + 16):
        with pytest.raises(binding.PrimaError):
            p.ctx.set_option(binding.OPT_L2_AHEAD_BYTES, bad)
    p.close()


@pytest.mark.parametrize("after", [2, 5, 9])
def test_a_launch_refused_in_mid_window_leaves_the_next_call_clean(gpu, after):
    """A launch in the middle of a window fails (injected on the host: the library is told to refuse it, nothing
    faulty reaches the GPU).  The call returns an error; the call after it gives the bits of an undisturbed context."""
    torch, binding = gpu
    cfg = synth.model_config("small")
    pos, n_tok = 60, 2
    h0 = synth.activations(53, n_tok, cfg["hidden"])
    p = Pair(gpu, cfg, seed=53, n_prefill=pos, with_globals=False)
    good = p.gpu_window(0, cfg["n_layers"], h0, pos)
    hin = torch.from_numpy(h0).cuda()
    hout = torch.empty_like(hin)
    p.ctx.set_option(binding.OPT_FAIL_AFTER_LAUNCHES, after)
    with pytest.raises(binding.PrimaError) as err:
        p.ctx.forward_window(0, cfg["n_layers"], hin, hout, pos, n_tok)
    assert err.value.code == binding.ERR_CUDA and "injected" in str(err.value)
    p.ctx.sync()
    again = p.gpu_window(0, cfg["n_layers"], h0, pos)
    assert np.array_equal(again.view(np.uint32), good.view(np.uint32))
    p.close()


def test_merge_inside_the_attention_kernel_matches_checker():
    """PRIMA_ATTN_MERGE=fused (read once per process, hence the child process): the last CTA of a KV head merges."""
    import os
    import subprocess
    import sys
    code = (
        "import numpy as np, torch, oracle\n"
        "from paper_2504_08791_b200 import binding, synth\n"
        "from tests.test_gpu_model import Pair, _hidden_close\n"
        "for name, pos in (('tiny', 0), ('small', 300), ('tiny', 5000)):\n"
        "    cfg = synth.model_config(name, kv_capacity=5100)\n"
        "    p = Pair((torch, binding), cfg, seed=59, n_prefill=pos)\n"
        "    h0 = synth.activations(59, 1, cfg['hidden'])\n"
        "    want = p.ref.forward_window(0, cfg['n_layers'], h0, pos)\n"
        "    a = p.gpu_window(0, cfg['n_layers'], h0, pos)\n"
        "    b = p.gpu_window(0, cfg['n_layers'], h0, pos)\n"
        "    _hidden_close(a, want)\n"
        "    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))\n"
        "    p.close()\n"
        "print('fused merge ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PRIMA_ATTN_MERGE="fused", PYTHONPATH=root)
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "fused merge ok" in out.stdout, out.stdout + out.stderr


def test_range_checked_build_gives_the_same_bits_and_raises_nothing(gpu):
    """The library built with -DPRIMA_BOUNDS (every weight request, accumulator index, cache append and partial-result
    slot checked against its array; a violation would raise bit 2 of the status word and skip the access) runs the
    same steps in a child process: no status is raised (prima_sync succeeds) and the hidden states and logits have the
    bits of the ordinary build.  Shapes with ragged tails, several tokens, several requests, a long context."""
    import os
    import subprocess
    import sys
    import tempfile
    torch, binding = gpu
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if not os.path.exists(os.path.join(root, "paper_2504_08791_b200", "libprima_bounds.so")):
        from paper_2504_08791_b200 import build as _build
        _build.build(bounds=True)
    code = (
        "import sys, numpy as np, torch\n"
        "from paper_2504_08791_b200 import binding, synth\n"
        "out = {}\n"
        "cases = [('tiny', {}, 37, 1), ('small', {}, 255, 5), ('small', dict(n_q_heads=10, n_kv_heads=2, hidden=1280, ffn=1280), 128, 7),\n"
        "         ('small', dict(n_q_heads=4, n_kv_heads=4, hidden=512, ffn=3328, vocab=1000), 0, 2), ('tiny', dict(kv_capacity=12000), 11000, 1)]\n"
        "for i, (name, over, pos, n_tok) in enumerate(cases):\n"
        "    cfg = synth.model_config(name, max_n_tok=16, **over)\n"
        "    ctx = binding.Context(cfg)\n"
        "    for layer, tid, rows, cols, data in synth.iter_model_tensors(71, cfg):\n"
        "        ctx.load(layer, tid, data, rows, cols)\n"
        "    for l in range(cfg['n_layers']):\n"
        "        if pos:\n"
        "            k, v = synth.kv_prefill(71, l, pos, cfg['n_kv_heads'], cfg['head_dim'])\n"
        "            ctx.kv_load(l, 0, k, v)\n"
        "            ctx.kv_load(l, 0, k[:min(pos, 90)], v[:min(pos, 90)], seq=3)\n"
        "    h = torch.from_numpy(synth.activations(71, n_tok, cfg['hidden'])).cuda()\n"
        "    o = torch.empty_like(h)\n"
        "    ctx.forward_window(0, cfg['n_layers'], h, o, pos, n_tok)\n"
        "    lg = torch.empty((n_tok, cfg['vocab']), dtype=torch.float32, device='cuda')\n"
        "    ctx.logits(o, n_tok, lg)\n"
        "    ctx.sync()\n"
        "    out['h%d' % i] = o.cpu().numpy(); out['l%d' % i] = lg.cpu().numpy()\n"
        "    if pos:\n"
        "        h2 = torch.from_numpy(synth.activations(72, 2, cfg['hidden'])).cuda()\n"
        "        o2 = torch.empty_like(h2)\n"
        "        ctx.forward_window_seqs(0, cfg['n_layers'], h2, o2, [0, 3], [pos, min(pos, 90)])\n"
        "        ctx.sync()\n"
        "        out['s%d' % i] = o2.cpu().numpy()\n"
        "    ctx.close()\n"
        "np.savez(sys.argv[1], **out)\n"
        "print('steps ok')\n")
    got = {}
    with tempfile.TemporaryDirectory() as tmp:
        for which in ("plain", "bounds"):
            env = dict(os.environ, PYTHONPATH=root)
            env.pop("PRIMA_LIB", None)
            if which == "bounds":
                env["PRIMA_LIB"] = "bounds"
            path = os.path.join(tmp, which + ".npz")
            run = subprocess.run([sys.executable, "-c", code, path], cwd=root, env=env, capture_output=True, text=True, timeout=900)
            assert run.returncode == 0 and "steps ok" in run.stdout, which + ": " + run.stdout + run.stderr
            with np.load(path) as z:
                got[which] = {k: z[k] for k in z.files}
    assert sorted(got["plain"]) == sorted(got["bounds"]) and len(got["plain"]) >= 14
    for k, a in got["plain"].items():
        assert np.isfinite(a).all(), k
        assert np.array_equal(a.view(np.uint32), got["bounds"][k].view(np.uint32)), k
