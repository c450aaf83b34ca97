"""Q6_K, Q8_0 and FP16 matrices on the GPU against the CPU checker: dequantisation bit for bit, the product row by
row within 1e-3 * sum |w x|, through the C ABI."""
import numpy as np
import pytest

import oracle.kquants as kq
from paper_2504_08791_b200 import synth
from tests.golden._read import kquants_blocks

pytestmark = pytest.mark.gpu

ROW_TOL = 1e-3
ORC = {synth.FMT_Q6_K: kq.Q6_K, synth.FMT_Q8_0: kq.Q8_0, synth.FMT_F16: kq.F16}


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def _dequant_gpu(gpu, fmt, blocks):
    torch, binding = gpu
    blocks = np.ascontiguousarray(blocks, np.uint8).reshape(-1)
    n = blocks.size // synth.FMT_BLOCK_BYTES[fmt]
    out = torch.full((n * synth.FMT_BLOCK_WEIGHTS[fmt],), float("nan"), dtype=torch.float32, device="cuda")
    binding.prima_dequant_fmt(fmt, torch.from_numpy(blocks).cuda(), n, out)
    return out.cpu().numpy()


@pytest.mark.parametrize("fmt", [synth.FMT_Q6_K, synth.FMT_Q8_0, synth.FMT_F16])
def test_dequant_is_bit_exact(gpu, fmt):
    rng = np.random.default_rng(fmt)
    n = 777
    blocks = rng.integers(0, 256, (n, synth.FMT_BLOCK_BYTES[fmt]), dtype=np.uint8)
    d_hi = {synth.FMT_Q6_K: 209, synth.FMT_Q8_0: 1, synth.FMT_F16: 1}[fmt]
    blocks[:, d_hi] &= 0xBF                                   # finite scales
    blocks[:50, d_hi] = 0                                     # some subnormal scales
    want = kq.dequant(ORC[fmt], blocks, np.float32)
    got = _dequant_gpu(gpu, fmt, blocks)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(want.astype(np.float64), kq.dequant(ORC[fmt], blocks))      # and the fp32 value is the exact one


def test_handbuilt_blocks_on_the_gpu(gpu):
    for name, b in kquants_blocks().items():
        fmt = synth.FMT_Q6_K if b["fmt"] == "q6_k" else synth.FMT_Q8_0
        got = _dequant_gpu(gpu, fmt, b["bytes"])
        for k, v in b["w"].items():
            assert float(got[k]) == v, (name, k)


@pytest.mark.parametrize("fmt,rows,cols,n_cols", [
    (synth.FMT_Q6_K, 1000, 2048, 1), (synth.FMT_Q6_K, 37, 5120, 3), (synth.FMT_Q6_K, 301, 1280, 4), (synth.FMT_Q6_K, 520, 28672, 1),
    (synth.FMT_Q8_0, 1000, 2048, 1), (synth.FMT_Q8_0, 37, 5120, 4), (synth.FMT_Q8_0, 9, 256, 2), (synth.FMT_Q8_0, 260, 28672, 1),
    (synth.FMT_F16, 513, 4096, 2), (synth.FMT_F16, 3, 256, 1),
])
def test_gemv_rows_within_the_bound(gpu, fmt, rows, cols, n_cols):
    torch, binding = gpu
    w = synth.fmt_tensor(11, fmt, rows, cols)
    x = synth.activations(11, n_cols, cols)
    want, s_abs = kq.gemv(ORC[fmt], w, rows, cols, x)
    # the matrix deliberately starts at an odd multiple of 2 bytes inside a larger buffer: rows need not be 16-byte aligned
    pad = 2 * 7
    buf = torch.zeros(w.size + 64, dtype=torch.uint8, device="cuda")
    buf[pad:pad + w.size] = torch.from_numpy(w).cuda()
    y = torch.full((n_cols, rows), float("nan"), dtype=torch.float32, device="cuda")
    binding.prima_gemv_fmt(fmt, buf[pad:pad + w.size], rows, cols, torch.from_numpy(x).cuda(), n_cols, y)
    torch.cuda.synchronize()
    got = y.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= ROW_TOL * s_abs + 1e-30)
    y2 = torch.empty_like(y)
    binding.prima_gemv_fmt(fmt, buf[pad:pad + w.size], rows, cols, torch.from_numpy(x).cuda(), n_cols, y2)
    torch.cuda.synchronize()
    assert np.array_equal(y2.cpu().numpy().view(np.uint32), y.cpu().numpy().view(np.uint32))      # run to run


def test_formats_reject_bad_arguments(gpu):
    torch, binding = gpu
    w = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    x = torch.zeros(4096, dtype=torch.float32, device="cuda")
    y = torch.zeros(64, dtype=torch.float32, device="cuda")
    for args in [(9, w, 1, 256, x, 1, y), (synth.FMT_Q6_K, w, 1, 200, x, 1, y), (synth.FMT_Q8_0, w, 1, 256, x, 5, y),
                 (synth.FMT_Q8_0, w, 1, 65536, x, 1, y)]:
        with pytest.raises(binding.PrimaError):
            binding.prima_gemv_fmt(*args)
    assert binding.lib().prima_fmt_block_bytes(synth.FMT_Q6_K) == 210 and binding.lib().prima_fmt_block_weights(synth.FMT_Q8_0) == 32
