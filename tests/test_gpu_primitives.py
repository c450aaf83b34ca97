"""GPU parity of the two primitives against the CPU checker: bit-exact Q4_K unpacking and the
per-row bound |y - y_ref| <= 1e-3 * sum_k |w_k x_k| of every projection shape."""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth
from tests.golden._read import handbuilt_blocks

pytestmark = pytest.mark.gpu

ROW_TOL = 1e-3      # of sum |w x| per row


@pytest.fixture(scope="module")
def gpu():
    import torch
    from paper_2504_08791_b200 import binding
    assert torch.cuda.is_available()
    binding.lib()
    return torch, binding


def _to_dev(torch, a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _dequant_gpu(gpu, blocks):
    torch, binding = gpu
    blocks = np.ascontiguousarray(blocks, np.uint8).reshape(-1)
    n_sb = blocks.size // 144
    out = torch.empty(n_sb * 256, dtype=torch.float32, device="cuda")
    binding.prima_dequant_q4k(_to_dev(torch, blocks), n_sb, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def test_dequant_bit_exact_on_handbuilt_and_edge_blocks(gpu):
    hb = handbuilt_blocks()
    edge = [hb["A"]["bytes"], hb["B"]["bytes"]]
    # zero scales, largest finite halves, subnormal scales with all field values at their extremes
    for d_bits, dmin_bits in [(0, 0), (0x7BFF, 0x7BFF), (0x0001, 0x0001), (0x03FF, 0x0400), (0x8001, 0x83FF)]:
        for q in (0, 15):
            edge.append(synth.build_blocks([d_bits], [dmin_bits], [63, 0, 1, 32, 31, 16, 47, 63], [0, 63, 32, 1, 16, 31, 63, 47],
                                           np.full(256, q, np.uint8))[0])
    blocks = np.stack(edge)
    got = _dequant_gpu(gpu, blocks)
    want = oracle.q4k_dequant(blocks, np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_dequant_bit_exact_on_random_blocks(gpu):
    w, _ = synth.gemv_case(seed=0, rows=512, cols=2048)
    got = _dequant_gpu(gpu, w)
    want = oracle.q4k_dequant(w, np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    wm = synth.model_tensor(3, 0, synth.W_DOWN, 64, 28672)      # includes subnormal d
    got = _dequant_gpu(gpu, wm)
    want = oracle.q4k_dequant(wm, np.float32)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert _dequant_gpu(gpu, np.zeros(0, np.uint8)).size == 0


def _gemv_gpu(gpu, w, rows, cols, x):
    torch, binding = gpu
    n_cols = x.shape[0]
    y = torch.full((n_cols, rows), float("nan"), dtype=torch.float32, device="cuda")
    binding.prima_gemv_q4k(_to_dev(torch, w), rows, cols, _to_dev(torch, x), n_cols, y)
    return y.cpu().numpy()


def _check_rows(got, want, s_abs, tol=ROW_TOL):
    err = np.abs(got.astype(np.float64) - want)
    bound = tol * s_abs
    worst = float((err / np.maximum(bound, 1e-300)).max())
    assert np.all(err <= bound), f"worst row error is {worst:.3f} of the bound"
    return worst


@pytest.mark.parametrize("rows,cols,n_cols", [
    (4096, 4096, 1),      # the single-GEMV workload
    (8, 256, 1), (1, 256, 1), (13, 768, 1), (100, 512, 3), (4096, 4096, 2), (1000, 1024, 5), (264, 1280, 8),
    (1000, 2048, 9), (264, 1280, 13), (520, 4096, 16), (9, 256, 16),      # two column blocks of eight
])
def test_gemv_literal_distribution(gpu, rows, cols, n_cols):
    w, x = synth.gemv_case(seed=0, rows=rows, cols=cols, n_cols=n_cols)
    want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
    got = _gemv_gpu(gpu, w, rows, cols, x)
    _check_rows(got, want, s_abs)


@pytest.mark.parametrize("name,tid", [("8b", synth.WQ), ("8b", synth.W_DOWN), ("32b", synth.WK), ("32b", synth.W_DOWN),
                                      ("70b", synth.WO), ("70b", synth.W_DOWN), ("70b", synth.W_UP)])
def test_gemv_projection_shapes_zero_mean_weights(gpu, name, tid):
    cfg = synth.model_config(name)
    rows, cols = synth.tensor_shape(cfg, tid)
    rows = min(rows, 2048)                      # full width, a slice of the rows: the CPU side stays in seconds
    w = synth.model_tensor(5, 0, tid, rows, cols)
    x = synth.activations(5, 1, cols)
    want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
    got = _gemv_gpu(gpu, w, rows, cols, x)
    _check_rows(got, want, s_abs)


def test_gemv_activation_scales_and_special_vectors(gpu):
    rows, cols = 256, 1024
    w = synth.model_tensor(6, 0, synth.WQ, rows, cols)
    base = synth.activations(6, 1, cols)
    for x in (base * 1e-6, base * 3e4, np.ones_like(base), np.zeros_like(base), np.abs(base) * 50.0):
        want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
        got = _gemv_gpu(gpu, w, rows, cols, x)
        if not x.any():
            assert not got.any()
        else:
            _check_rows(got, want, s_abs)
    # one large outlier next to small values
    x = base.copy()
    x[0, 17] = 900.0
    want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
    _check_rows(_gemv_gpu(gpu, w, rows, cols, x), want, s_abs)


@pytest.mark.parametrize("n", [6, 11])
def test_gemv_several_tokens_with_outliers_and_mixed_scales(gpu, n):
    # 4..16 columns go through the kernel that quantises a column's 256 activations with one step
    rows, cols = 264, 2048
    w = synth.model_tensor(8, 0, synth.WQ, rows, cols)
    x = synth.activations(8, n, cols)
    x[1] *= 1e-4
    x[2] *= 2e3
    x[3, 5] = 700.0          # one large value in a block of small ones
    x[4, 256:512] = 0.0      # an all-zero block
    x[5] = np.abs(x[5])
    x[n - 1] = -np.abs(x[n - 1]) * 40.0      # sub-block sums near the top of their 20-bit range
    want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
    got = _gemv_gpu(gpu, w, rows, cols, x)
    _check_rows(got, want, s_abs)
    # the same columns one by one (other kernel) agree within the same bound
    for c in range(n):
        one = _gemv_gpu(gpu, w, rows, cols, x[c:c + 1])
        _check_rows(one, want[c:c + 1], s_abs[c:c + 1])


def test_gemv_reports_sums_outside_the_accumulator_range(gpu):
    torch, binding = gpu
    w, x = synth.gemv_case(seed=3, rows=64, cols=2048)       # literal distribution: weights of mean +1.6
    y = torch.zeros((1, 64), dtype=torch.float32, device="cuda")
    binding.prima_gemv_q4k(_to_dev(torch, w), 64, 2048, _to_dev(torch, np.abs(x) * 1e3), 1, y)          # sums ~2.6e6: fine
    with pytest.raises(binding.PrimaError) as err:
        binding.prima_gemv_q4k(_to_dev(torch, w), 64, 2048, _to_dev(torch, np.abs(x) * 1e6), 1, y)      # sums ~2.6e9 > 2^27
    assert err.value.code == binding.ERR_DEVICE
    # the library stays usable
    binding.prima_gemv_q4k(_to_dev(torch, w), 64, 2048, _to_dev(torch, x), 1, y)


def test_gemv_run_to_run_bits_are_identical(gpu):
    w, x = synth.gemv_case(seed=2, rows=2048, cols=4096)
    a = _gemv_gpu(gpu, w, 2048, 4096, x)
    b = _gemv_gpu(gpu, w, 2048, 4096, x)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_gemv_rejects_bad_arguments(gpu):
    torch, binding = gpu
    w = torch.zeros(144, dtype=torch.uint8, device="cuda")
    x = torch.zeros(200, dtype=torch.float32, device="cuda")
    y = torch.zeros(1, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PrimaError):
        binding.prima_gemv_q4k(w, 1, 200, x, 1, y)
    with pytest.raises(binding.PrimaError):
        binding.prima_gemv_q4k(w, 1, 256, x, 17, y)
