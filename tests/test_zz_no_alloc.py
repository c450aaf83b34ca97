"""prima_gemv_q4k_noalloc: the matrix-vector product for callers that may not allocate GPU memory
(engines that own the whole device through their own arena, loops that cannot afford cudaMalloc).

It must give the same answers as prima_gemv_q4k -- here: both within the per-row bound of the CPU
checker, and within twice that bound of each other -- on two calls in a row that reuse the
library's built-in scratch array, and it must refuse products larger than that array.
This file sorts last on purpose, so a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest

import oracle
from paper_2504_08791_b200 import synth

pytestmark = pytest.mark.gpu

ROW_TOL = 1e-3      # of sum |w x| per row, as in the other GEMV tests


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    import torch
    from paper_2504_08791_b200 import binding

    cases = [(1000, 2048, 3, 31), (264, 1280, 1, 32)]     # the second call is smaller: stale partials stay in the array
    for rows, cols, n_cols, seed in cases:
        w, x = synth.gemv_case(seed=seed, rows=rows, cols=cols, n_cols=n_cols)
        want, s_abs = oracle.gemv_q4k(w, rows, cols, x)
        dw, dx = torch.from_numpy(w).cuda(), torch.from_numpy(x).cuda()
        y_old = torch.full((n_cols, rows), float("nan"), dtype=torch.float32, device="cuda")
        y_new = torch.full((n_cols, rows), float("nan"), dtype=torch.float32, device="cuda")
        binding.prima_gemv_q4k(dw, rows, cols, dx, n_cols, y_old)
        binding.prima_gemv_q4k_noalloc(dw, rows, cols, dx, n_cols, y_new)
        torch.cuda.synchronize()
        a, b = y_old.cpu().numpy().astype(np.float64), y_new.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(b - want) <= ROW_TOL * s_abs)
        assert np.all(np.abs(a - want) <= ROW_TOL * s_abs)
        assert np.all(np.abs(a - b) <= 2 * ROW_TOL * s_abs)


def test_sizes_beyond_the_built_in_scratch_are_refused_with_a_clear_message():
    import torch
    from paper_2504_08791_b200 import binding

    d = torch.zeros(1024, dtype=torch.uint8, device="cuda")
    f = torch.zeros(1024, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PrimaError) as e:
        binding.prima_gemv_q4k_noalloc(d, 1 << 20, 2048, f, 1, f)      # 2^20 * 8 partials > 4 Mi: refused before any launch
    assert "exceeds the built-in scratch" in str(e.value)
    with pytest.raises(binding.PrimaError) as e:
        binding.prima_gemv_q4k_noalloc(d, 1 << 22, 256 << 42, f, 1, f)   # rows * (cols/256) wraps to 0 in 64 bits: still refused by size
    assert e.value.code == binding.ERR_ARG and "exceeds the built-in scratch" in str(e.value)
    with pytest.raises(binding.PrimaError):
        binding.prima_gemv_q4k_noalloc(d, 8, 200, f, 1, f)             # cols not a multiple of 256
