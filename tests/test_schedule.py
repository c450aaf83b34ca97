"""Pipelined-ring schedule arithmetic against the paper's worked examples and against brute force."""
import itertools

import numpy as np
import pytest

from paper_2504_08791_b200 import schedule
from tests.golden import _read


def test_the_80_layer_example_of_the_paper():
    ex = _read.prp_schedules()["a12_80_layers"]
    ws = schedule.windows(ex["layers"], ex["window_sizes"])
    assert [(w.round, w.device, w.layer_begin + 1, w.layer_end) for w in ws] == ex["w"]     # the paper counts layers from 1, inclusive
    assert schedule.rounds(ex["layers"], ex["window_sizes"]) == ex["rounds"]
    assert schedule.layers_per_device(ex["layers"], ex["window_sizes"]) == [20, 20, 20, 20]


def test_the_36_layer_figure_of_the_paper():
    ex = _read.prp_schedules()["fig_36_layers"]
    ws = schedule.windows(ex["layers"], ex["window_sizes"])
    assert len(ws) == ex["n_windows"]
    assert schedule.rounds(ex["layers"], ex["window_sizes"]) == ex["rounds"]
    assert schedule.windows_per_device(ex["layers"], ex["window_sizes"]) == [ex["windows_per_device"]] * 6
    assert all(w.layer_end - w.layer_begin == 2 for w in ws)


def test_windows_tile_the_layers_in_ring_order():
    rng = np.random.default_rng(0)
    for _ in range(200):
        m = int(rng.integers(1, 7))
        sizes = [int(rng.integers(1, 9)) for _ in range(m)]
        n_layers = int(rng.integers(1, 120))
        ws = schedule.windows(n_layers, sizes)
        assert ws[0].layer_begin == 0 and ws[-1].layer_end == n_layers
        for a, b in zip(ws, ws[1:]):
            assert a.layer_end == b.layer_begin                                     # contiguous, nothing twice
            assert (b.round, b.device) == ((a.round, a.device + 1) if a.device + 1 < m else (a.round + 1, 0))
        for w in ws[:-1]:
            assert w.layer_end - w.layer_begin == sizes[w.device]                   # only the last window may be short


def test_closed_forms_equal_brute_force_counts():
    for n_layers, sizes in itertools.product(range(1, 60), [[1], [3], [2, 2], [1, 4], [5, 2, 3], [1, 1, 1, 1], [4, 7, 2, 6, 1]]):
        ws = schedule.windows(n_layers, sizes)
        layers = [sum(w.layer_end - w.layer_begin for w in ws if w.device == m) for m in range(len(sizes))]
        count = [sum(1 for w in ws if w.device == m) for m in range(len(sizes))]
        assert schedule.layers_per_device(n_layers, sizes) == layers, (n_layers, sizes)
        assert schedule.windows_per_device(n_layers, sizes) == count, (n_layers, sizes)
        # with the first n_m layers of every window on the GPU
        gpu = [max(0, w - 1) for w in sizes]
        brute = [sum(min(g, w.layer_end - w.layer_begin) for w in ws if w.device == m) for m, g in enumerate(gpu)]
        assert schedule.gpu_layers_per_device(n_layers, sizes, gpu) == brute, (n_layers, sizes)


def test_boundary_message_and_argument_checks():
    assert schedule.boundary_bytes(8192) == 32768           # 4e bytes for the 70B shape
    assert schedule.boundary_bytes(8192, 5) == 5 * 32768
    with pytest.raises(ValueError):
        schedule.windows(0, [1])
    with pytest.raises(ValueError):
        schedule.windows(10, [2, 0])
    with pytest.raises(ValueError):
        schedule.gpu_layers_per_device(10, [2, 2], [3, 0])
