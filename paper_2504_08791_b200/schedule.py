"""Pipelined-ring schedule arithmetic (paper Section 3.1 and Appendix A.12, "Mmap- and prefetch-based
PRP"; the closed forms of Appendix A.3, computation latency and device copy time).

The model's L layers are cut into contiguous windows that are dealt to the M devices in ring order,
device m taking w_m layers each time its turn comes, round after round, until the layers run out (the
last window may be shorter).  ``windows`` enumerates them; ``layers_per_device`` and
``windows_per_device`` are the paper's closed forms for how many layers and how many windows each
device ends up with.  ``run_schedule`` executes the windows of one step, in order, on one context
(every "device" of the ring is then the same GPU; what crosses a window boundary is the hidden state).
"""
from __future__ import annotations

from typing import List, NamedTuple, Sequence


class Window(NamedTuple):
    round: int          # 0-based round of the ring
    device: int         # 0-based position in the ring
    layer_begin: int    # 0-based, inclusive
    layer_end: int      # exclusive


def windows(n_layers: int, window_sizes: Sequence[int]) -> List[Window]:
    """All windows of one token step in execution order."""
    if n_layers < 1 or not window_sizes or any(w < 1 for w in window_sizes):
        raise ValueError("need n_layers >= 1 and window sizes >= 1")
    out, layer, rnd = [], 0, 0
    while layer < n_layers:
        for m, w in enumerate(window_sizes):
            if layer >= n_layers:
                break
            end = min(layer + w, n_layers)
            out.append(Window(rnd, m, layer, end))
            layer = end
        rnd += 1
    return out


def _remainder_share(n_layers: int, window_sizes: Sequence[int], m: int, unit: int) -> int:
    """min(unit, max(0, R - sum_{j<m} min(w_j, R))) with R = L mod W: what device m gets of the last, partial round."""
    total = sum(window_sizes)
    r = n_layers % total
    before = sum(min(w, r) for w in window_sizes[:m])
    return min(unit, max(0, r - before))


def layers_per_device(n_layers: int, window_sizes: Sequence[int]) -> List[int]:
    """l_m = floor(L / W) w_m + min(w_m, max(0, R - sum_{j<m} min(w_j, R))),  W = sum w_m,  R = L mod W."""
    total = sum(window_sizes)
    return [n_layers // total * w + _remainder_share(n_layers, window_sizes, m, w) for m, w in enumerate(window_sizes)]


def gpu_layers_per_device(n_layers: int, window_sizes: Sequence[int], gpu_layers: Sequence[int]) -> List[int]:
    """l_m^gpu = floor(L / W) n_m + min(n_m, max(0, R - sum_{j<m} min(w_j, R))),  n_m <= w_m layers of a window on the GPU."""
    if len(gpu_layers) != len(window_sizes) or any(n < 0 or n > w for n, w in zip(gpu_layers, window_sizes)):
        raise ValueError("need 0 <= n_m <= w_m for every device")
    total = sum(window_sizes)
    return [n_layers // total * n + _remainder_share(n_layers, window_sizes, m, n) for m, n in enumerate(gpu_layers)]


def windows_per_device(n_layers: int, window_sizes: Sequence[int]) -> List[int]:
    """W_m = floor(L / W) + min(1, max(0, R - sum_{j<m} min(w_j, R)))."""
    total = sum(window_sizes)
    return [n_layers // total + _remainder_share(n_layers, window_sizes, m, 1) for m in range(len(window_sizes))]


def rounds(n_layers: int, window_sizes: Sequence[int]) -> int:
    """k: rounds of the ring per token (the last one may be partial)."""
    total = sum(window_sizes)
    return -(-n_layers // total)


def boundary_bytes(hidden: int, n_tok: int = 1) -> int:
    """What crosses a window boundary: the hidden state, e fp32 values per token (Appendix A.3, 4e bytes)."""
    return 4 * hidden * n_tok


def run_schedule(ctx, schedule: Sequence[Window], hidden_in, hidden_out, pos: int, n_tok: int) -> None:
    """One token step: the windows in ring order on one context (prima_forward_window per window)."""
    src = hidden_in
    for w in schedule:
        ctx.forward_window(w.layer_begin, w.layer_end, src, hidden_out, pos, n_tok)
        src = hidden_out
