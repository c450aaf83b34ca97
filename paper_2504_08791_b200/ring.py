"""Pipelined-ring execution of one decoding step over several ranks (paper Section 3.1; Appendix A.12, "Mmap- and
prefetch-based PRP"): the windows of ``schedule.windows`` are dealt to the ranks in ring order, rank m runs the
windows whose ``device`` is m on the layers it holds, and what crosses a window boundary is the hidden state, e fp32
values per token (Appendix A.3: 4e bytes), sent point to point to the rank that owns the next window.  The head
(rank 0) feeds the first window and receives the output of the last one, as in the paper, where the head device
holds the input and output layers.

No collective is on the data path: one ``send`` and one ``recv`` per boundary whose two sides are different ranks.
On GPUs the executor is a ``binding.Context`` holding only this rank's layers, the buffers are CUDA tensors and the
process group is NCCL (the message lands in the receiver's own memory before any kernel reads it); the same code
runs on CPU ranks over gloo with any object that has ``forward_window(lb, le, hidden_in, hidden_out, pos, n_tok)``.
One micro-batch is in flight: a rank idles while the others work, which adds capacity, not speed, for one request.
"""
from __future__ import annotations

from typing import List, Sequence

from . import schedule


def my_windows(sched: Sequence[schedule.Window], rank: int) -> List[schedule.Window]:
    """The windows this rank executes, in order."""
    return [w for w in sched if w.device == rank]


def my_layers(sched: Sequence[schedule.Window], rank: int) -> List[int]:
    """The layers whose weights and KV caches this rank has to hold."""
    return [l for w in my_windows(sched, rank) for l in range(w.layer_begin, w.layer_end)]


def messages(sched: Sequence[schedule.Window], hidden: int, n_tok: int = 1):
    """(src rank, dst rank, bytes) of every hand-off of one step, in order, including the return to the head."""
    out = []
    for a, b in zip(sched, list(sched[1:]) + [None]):
        dst = 0 if b is None else b.device
        if a.device != dst:
            out.append((a.device, dst, schedule.boundary_bytes(hidden, n_tok)))
    return out


def ring_step(executor, dist, rank: int, sched: Sequence[schedule.Window], hidden, scratch, pos: int, n_tok: int):
    """One decoding step.  ``hidden``: on rank 0 the input [n_tok, e] of the first window; it is overwritten, and
    on rank 0 it holds the output of the last window when the call returns.  ``scratch``: a buffer of the same
    shape.  Every rank calls this with the same ``sched``, ``pos`` and ``n_tok``."""
    have = rank == 0          # does this rank hold the current hidden state?
    n = len(sched)
    for i, w in enumerate(sched):
        nxt = sched[i + 1].device if i + 1 < n else 0
        if w.device == rank:
            if not have:
                raise RuntimeError("ring schedule out of step: the hidden state has not arrived")
            executor.forward_window(w.layer_begin, w.layer_end, hidden, scratch, pos, n_tok)
            hidden.copy_(scratch)
            if nxt != rank:
                dist.send(hidden, dst=nxt)
                have = False
        elif nxt == rank and w.device != rank:
            dist.recv(hidden, src=w.device)
            have = True
    return hidden
