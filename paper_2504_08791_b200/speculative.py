"""Speculative decoding on top of the layer-window calls (paper Appendix A.9, "Run Prima.cpp with
Speculative Decoding", and Appendix A.12, "Speculative decoding").

A small draft model proposes ``n_draft`` tokens one by one; the target model then runs ONE step over
the last accepted token and the proposals (``n_draft + 1`` tokens at consecutive cache positions,
causal among themselves) and its own greedy choice after each of them is compared with the
proposals.  The longest agreeing prefix is kept and the target's choice after it is appended, so a
cycle yields between 1 and ``n_draft + 1`` tokens and the output is exactly what greedy decoding
with the target alone would give.  A rejected suffix needs no clean-up: the caches are addressed by
position and the next cycle overwrites the stale entries.

Only orchestration lives here: every model step is ``prima_embed`` / ``prima_forward_window`` /
``prima_logits`` / ``prima_argmax`` on a context.  torch is used for the device buffers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np


@dataclass
class SpeculativeStats:
    cycles: int = 0
    proposed: int = 0
    accepted: int = 0                      # proposals that the target confirmed
    per_cycle: List[int] = field(default_factory=list)   # tokens produced by each cycle

    @property
    def acceptance(self) -> float:
        return self.accepted / self.proposed if self.proposed else 0.0


class _Stepper:
    """One model behind a context: feed tokens at consecutive positions, get the greedy choices."""

    def __init__(self, ctx, windows: Optional[Sequence[int]] = None):
        import torch
        self.ctx = ctx
        cfg = ctx.cfg
        self.n_layers = cfg["n_layers"]
        bounds = list(windows) if windows is not None else [0, self.n_layers]
        if bounds[0] != 0 or bounds[-1] != self.n_layers or any(b <= a for a, b in zip(bounds, bounds[1:])):
            raise ValueError("windows must be ascending layer boundaries from 0 to n_layers")
        self.bounds = bounds
        n = cfg.get("max_n_tok", 8)
        self.max_n_tok = n
        self.hid = torch.empty((n, cfg["hidden"]), dtype=torch.float32, device="cuda")
        self.logits = torch.empty((n, cfg["vocab"]), dtype=torch.float32, device="cuda")

    def step(self, tokens: Sequence[int], pos: int) -> np.ndarray:
        """Tokens at positions pos, pos+1, ...: returns the greedy next token after each of them."""
        n = len(tokens)
        if not 1 <= n <= self.max_n_tok:
            raise ValueError("between 1 and max_n_tok tokens per step")
        hid, logits = self.hid[:n], self.logits[:n]
        self.ctx.embed(list(tokens), hid)
        for lb, le in zip(self.bounds, self.bounds[1:]):          # the ring schedule: window after window
            self.ctx.forward_window(lb, le, hid, hid, pos, n)
        self.ctx.logits(hid, n, logits)
        return self.ctx.argmax(logits, n)


class SpeculativeDecoder:
    """Greedy speculative decoding with a draft context and a target context that share a vocabulary.

    Both caches must hold the same ``pos`` positions of context when ``generate`` is called.
    ``draft_filter`` (tests only) may alter the proposals before verification.
    """

    def __init__(self, target, draft, n_draft: int = 4, target_windows: Optional[Sequence[int]] = None,
                 draft_filter: Optional[Callable[[List[int]], List[int]]] = None):
        if target.cfg["vocab"] != draft.cfg["vocab"]:
            raise ValueError("draft and target need the same vocabulary")
        if not 1 <= n_draft < target.cfg.get("max_n_tok", 8):
            raise ValueError("n_draft + 1 tokens must fit one step of the target")
        self.target = _Stepper(target, target_windows)
        self.draft = _Stepper(draft)
        self.n_draft = n_draft
        self.draft_filter = draft_filter
        self.capacity = min(target.cfg["kv_capacity"], draft.cfg["kv_capacity"])

    @classmethod
    def from_steppers(cls, target_step, draft_step, n_draft: int, capacity: int, max_n_tok: int = 8):
        """A decoder over two objects with ``step(tokens, pos) -> next tokens`` (how the accept/reject
        logic is exercised without a GPU)."""
        if not 1 <= n_draft < max_n_tok:
            raise ValueError("n_draft + 1 tokens must fit one step of the target")
        self = cls.__new__(cls)
        self.target, self.draft = target_step, draft_step
        self.n_draft, self.draft_filter, self.capacity = n_draft, None, capacity
        return self

    def generate(self, first_token: int, pos: int, n_new: int):
        """Continue from ``first_token`` (not yet in either cache) at position ``pos``; returns the
        ``n_new`` tokens that follow it and the statistics of the run."""
        stats = SpeculativeStats()
        out: List[int] = []
        history = {pos: int(first_token)}      # token at each position from `pos` on
        last_pos = pos                         # position of the newest token, present in no cache yet
        draft_valid = pos                      # the draft cache holds positions < draft_valid
        capacity = self.capacity
        while len(out) < n_new:
            n_draft = min(self.n_draft, capacity - last_pos - 1)
            if n_draft < 1:
                raise ValueError("the KV caches are full")
            # ---- draft: first catch up with tokens the draft has not consumed (at most one, after a
            #      cycle in which every proposal was accepted), then propose one token at a time
            proposals: List[int] = []
            feed = [history[p] for p in range(draft_valid, last_pos + 1)]
            nxt = int(self.draft.step(feed, draft_valid)[-1])
            draft_valid = last_pos + 1
            proposals.append(nxt)
            while len(proposals) < n_draft:
                nxt = int(self.draft.step([proposals[-1]], draft_valid)[0])
                draft_valid += 1
                proposals.append(nxt)
            consumed = proposals[:-1]          # what the draft cache now holds after history[last_pos]
            if self.draft_filter is not None:
                proposals = [int(t) for t in self.draft_filter(list(proposals))]
            # ---- target: one step over the newest token and the proposals
            choice = self.target.step([history[last_pos]] + proposals, last_pos)
            k = 0
            while k < n_draft and proposals[k] == int(choice[k]):
                k += 1
            new = [int(t) for t in choice[:k + 1]]       # k confirmed proposals + the target's own next token
            stats.cycles += 1
            stats.proposed += n_draft
            stats.accepted += k
            stats.per_cycle.append(len(new))
            for i, t in enumerate(new):
                history[last_pos + 1 + i] = t
            out.extend(new)
            # the draft cache stays valid as far as what it consumed is what was kept; the newest token is
            # always fed again, because its successor has to be proposed
            v = 0
            while v < len(consumed) and v < len(new) - 1 and consumed[v] == new[v]:
                v += 1
            draft_valid = last_pos + 1 + v
            last_pos += len(new)
        return out[:n_new], stats
