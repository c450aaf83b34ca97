"""Continuous batching of concurrent requests on the head device (paper Appendix A.11, "Ablation Study on
Multi-Request Workloads", and Appendix A.12, "Multi-request batching").

What the paper fixes: a job queue is kept on the head device; the active requests are merged at the token step;
every request has its own KV cache; only ONE micro-batch is in flight at a time, and the ring schedule is unchanged
(the micro-batch passes window after window exactly as a single request does).

Here a micro-batch is one call chain ``prima_embed`` -> ``prima_forward_window_seqs`` per window ->
``prima_logits`` -> ``prima_argmax`` over one token of each active request (at most ``PRIMA_MAX_N_SEQ`` of them).  A
request that is still reading its prompt feeds its next prompt token and ignores the logits; a request past its
prompt feeds the token it produced in the step before.  Requests join as soon as a cache slot is free and leave as
soon as they have produced their tokens, both between steps.  Decoding is greedy, so the tokens of a request do not
depend on which other requests shared its steps.  Only orchestration lives here; the executor does the model steps.
"""
from __future__ import annotations

from collections import deque
from dataclasses import dataclass, field
from typing import Deque, Dict, List, Optional, Sequence

import numpy as np


@dataclass
class Job:
    """One request: a prompt (at least one token) and how many tokens to produce after it."""
    job_id: int
    prompt: List[int]
    max_new_tokens: int
    eos_token: Optional[int] = None
    output: List[int] = field(default_factory=list)
    # filled by the queue
    slot: int = -1            # cache (sequence id) the request holds while it is active
    fed: int = 0              # tokens fed so far = position of the next token in the request's cache
    joined_at_step: int = -1
    left_at_step: int = -1

    @property
    def done(self) -> bool:
        return len(self.output) >= self.max_new_tokens or (self.eos_token is not None and bool(self.output) and self.output[-1] == self.eos_token)


class ContextExecutor:
    """The model steps of a micro-batch on a library context (``binding.Context``), window after window."""

    def __init__(self, ctx, windows: Optional[Sequence[int]] = None, max_batch: Optional[int] = None):
        import torch
        self.ctx = ctx
        cfg = ctx.cfg
        bounds = list(windows) if windows is not None else [0, cfg["n_layers"]]
        if bounds[0] != 0 or bounds[-1] != cfg["n_layers"] or any(b <= a for a, b in zip(bounds, bounds[1:])):
            raise ValueError("windows must be ascending layer boundaries from 0 to n_layers")
        self.bounds = bounds
        self.max_batch = int(max_batch if max_batch is not None else cfg.get("max_n_tok", 8))
        self.kv_capacity = int(cfg["kv_capacity"])
        self.hid = torch.empty((self.max_batch, cfg["hidden"]), dtype=torch.float32, device="cuda")
        self.logits = torch.empty((self.max_batch, cfg["vocab"]), dtype=torch.float32, device="cuda")

    def step(self, tokens: Sequence[int], slots: Sequence[int], positions: Sequence[int]) -> np.ndarray:
        """One token of each request (its cache, its position): the greedy next token of each."""
        n = len(tokens)
        hid, logits = self.hid[:n], self.logits[:n]
        self.ctx.embed(list(tokens), hid)
        for lb, le in zip(self.bounds, self.bounds[1:]):
            self.ctx.forward_window_seqs(lb, le, hid, hid, list(slots), list(positions))
        self.ctx.logits(hid, n, logits)
        return self.ctx.argmax(logits, n)


class JobQueue:
    """The head device's queue: ``submit`` jobs at any time, ``step`` runs one micro-batch, ``run`` until all are done."""

    def __init__(self, executor, max_batch: Optional[int] = None, n_slots: Optional[int] = None):
        self.executor = executor
        self.max_batch = int(max_batch if max_batch is not None else executor.max_batch)
        if self.max_batch < 1 or self.max_batch > executor.max_batch:
            raise ValueError("max_batch outside 1 .. the executor's limit")
        n_slots = int(n_slots if n_slots is not None else self.max_batch)
        if n_slots < self.max_batch:
            raise ValueError("fewer cache slots than requests per step")
        self.free_slots: Deque[int] = deque(range(n_slots))
        self.waiting: Deque[Job] = deque()
        self.active: List[Job] = []          # in order of admission
        self.finished: Dict[int, Job] = {}
        self.steps = 0
        self.batch_sizes: List[int] = []
        self._next_id = 0

    def submit(self, prompt: Sequence[int], max_new_tokens: int, eos_token: Optional[int] = None) -> int:
        prompt = [int(t) for t in prompt]
        if not prompt:
            raise ValueError("a prompt has at least one token")
        if max_new_tokens < 1:
            raise ValueError("max_new_tokens must be positive")
        if len(prompt) + max_new_tokens - 1 > self.executor.kv_capacity:
            raise ValueError("prompt + new tokens exceed the cache capacity")
        job = Job(self._next_id, prompt, int(max_new_tokens), eos_token)
        self._next_id += 1
        self.waiting.append(job)
        return job.job_id

    def _admit(self):
        while self.waiting and self.free_slots and len(self.active) < self.max_batch:
            job = self.waiting.popleft()
            job.slot = self.free_slots.popleft()
            job.joined_at_step = self.steps
            self.active.append(job)

    def step(self) -> int:
        """Admit waiting jobs into free slots, run one micro-batch, retire the jobs that are done.  Returns the number
        of requests in the micro-batch (0: nothing to do)."""
        self._admit()
        batch = self.active[:self.max_batch]
        if not batch:
            return 0
        tokens = [job.prompt[job.fed] if job.fed < len(job.prompt) else job.output[-1] for job in batch]
        picked = self.executor.step(tokens, [job.slot for job in batch], [job.fed for job in batch])
        self.steps += 1
        self.batch_sizes.append(len(batch))
        for job, tok in zip(batch, picked):
            job.fed += 1
            if job.fed >= len(job.prompt):      # the prompt is in: the model's choice after this token counts
                job.output.append(int(tok))
            if job.done:
                job.left_at_step = self.steps
                self.active.remove(job)
                self.free_slots.append(job.slot)      # the next holder starts at position 0 and overwrites the cache
                self.finished[job.job_id] = job
        return len(batch)

    def run(self, max_steps: int = 1 << 30) -> Dict[int, List[int]]:
        """Steps until the queue is empty; the tokens of every finished job by job id."""
        for _ in range(max_steps):
            if self.step() == 0:
                break
        return {jid: job.output for jid, job in self.finished.items()}
