"""The ring over several ranks on CPU (gloo): every rank holds only its own windows' layers in a CPU checker model,
the hidden state travels rank to rank, and the head ends up with exactly the bits of a single full-depth pass."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2504_08791_b200 import ring, schedule, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


class _OracleExecutor:
    """forward_window of the ring interface on top of a checker model that holds a subset of the layers."""

    def __init__(self, cfg, seed, layers, n_prefill):
        self.mdl = oracle.Model(cfg, n_threads=2)
        for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg, layers=layers, with_globals=False):
            self.mdl.load(layer, tid, data, rows, cols)
        for l in layers:
            k, v = synth.kv_prefill(seed, l, n_prefill, cfg["n_kv_heads"], cfg["head_dim"])
            self.mdl.kv_load(l, 0, k, v)

    def forward_window(self, lb, le, hidden_in, hidden_out, pos, n_tok):
        hidden_out.copy_(torch.from_numpy(self.mdl.forward_window(lb, le, hidden_in.numpy(), pos)))


def _worker(rank, world, port, sizes, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = synth.model_config("tiny", n_layers=5)
    seed, pos0, n_tok, steps = 83, 20, 2, 3
    sched = schedule.windows(cfg["n_layers"], sizes)
    ex = _OracleExecutor(cfg, seed, ring.my_layers(sched, rank), pos0)
    hidden = torch.zeros((n_tok, cfg["hidden"]), dtype=torch.float32)
    scratch = torch.zeros_like(hidden)
    results = []
    for s in range(steps):
        if rank == 0:
            hidden.copy_(torch.from_numpy(synth.activations(seed + s, n_tok, cfg["hidden"])))
        ring.ring_step(ex, dist, rank, sched, hidden, scratch, pos0 + s * n_tok, n_tok)
        if rank == 0:
            results.append(hidden.numpy().copy())
    if rank == 0:
        out.put(results)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,sizes", [(2, [1, 1]), (2, [2, 1]), (3, [1, 2, 1])])
def test_ring_over_gloo_ranks_reproduces_the_single_pass(world, sizes):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, sizes, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = synth.model_config("tiny", n_layers=5)
    seed, pos0, n_tok = 83, 20, 2
    full = _OracleExecutor(cfg, seed, range(cfg["n_layers"]), pos0)
    for s, g in enumerate(got):
        h0 = synth.activations(seed + s, n_tok, cfg["hidden"])
        want = full.mdl.forward_window(0, cfg["n_layers"], h0, pos0 + s * n_tok)
        assert np.array_equal(g.view(np.uint32), want.view(np.uint32))


def test_ring_bookkeeping_matches_the_papers_example():
    # Appendix A.12: 80 layers, 4 devices, window 10: two rounds, device m runs layers 10m..10m+9 and 40+10m..
    sched = schedule.windows(80, [10, 10, 10, 10])
    assert [(w.layer_begin, w.layer_end) for w in ring.my_windows(sched, 2)] == [(20, 30), (60, 70)]
    assert ring.my_layers(sched, 0) == list(range(0, 10)) + list(range(40, 50))
    msgs = ring.messages(sched, hidden=8192, n_tok=1)
    assert len(msgs) == 8 and all(b == 4 * 8192 for _, _, b in msgs)          # 4e bytes per hand-off
    assert [m[:2] for m in msgs] == [(0, 1), (1, 2), (2, 3), (3, 0), (0, 1), (1, 2), (2, 3), (3, 0)]
    # a single device: no message at all
    assert ring.messages(schedule.windows(12, [4]), 1024) == []
    # uneven windows, partial last round: the last window's owner returns the state to the head
    sched = schedule.windows(7, [3, 2])
    assert [(w.device, w.layer_begin, w.layer_end) for w in sched] == [(0, 0, 3), (1, 3, 5), (0, 5, 7)]
    assert [m[:2] for m in ring.messages(sched, 512)] == [(0, 1), (1, 0)]
