"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, no data-path
collective; only the timing is reduced (max over ranks) and rank seeds differ."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
from paper_2504_08791_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms_local = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.aggregate_over_ranks(ms_local, dist)
    seed = bench.SEEDS["70b"] + 1000 * rank            # what run_ours gives each replica
    w = synth.model_tensor(seed, 0, synth.WQ, 8, 256)
    gathered = [None] * world
    dist.all_gather_object(gathered, (ms, int(w.sum())))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_time_by_max_and_use_distinct_replicas():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [15.0, 15.0]          # both ranks see the slowest rank's time
    assert res[0][1] != res[1][1]                        # different seeds -> different replicas
    v = bench.job_value(15.0, 2)
    assert v["ms_per_token"] == 7.5 and abs(v["tokens_per_s"] - 2e3 / 15.0) < 1e-9


def test_single_process_needs_no_process_group():
    assert bench.aggregate_over_ranks(3.25, None) == 3.25
    b = bench.bytes_per_token(synth.model_config("70b"), 4096)
    # the paper's device-loading model: per layer b + 2 (h_k e_k + h_v e_v) n_kv, plus the output layer
    assert b["layer_weights"] == 481296384 and b["layer_kv"] == 2 * (8 * 128 * 2) * 4096
    assert b["total"] == 80 * (481296384 + 16777216) + 128256 * 32 * 144
