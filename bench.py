#!/usr/bin/env python
"""Decode benchmark of the Q4_K layer-window hot path.

One "step" is one decoded token: the hidden state of the newest token goes through every layer of
the model, issued as contiguous layer windows (4 windows of 20 layers for the 70B shape, the
paper's ring schedule with window 20), then through the output layer.  Weights are synthetic
random-init Q4_K tensors of the named shape; the KV cache is prefilled with N(0,1) fp16 entries.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 70b|32b|8b] [--n-tok T] [--impl ours|reference]

With --n-tok T > 1 a step is one verification pass of speculative decoding: T tokens at consecutive
positions go through the model together (causal among themselves) and the time is reported per step.
Other lines: --requests R (one token of each of R concurrent requests per step, own caches), --ctx N (cached
positions), --speculative 8b (speculative cycles with a draft model), --resident-layers N (the layers from N on
are streamed from pinned host memory every token; reported against the host-link rate measured in the same run),
--gemv-fmt q6_k|q8_0|f16 (the single product in another weight format), --l2-ahead-mb / --l2-ahead-o-mb (how much
of the gate/up matrix is asked into L2 during attention and the O product), --repeats (timed regions; the value is
their median).

With N > 1 (launched by torch.distributed.run) every rank decodes its own request on its own
GPU: the path does not shard, ranks are independent replicas and no collective is on the data
path; the barrier and the max-over-ranks reduction only bracket the timing.
Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2504_08791_b200 import schedule, synth  # noqa: E402

WORKLOADS = {
    # name: (shape, context length, number of windows, description)
    "70b": ("70b", 4096, 4, "Llama-3-70B-shaped random-init Q4_K, 80 layers as 4 windows x 20, fp16 KV context 4096, batch 1"),
    "32b": ("32b", 4096, 1, "Qwen2.5-32B-shaped random-init Q4_K, 64 layers, fp16 KV context 4096, batch 1"),
    "8b": ("8b", 1024, 1, "Llama-3-8B-shaped random-init Q4_K, 32 layers, fp16 KV context 1024, batch 1"),
}
SEEDS = {"70b": 3, "32b": 2, "8b": 1}
# dram__bytes_read.sum + dram__bytes_write.sum over the four 70B-shaped layer matrices / their Q4_K bytes
# (one ncu capture of gemv_partials_kernel<1>, profiles/gemv_partials_70b_matrices.md)
NCU_TRAFFIC_RATIO = (496.9 + 7.8 - 14.2) / 481.3      # read + written, without the bytes the O product asks ahead for gate/up


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def L_kv_bytes(cfg: dict, n_ctx: int) -> int:
    """K and V bytes of one request's attended positions over all layers."""
    return cfg["n_layers"] * 2 * (cfg["n_kv_heads"] * cfg["head_dim"] * 2) * n_ctx


def bytes_per_token(cfg: dict, n_ctx: int, n_layers: int | None = None, with_head: bool = True) -> dict:
    """Algorithmic bytes one decoded token must move: Q4_K weight bytes touched + K and V bytes of
    the attended positions (the paper's device-loading model: b + 2(h_k e_k + h_v e_v) n_kv per
    layer, b_o for the output layer)."""
    L = cfg["n_layers"] if n_layers is None else n_layers
    layer_w = synth.weight_bytes(cfg, (synth.WQ, synth.WK, synth.WV, synth.WO, synth.W_GATE, synth.W_UP, synth.W_DOWN))
    kv = 2 * (cfg["n_kv_heads"] * cfg["head_dim"] * 2) * n_ctx
    head = synth.weight_bytes(cfg, (synth.W_HEAD,)) if with_head else 0
    return dict(layer_weights=layer_w, layer_kv=kv, head=head, total=L * (layer_w + kv) + head)


# ------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi sampled every 200 ms while the timed region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.device = device
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "200",
                                          "-i", str(self.device)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        try:
            for line in open(self.path):
                f = [t.strip() for t in line.split(",")]
                if len(f) >= 9:
                    rows.append(f)
            os.unlink(self.path)
        except Exception:
            pass
        if not rows:
            return out
        sm = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in rows if r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        out.update(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None, reasons=sorted(reasons),
                   samples=len(rows))
        return out


# ------------------------------------------------------------------------------------ multi-rank
def aggregate_over_ranks(ms_local: float, dist, device=None) -> float:
    """Max over ranks of a rank's device time (ranks are independent replicas; the job takes as long
    as its slowest rank).  `dist` is torch.distributed or None for a single process."""
    if dist is None:
        return ms_local
    import torch
    t = torch.tensor([ms_local], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(ms_per_step_max: float, world: int) -> dict:
    """Whole-job numbers of N replicas that each decode one token per step."""
    return {"ms_per_token": ms_per_step_max / world, "tokens_per_s": world * 1e3 / ms_per_step_max}


# ------------------------------------------------------------------------------------ the GPU arm
def build_gpu_model(binding, cfg, seed, n_ctx, device, n_layers=None, n_requests=1, on_layer=None, on_globals=None,
                    resident_layers=None, stream_slots=None):
    """Generate the synthetic model layer by layer and make it resident.  on_layer(l, tensors, k, v) and
    on_globals(tensors) see the same host arrays (the CPU-baseline leg runs the checker on them, so the 39 GB of
    a 70B-shaped model are generated once and never held in host memory all at once)."""
    import torch
    t0 = time.time()
    ctx = binding.Context(cfg, device=device)
    if resident_layers is not None:
        ctx.set_option(binding.OPT_RESIDENT_LAYERS, resident_layers)
        if stream_slots:
            ctx.set_option(binding.OPT_STREAM_SLOTS, stream_slots)
    layers = range(cfg["n_layers"]) if n_layers is None else range(n_layers)
    for l in layers:
        tensors = {}
        for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg, layers=[l], with_globals=False):
            ctx.load(layer, tid, data, rows, cols)
            tensors[tid] = (rows, cols, data)
        k, v = synth.kv_prefill(seed, l, n_ctx, cfg["n_kv_heads"], cfg["head_dim"])
        for r in range(n_requests):               # every request gets a cache of its own (same synthetic content)
            ctx.kv_load(l, 0, k, v, seq=r)
        if on_layer is not None:
            on_layer(l, tensors, k, v)
    tensors = {}
    for tid in synth.GLOBAL_TENSORS:
        rows, cols = synth.tensor_shape(cfg, tid)
        data = synth.make_tensor(seed, cfg, -1, tid)
        ctx.load(-1, tid, data, rows, cols)
        tensors[tid] = (rows, cols, data)
    if on_globals is not None:
        on_globals(tensors)
    torch.cuda.synchronize()
    log(f"[bench] model resident after {time.time() - t0:.1f}s")
    return ctx


class WholeTokenOracle:
    """The CPU checker, as it stands, run over ONE whole token of the workload while the model is being generated:
    layer l is loaded into a one-layer checker model, run on the hidden state that layer l-1 left, and dropped;
    then the output layer.  Only the checker's own calls are timed (not the generation of the weights)."""

    def __init__(self, cfg, seed, n_ctx, n_tok=1):
        import oracle
        self.oracle, self.cfg, self.n_ctx = oracle, cfg, n_ctx
        self.cores = oracle.default_threads()
        self.h = synth.activations(seed, n_tok, cfg["hidden"])
        self.seconds, self.layers_done, self.logits = 0.0, 0, None

    def on_layer(self, l, tensors, k, v):
        one = dict(self.cfg, n_layers=1)
        mdl = self.oracle.Model(one, n_threads=self.cores)
        for tid, (rows, cols, data) in tensors.items():
            mdl.load(0, tid, data, rows, cols)
        mdl.kv_load(0, 0, k, v)
        t0 = time.perf_counter()
        self.h = mdl.forward_window(0, 1, self.h, self.n_ctx)
        self.seconds += time.perf_counter() - t0
        self.layers_done += 1
        mdl.close()

    def on_globals(self, tensors):
        one = dict(self.cfg, n_layers=1)
        mdl = self.oracle.Model(one, n_threads=self.cores)
        for tid in (synth.OUT_NORM, synth.W_HEAD):
            rows, cols, data = tensors[tid]
            mdl.load(-1, tid, data, rows, cols)
        t0 = time.perf_counter()
        self.logits = mdl.logits(self.h)
        self.seconds += time.perf_counter() - t0
        mdl.close()

    def result(self, n_tok=1):
        return {"value": self.seconds * 1e3, "unit": "ms/token" if n_tok == 1 else "ms/step", "cores": self.cores, "kind": "oracle",
                "sample": f"one whole {'token' if n_tok == 1 else 'step of %d tokens' % n_tok}: all {self.layers_done} layers at full width and "
                          f"{self.n_ctx} cached positions + the output layer, layer by layer (only the checker's calls are timed)"}


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2504_08791_b200 import binding

    binding.lib()
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    shape, n_ctx, n_windows, desc = WORKLOADS[args.workload]
    if args.ctx:
        n_ctx = args.ctx
    cfg = synth.model_config(shape)
    if args.layers:
        cfg["n_layers"] = args.layers
    cfg["kv_capacity"] = max(cfg["kv_capacity"], n_ctx + 64 * args.n_tok)
    cfg["max_n_tok"] = max(cfg.get("max_n_tok", 8), args.requests)
    L = cfg["n_layers"]
    seed = SEEDS[args.workload] + 1000 * rank
    R = args.requests
    if R > 1 and args.n_tok > 1:
        raise SystemExit("--requests and --n-tok are alternatives")
    whole = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and R == 1 and not args.layers:
        whole = WholeTokenOracle(cfg, seed, n_ctx, args.n_tok)
    resident = args.resident_layers if args.resident_layers >= 0 else None
    ctx = build_gpu_model(binding, cfg, seed, n_ctx, local_rank, n_requests=R,
                          on_layer=whole.on_layer if whole else None, on_globals=whole.on_globals if whole else None,
                          resident_layers=resident, stream_slots=args.stream_slots)
    if args.l2_ahead_mb >= 0:
        ctx.set_option(binding.OPT_L2_AHEAD_BYTES, args.l2_ahead_mb << 20)
    if args.l2_ahead_o_mb >= 0:
        ctx.set_option(binding.OPT_L2_AHEAD_O_BYTES, args.l2_ahead_o_mb << 20)
    bpt = bytes_per_token(cfg, n_ctx)
    if R > 1:                                     # the weights are read once per step, every request's cache once
        bpt = dict(bpt, total=bpt["total"] + (R - 1) * L_kv_bytes(cfg, n_ctx))
    # the ring schedule with equal windows and one round: n_windows "devices" of L / n_windows layers each
    ring = schedule.windows(L, [-(-L // n_windows)] * n_windows)
    bounds = [w.layer_begin for w in ring] + [L]
    n_windows = len(ring)

    T = args.n_tok if R == 1 else R
    h0 = torch.from_numpy(synth.activations(seed, T, cfg["hidden"])).cuda()
    hid = torch.empty_like(h0)
    logits = torch.empty((T, cfg["vocab"]), dtype=torch.float32, device="cuda")

    def windows(pos):
        for w in range(n_windows):
            if R > 1:                              # one token of each of R requests, all at the same depth of their caches
                ctx.forward_window_seqs(bounds[w], bounds[w + 1], hid, hid, list(range(R)), [pos] * R)
            else:
                ctx.forward_window(bounds[w], bounds[w + 1], hid, hid, pos, T)

    def device_step(pos):
        hid.copy_(h0)
        windows(pos)
        ctx.logits(hid, T, logits)

    def e2e_step(tok, pos):
        ctx.embed([tok] * T, hid)                  # host token ids -> device (4 bytes each)
        windows(pos)
        ctx.logits(hid, T, logits)
        return int(ctx.argmax(logits, T)[T - 1])   # device -> host (4 bytes each), waits

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        return aggregate_over_ranks(ms, dist, "cuda")

    for _ in range(args.warmup):
        device_step(n_ctx)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = ctx.launch_count()
    # the timed region (exactly --steps steps between two events, barrier and synchronize on both sides), taken
    # --repeats times back to back: the median region is the reported one, min and all are listed in `config`
    regions = []
    launches = 0
    for rep in range(max(1, args.repeats)):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(args.steps):
            device_step(n_ctx)
        ev1.record()
        barrier()
        if rep == 0:
            launches = ctx.launch_count() - launches0
        regions.append(max_over_ranks(ev0.elapsed_time(ev1)) / args.steps)
    ms_step = float(np.median(regions))

    # end to end through the ABI: host token in, host token out, every step
    adv = 1 if R > 1 else T                        # positions a step advances a cache by
    tok = 0
    for i in range(min(args.warmup, 3)):
        tok = e2e_step(tok, n_ctx + i * adv)
    barrier()
    e2e_steps = min(args.steps, (cfg["kv_capacity"] - n_ctx - 3 * adv) // adv)
    ev2, ev3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.perf_counter()
    ev2.record()
    for i in range(e2e_steps):
        tok = e2e_step(tok, n_ctx + (3 + i) * adv)
    ev3.record()
    torch.cuda.synchronize()
    wall_ms = (time.perf_counter() - wall0) * 1e3
    e2e_ms = max_over_ranks(max(ev2.elapsed_time(ev3), wall_ms)) / e2e_steps
    clocks = sampler.stop()

    # dominant kernel inside the running step: the kernels stamp the GPU timer themselves (first CTA past its
    # dependency wait .. last CTA done), launch sequence unchanged
    prof_steps = max(1, min(args.steps, 10))
    ctx.profile_enable(2)
    ev4, ev5 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev4.record()
    for _ in range(prof_steps):
        device_step(n_ctx)
    ev5.record()
    g_ms, g_n, g_bytes = ctx.profile_read(binding.PROF_GEMV)
    a_ms, a_n, a_bytes = ctx.profile_read(binding.PROF_ATTENTION)
    by_matrix = {}
    for name, klass in (("qkv", binding.PROF_GEMV_QKV), ("o", binding.PROF_GEMV_O), ("gate_up", binding.PROF_GEMV_GATE_UP),
                        ("down", binding.PROF_GEMV_DOWN), ("head", binding.PROF_GEMV_HEAD)):
        m_ms, m_n, m_bytes = ctx.profile_read(klass)
        if m_n:
            by_matrix[name] = {"avg_launch_us": m_ms * 1e3 / m_n, "GB/s": m_bytes / (m_ms * 1e-3) / 1e9, "MB": m_bytes / m_n / 1e6}
    stamped_ms_step = ev4.elapsed_time(ev5) / prof_steps
    # the same kernels in isolation: a pair of events around every launch (serialises them)
    ctx.profile_enable(1)
    iso_steps = max(1, min(args.steps, 5))
    for _ in range(iso_steps):
        device_step(n_ctx)
    gi_ms, gi_n, gi_bytes = ctx.profile_read(binding.PROF_GEMV)
    ai_ms, ai_n, ai_bytes = ctx.profile_read(binding.PROF_ATTENTION)
    ctx.profile_enable(0)

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = 6650.0, "fallback"
    gemv_gbs = g_bytes / (g_ms * 1e-3) / 1e9 if g_ms > 0 else 0.0
    attn_gbs = a_bytes / (a_ms * 1e-3) / 1e9 if a_ms > 0 else 0.0
    gemv_iso_gbs = gi_bytes / (gi_ms * 1e-3) / 1e9 if gi_ms > 0 else 0.0
    attn_iso_gbs = ai_bytes / (ai_ms * 1e-3) / 1e9 if ai_ms > 0 else 0.0
    kernel_name = "gemv_partials_kernel<%d>" % T if T <= 4 else "gemv_tokens_kernel"
    step_gbs = bpt["total"] / (ms_step * 1e-3) / 1e9

    result = {
        "metric": "decode_ms_per_token",
        "value": job_value(ms_step, world)["ms_per_token"],
        "unit": "ms/token",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step,
        "higher_is_better": False,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "q4_k weights x int16 activations, int32/fp32 accumulate",
        "data": "synthetic",
        "tokens_per_s": job_value(ms_step, world)["tokens_per_s"] * (R if R > 1 else 1),
        "config": {"workload": desc, "layers": L, "windows": n_windows, "n_ctx": n_ctx, "n_tok": T,
                   "value_is": ("ms per decoded token" if T == 1 else "ms per verification step of %d tokens" % T) if R == 1
                   else "ms per step of %d concurrent requests (one token each)" % R, "requests": R,
                   "parallelism": "replicas only" if world > 1 else "1 gpu", "l2": "inputs larger than L2 (>= 4.9 GB per step)",
                   "bytes_per_token": bpt["total"], "repeats": len(regions), "ms_per_step_min": min(regions),
                   "ms_per_step_all": regions, "value_is_median_of_repeats": True},
        "step_roofline": {"bound": "hbm", "achieved": step_gbs, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                          "frac": step_gbs / peak, "frac_of_nominal_8000": step_gbs / 8000.0},
        "roofline": {"kernel": kernel_name, "bound": "hbm", "achieved": gemv_gbs, "peak": peak, "peak_source": peak_src,
                     "unit": "GB/s", "frac": gemv_gbs / peak,
                     "traffic": None,
                     "traffic_estimated": (NCU_TRAFFIC_RATIO * g_bytes / g_n) if (g_n and T == 1 and args.workload == "70b") else None,
                     "traffic_note": "no DRAM counters for the kernel as it stands in this run; traffic_estimated = algorithmic bytes per "
                                     "launch x the DRAM read+write / Q4_K bytes ratio of the ncu capture named in profiles/",
                     "launches": g_n // prof_steps, "avg_launch_us": (g_ms * 1e3 / g_n) if g_n else None,
                     "kernel_ms_per_step": g_ms / prof_steps, "step_ms_in_this_pass": stamped_ms_step, "by_matrix": by_matrix,
                     "timing": f"in situ: every launch stamps the GPU timer (first CTA past its dependency wait .. last CTA done), "
                               f"launch sequence unchanged, pass of {prof_steps} steps after the timed region"},
        "roofline_isolated": {"kernel": kernel_name, "achieved": gemv_iso_gbs, "unit": "GB/s", "frac": gemv_iso_gbs / peak,
                              "avg_launch_us": (gi_ms * 1e3 / gi_n) if gi_n else None,
                              "timing": f"cuda events around each launch (serialised), separate pass of {iso_steps} steps"},
        "attention_kernel": {"achieved": attn_gbs, "unit": "GB/s", "frac": attn_gbs / peak, "launches": a_n // prof_steps,
                             "kernel_ms_per_step": a_ms / prof_steps, "isolated_achieved": attn_iso_gbs},
        "e2e": {"value": e2e_ms / world, "unit": "ms/token", "h2d_bytes_per_step": 4 * T, "d2h_bytes_per_step": 4 * T, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if resident is not None:
        result["streaming"] = streaming_report(torch, ctx, cfg, resident, args, ms_step)
    if args.speculative and world == 1:
        result["speculative"] = speculative_cycle(args, binding, ctx, cfg, seed, n_ctx, bounds)
    ctx.close()
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = whole.result(args.n_tok) if whole else cpu_baseline(args.workload, budget_s=args.cpu_budget)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return result


def streaming_report(torch, ctx, cfg, resident, args, ms_step) -> dict:
    """Layers streamed from pinned host memory: what a token has to bring over the host link, the link's rate for a
    plain pinned copy measured here, and the rate the decoding loop achieved."""
    n_streamed = cfg["n_layers"] - resident
    layer_bytes = synth.weight_bytes(cfg, (synth.WQ, synth.WK, synth.WV, synth.WO, synth.W_GATE, synth.W_UP, synth.W_DOWN))
    per_token = n_streamed * layer_bytes if n_streamed > max(1, args.stream_slots or 2) - 0 else 0
    src = torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(1 << 30, dtype=torch.uint8, device="cuda")
    dst.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        dst.copy_(src, non_blocking=True)
    e1.record()
    torch.cuda.synchronize()
    link_gbs = 3 * (1 << 30) / (e0.elapsed_time(e1) * 1e-3) / 1e9
    copied, copy_ms = ctx.stream_stats()
    achieved = per_token / (ms_step * 1e-3) / 1e9
    return {"resident_layers": resident, "streamed_layers": n_streamed, "slots": args.stream_slots or 2,
            "streamed_bytes_per_token": per_token, "host_link_GBs_plain_pinned_copy": link_gbs,
            "achieved_GBs_over_the_step": achieved, "frac_of_host_link": achieved / link_gbs if link_gbs else None,
            "floor_ms_per_token_at_host_link": per_token / (link_gbs * 1e9) * 1e3 if link_gbs else None,
            "copies_GBs_while_copying": copied / (copy_ms * 1e-3) / 1e9 if copy_ms else None,
            "note": "bound: the host link, not HBM; step_roofline above is against HBM and does not apply to this run"}


def speculative_cycle(args, binding, target, cfg, seed, n_ctx, bounds) -> dict:
    """Speculative decoding with a random-init draft of the named shape: time per cycle (4 draft steps + one
    5-token step of the target), end to end with the host in the loop.  Random-init models agree almost never,
    so besides the measured rate the tokens/s that k confirmed proposals per cycle would give are listed."""
    import torch
    from paper_2504_08791_b200.speculative import SpeculativeDecoder
    dcfg = synth.model_config(args.speculative)
    dcfg["kv_capacity"] = cfg["kv_capacity"]
    dcfg["vocab"] = cfg["vocab"]
    draft = build_gpu_model(binding, dcfg, seed + 7, n_ctx, torch.cuda.current_device())
    dec = SpeculativeDecoder(target, draft, n_draft=4, target_windows=bounds)
    dec.generate(0, n_ctx, 3)                                    # warm-up
    torch.cuda.synchronize()
    n_new = max(4, min(args.steps, 12))
    t0 = time.perf_counter()
    _, stats = dec.generate(0, n_ctx, n_new)
    torch.cuda.synchronize()
    total = time.perf_counter() - t0
    cycle_ms = total * 1e3 / stats.cycles
    draft.close()
    return {"draft": args.speculative + "-shaped random-init Q4_K", "n_draft": 4, "cycle_ms": cycle_ms, "cycles": stats.cycles,
            "measured_acceptance": stats.acceptance, "measured_tokens_per_s": sum(stats.per_cycle) / total,
            "tokens_per_s_if_k_confirmed_per_cycle": {str(k): (k + 1) * 1e3 / cycle_ms for k in range(5)},
            "timing": "wall clock around generate(); every step ends with a host read of the chosen tokens"}


# ------------------------------------------------------------------------------- the CPU checker arm
def cpu_baseline(workload: str, budget_s: float = 20.0, repeat: int = 1) -> dict:
    """Fallback sample of the CPU checker (used when the whole-token run is not possible: several requests, a
    truncated model, and for the per-step samples of the reference arm): one full-width layer at full context,
    scaled to the token by algorithmic bytes."""
    import oracle
    shape, n_ctx, _, _ = WORKLOADS[workload]
    cfg = synth.model_config(shape)
    seed = SEEDS[workload]
    cores = oracle.default_threads()
    one = dict(cfg, n_layers=1)
    mdl = oracle.Model(one, n_threads=cores)
    for layer, tid, rows, cols, data in synth.iter_model_tensors(seed, one, with_globals=False):
        mdl.load(layer, tid, data, rows, cols)
    k, v = synth.kv_prefill(seed, 0, n_ctx, cfg["n_kv_heads"], cfg["head_dim"])
    mdl.kv_load(0, 0, k, v)
    h0 = synth.activations(seed, 1, cfg["hidden"])
    times = []
    t_start = time.perf_counter()
    while len(times) < max(1, repeat) or (time.perf_counter() - t_start < budget_s * 0.5 and len(times) < 8):
        t0 = time.perf_counter()
        mdl.forward_window(0, 1, h0, n_ctx)
        times.append(time.perf_counter() - t0)
    mdl.close()
    bpt_layer = bytes_per_token(one, n_ctx, with_head=False)["total"]
    bpt_all = bytes_per_token(cfg, n_ctx)["total"]
    per_layer = float(np.median(times))
    return {"value": per_layer * 1e3 * bpt_all / bpt_layer, "unit": "ms/token", "cores": cores, "kind": "oracle",
            "sample": f"1 of {cfg['n_layers']} layers at full width and {n_ctx} cached positions, {len(times)} runs, median "
                      f"{per_layer * 1e3:.0f} ms per layer, scaled to the whole token by algorithmic bytes"}


def oracle_whole_token(workload: str, n_tok: int = 1) -> dict:
    """One whole token of the workload through the CPU checker, the model generated layer by layer (no GPU involved)."""
    shape, n_ctx, _, _ = WORKLOADS[workload]
    cfg = synth.model_config(shape)
    seed = SEEDS[workload]
    whole = WholeTokenOracle(cfg, seed, n_ctx, n_tok)
    for l in range(cfg["n_layers"]):
        tensors = {tid: (rows, cols, data) for _, tid, rows, cols, data in synth.iter_model_tensors(seed, cfg, layers=[l], with_globals=False)}
        k, v = synth.kv_prefill(seed, l, n_ctx, cfg["n_kv_heads"], cfg["head_dim"])
        whole.on_layer(l, tensors, k, v)
    whole.on_globals({tid: synth.tensor_shape(cfg, tid) + (synth.make_tensor(seed, cfg, -1, tid),) for tid in (synth.OUT_NORM, synth.W_HEAD)})
    return whole.result(n_tok)


def run_reference(args):
    """The reference arm: the CPU checker as it stands on the host cores.  One whole token is timed once (the value);
    every one of the --steps steps additionally times a bounded sample (one full-width layer, scaled by bytes), listed
    beside it to show the spread."""
    shape, n_ctx, n_windows, desc = WORKLOADS[args.workload]
    base = oracle_whole_token(args.workload)
    samples = [cpu_baseline(args.workload, budget_s=1.0)["value"] for _ in range(max(1, min(args.steps, 5)))]
    base["one_layer_samples_scaled_ms"] = samples
    v = base["value"]
    cfg = synth.model_config(shape)
    return {
        "impl": "reference", "metric": "decode_ms_per_token", "value": v, "unit": "ms/token", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": v, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": desc, "layers": cfg["n_layers"], "windows": n_windows, "n_ctx": n_ctx, "n_tok": 1},
        "cpu_baseline": base,
        "e2e": {"value": v, "unit": "ms/token", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def run_gemv_fmt(args):
    """Micro-benchmark of the single product in one of the other formats (not the headline): 70B-shaped matrices in
    standard layout, a ring of distinct matrices larger than L2 so that every launch reads from HBM."""
    import torch
    from paper_2504_08791_b200 import binding
    binding.lib()
    fmt = {"q6_k": synth.FMT_Q6_K, "q8_0": synth.FMT_Q8_0, "f16": synth.FMT_F16}[args.gemv_fmt]
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
    out = {"metric": "gemv_GBs", "format": args.gemv_fmt, "unit": "GB/s", "peak": peak, "shapes": {}}
    for rows, cols in ((8192, 8192), (8192, 28672)):
        nbytes = rows * cols // synth.FMT_BLOCK_WEIGHTS[fmt] * synth.FMT_BLOCK_BYTES[fmt]
        n_mats = max(2, int(400e6 // nbytes) + 1)
        mats = [torch.from_numpy(synth.fmt_tensor(20 + i, fmt, rows, cols)).cuda() for i in range(n_mats)]
        x = torch.from_numpy(synth.activations(20, 1, cols)).cuda()
        y = torch.empty((1, rows), dtype=torch.float32, device="cuda")
        try:
            for m in mats:
                binding.prima_gemv_fmt(fmt, m, rows, cols, x, 1, y)
        except binding.PrimaError as err:      # a row too long for the kernel's shared memory: the library says so
            out["shapes"][f"{rows}x{cols}"] = {"unsupported": str(err)}
            continue
        torch.cuda.synchronize()
        reps = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            for m in mats:
                binding.prima_gemv_fmt(fmt, m, rows, cols, x, 1, y)
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / (reps * n_mats)
        gbs = nbytes / (us * 1e-6) / 1e9
        out["shapes"][f"{rows}x{cols}"] = {"bytes": nbytes, "us": us, "GB/s": gbs, "frac_of_measured_peak": gbs / peak,
                                           "distinct_matrices": n_mats}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="70b", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (profiling captures)")
    ap.add_argument("--n-tok", type=int, default=1, help="tokens per step (speculative verification pass when > 1)")
    ap.add_argument("--ctx", type=int, default=0, help="override the KV context length (profiling captures)")
    ap.add_argument("--requests", type=int, default=1, help="concurrent requests per step, one token each, own KV caches")
    ap.add_argument("--speculative", default="", choices=["", "8b", "32b"],
                    help="also time speculative decoding cycles with a draft model of this shape")
    ap.add_argument("--repeats", type=int, default=5, help="how many times the timed region of --steps steps is taken (median reported)")
    ap.add_argument("--resident-layers", type=int, default=-1,
                    help="keep only the first N layers' matrices on the GPU, stream the others from pinned host memory every token")
    ap.add_argument("--stream-slots", type=int, default=0, help="device buffers for streamed layers (default 2)")
    ap.add_argument("--l2-ahead-mb", type=int, default=-1, help="MiB of the gate/up matrix asked into L2 during attention (default: the library's)")
    ap.add_argument("--l2-ahead-o-mb", type=int, default=-1, help="MiB more of it asked into L2 during the O product (default: the library's)")
    ap.add_argument("--gemv-fmt", default="", choices=["", "q6_k", "q8_0", "f16"],
                    help="micro-benchmark of the single product in another weight format instead of the decoding loop")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=20.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    if args.gemv_fmt:
        if rank == 0:
            print(json.dumps(run_gemv_fmt(args)), flush=True)
        return
    if args.warmup < 3:
        log("[bench] fewer than 3 warm-up steps: the number is not a valid measurement")
    res = run_ours(args, rank, world, local_rank)
    if rank == 0:
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
