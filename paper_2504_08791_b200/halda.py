"""Layer-to-device assignment (LDA) and the Halda scheduler (paper Section 3.2, Definition 1, Eqs. 1-5; Section 3.3,
Algorithm 1; Appendix A.3, "Layer-to-Device Assignment: From Latency Analysis to Vectorized Model").

The scheduler decides, for a ring of M devices, the layer window w_m of every device and how many layers n_m of a
window run on its GPU, so that the modelled time per output token is smallest.  The model (Appendix A.3) adds, per
device, computation (FLOPs of a layer per format over the device's throughput for that format and backend), memory
access (KV append, hidden-state copies between RAM and VRAM once per window, and the bytes a layer has to bring
to the cores: weights b plus 2(h_k e_k + h_v e_v) n_kv bytes of KV cache), disk loading (what the OS has to
reload because the layers do not fit: four cases by OS and memory pressure, the sets M1..M4) and one hidden-state
message of 4e bytes per window.  With L = k W (every device gets k full windows) the objective is linear in
(w, n) for fixed k and fixed sets:

    T = k * sum_m (a_m w_m + b_m n_m + c_m) + kappa

and Halda (Algorithm 1) solves one small integer linear program per divisor k of L, re-derives the sets from the
solution, and repeats until the sets stop changing; if some GPU still has room while another device is
overloaded, the overloaded device with the slowest disk is forced into M4 (no overload allowed) and the problem is
solved again.  Devices that end up with at most one layer are dropped (device selection) and the rest is re-solved.

This module is host-side planning code (numpy + scipy's HiGHS-based `milp`, the solver family the paper names);
its output feeds `schedule.windows` / `ring.ring_step`, and, for a GPU whose share of the model exceeds its
memory, the residency budget of the window executor (layers that do not fit are streamed from pinned host memory).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

FORMATS = ("q4k", "q5k", "q6k", "q80", "fp16", "fp32")          # the set Q of Appendix A.3
MACOS_NO_METAL, MACOS_METAL, LINUX, ANDROID = "macos", "macos_metal", "linux", "android"
DISK_THRESHOLD = 50e6      # bytes/s: below this a device is never allowed to overload (Case 4, "low disk speed")


@dataclass
class ModelProfile:
    """What the model profiler reports (Appendix A.3): FLOPs per layer and of the output layer by format, bytes of a
    layer / the input table / the output layer, KV bytes per token and layer, context length, buffer sizes."""
    n_layers: int
    flops_layer: Dict[str, float]
    flops_out: Dict[str, float]
    b: float                    # weight bytes of one layer
    b_i: float                  # input (embedding) table bytes
    b_o: float                  # output layer bytes
    vocab: int
    kv_bytes_per_token: float   # 2 (h_k e_k + h_v e_v)
    n_kv: int
    hidden: int
    c_cpu: float = 0.0          # compute buffer in RAM
    c_gpu: float = 0.0          # compute buffer in VRAM / shared memory

    @property
    def b_prime(self) -> float:
        return self.b + self.kv_bytes_per_token * self.n_kv


@dataclass
class DeviceProfile:
    """What the device profiler reports for one device (Appendix A.3)."""
    name: str
    os: str = LINUX
    gpu: str = "none"                       # "none", "cuda", "metal"
    uma: bool = False
    s_cpu: Dict[str, float] = field(default_factory=dict)     # FLOPS by format
    s_gpu: Dict[str, float] = field(default_factory=dict)
    T_cpu: float = 1e10                     # bytes/s from RAM to the cores
    T_gpu: float = 1e11                     # bytes/s from VRAM to the cores
    t_kv_cpy_cpu: float = 0.0
    t_kv_cpy_gpu: float = 0.0
    t_ram_vram: float = 0.0
    t_vram_ram: float = 0.0
    t_comm: float = 0.0                     # 4e bytes to the next device
    s_disk: float = 1e9                     # bytes/s (random reads on macOS, sequential on Linux)
    d_avail: float = 0.0                    # available RAM
    d_avail_metal: float = 0.0              # Metal's recommended working set
    d_avail_cuda: float = 0.0               # free VRAM
    bytes_can_swap: float = 0.0             # Android
    swap_avail: float = 0.0

    @property
    def has_gpu(self) -> bool:
        return self.gpu in ("cuda", "metal")


def _sum_over_formats(flops: Dict[str, float], speed: Dict[str, float]) -> float:
    return sum(f / speed[q] for q, f in flops.items() if f)


def _b_cio(model: ModelProfile, m: int) -> float:
    return (model.b_i / model.vocab + model.b_o) * (m == 0) + model.c_cpu


def swapout(model: ModelProfile, dev: DeviceProfile, m: int, l_cpu: float) -> float:
    """d_m^swapout of an Android device that runs l_cpu layers on its CPU (Appendix A.3)."""
    if dev.os != ANDROID:
        return 0.0
    need = l_cpu * model.b + (model.b_i / model.vocab + model.b_o) * (m == 0) + model.kv_bytes_per_token * model.n_kv * l_cpu + model.c_cpu
    return min(max(0.0, need - dev.d_avail), min(dev.bytes_can_swap, dev.swap_avail))


# ------------------------------------------------------------------------------------- the latency model, written out
def device_layers(n_layers: int, w: Sequence[int], n: Sequence[int]) -> Tuple[List[int], List[int], List[int]]:
    """l_m, l_m^gpu and the number of windows W_m of every device (closed forms of Appendix A.3, any remainder R)."""
    from . import schedule
    return (schedule.layers_per_device(n_layers, w), schedule.gpu_layers_per_device(n_layers, w, n),
            schedule.windows_per_device(n_layers, w))


def tpot(model: ModelProfile, devices: Sequence[DeviceProfile], w: Sequence[int], n: Sequence[int]) -> float:
    """Modelled seconds per output token: the sum over devices of computation, memory access, disk loading and
    communication latency, each term as Appendix A.3 writes it (with its max operators; no set assignment needed)."""
    L = model.n_layers
    l, lg, nw = device_layers(L, w, n)
    kvb = model.kv_bytes_per_token * model.n_kv
    bio_head = model.b_i / model.vocab + model.b_o
    total = 0.0
    for m, d in enumerate(devices):
        head = m == 0
        l_cpu = l[m] - lg[m]
        comp = l_cpu * _sum_over_formats(model.flops_layer, d.s_cpu) if l_cpu else 0.0
        if lg[m]:
            comp += lg[m] * _sum_over_formats(model.flops_layer, d.s_gpu)
        if head:
            comp += _sum_over_formats(model.flops_out, d.s_cpu)
        mem = l_cpu * d.t_kv_cpy_cpu + lg[m] * d.t_kv_cpy_gpu
        if d.has_gpu:
            mem += nw[m] * (d.t_ram_vram + d.t_vram_ram) * (0 if d.uma else 1)
        mem += (l_cpu / d.T_cpu + (lg[m] / d.T_gpu if lg[m] else 0.0)) * (model.b + kvb) + (bio_head / d.T_cpu if head else 0.0)
        lookup = model.b_i / model.vocab if head else 0.0      # only the head reads the lookup table
        if d.os == MACOS_NO_METAL:
            disk = max(l[m] * model.b + bio_head * head + kvb * l[m] + model.c_cpu - d.d_avail, lookup) / d.s_disk
        elif d.os == MACOS_METAL:
            over = l[m] * model.b + bio_head * head + kvb * l[m] + model.c_cpu + model.c_gpu - d.d_avail_metal > 0
            disk = max((l[m] * model.b + bio_head * head) * over, lookup) / d.s_disk
        else:
            so = swapout(model, d, m, l_cpu)
            disk = max(l_cpu * (model.b + kvb) + bio_head * head + model.c_cpu - d.d_avail - so, lookup) / d.s_disk
        comm = nw[m] * d.t_comm
        total += comp + mem + disk + comm
    return total


# ------------------------------------------------------------------------------------------ sets and coefficients
def assign_sets(model: ModelProfile, devices: Sequence[DeviceProfile], w: Sequence[int], n: Sequence[int], k: int,
                forced_m4: Sequence[int] = ()) -> List[int]:
    """Case (1..4) of every device for the assignment (w, n) with k rounds (Appendix A.3, Cases 1-4)."""
    kvb = model.kv_bytes_per_token * model.n_kv
    sets = []
    for m, d in enumerate(devices):
        l_m, l_g = k * w[m], k * n[m]
        bio = (model.b_i / model.vocab + model.b_o) * (m == 0)
        fast_disk = d.s_disk > DISK_THRESHOLD
        case = 4
        if m not in forced_m4 and fast_disk:
            if d.os == MACOS_NO_METAL:
                if l_m * model.b + bio + kvb * l_m + model.c_cpu > d.d_avail:
                    case = 1
            elif d.os == MACOS_METAL:
                if l_m * model.b + bio + kvb * l_m + model.c_cpu + model.c_gpu > d.d_avail_metal:
                    case = 2
            else:
                if (l_m - l_g) * (model.b + kvb) + bio + model.c_cpu > d.d_avail + swapout(model, d, m, l_m - l_g):
                    case = 3
        sets.append(case)
    return sets


def coefficients(model: ModelProfile, devices: Sequence[DeviceProfile], sets: Sequence[int], w: Sequence[int], n: Sequence[int], k: int):
    """(a, b, c, kappa) of T = k * sum_m (a_m w_m + b_m n_m + c_m) + kappa for the given sets."""
    bp = model.b_prime
    a, b, c = [], [], []
    kappa = _sum_over_formats(model.flops_out, devices[0].s_cpu) + (model.b_i / model.vocab + model.b_o) / devices[0].T_cpu
    kappa += model.b_i / model.vocab / devices[0].s_disk + (model.b_o / devices[0].s_disk if sets[0] != 4 else 0.0)
    for m, d in enumerate(devices):
        alpha = _sum_over_formats(model.flops_layer, d.s_cpu) + d.t_kv_cpy_cpu + bp / d.T_cpu
        if d.has_gpu:
            beta = (_sum_over_formats(model.flops_layer, d.s_gpu) - _sum_over_formats(model.flops_layer, d.s_cpu)
                    + d.t_kv_cpy_gpu - d.t_kv_cpy_cpu + bp / d.T_gpu - bp / d.T_cpu)
            xi = (d.t_ram_vram + d.t_vram_ram) * (0 if d.uma else 1) + d.t_comm
        else:
            beta, xi = 0.0, d.t_comm
        s = sets[m]
        if s == 1:
            a.append(alpha + bp / d.s_disk); b.append(0.0)
        elif s == 2:
            a.append(alpha + model.b / d.s_disk); b.append(beta)
        elif s == 3:
            a.append(alpha + bp / d.s_disk); b.append(beta - bp / d.s_disk)
        else:
            a.append(alpha); b.append(beta)
        c.append(xi)
        if s in (1, 3):
            kappa += (model.c_cpu - d.d_avail - swapout(model, d, m, k * (w[m] - n[m]))) / d.s_disk
    return np.array(a), np.array(b), np.array(c), kappa


def _bounds(model: ModelProfile, devices: Sequence[DeviceProfile], sets: Sequence[int], w_cur: Sequence[int], n_cur: Sequence[int], k: int):
    """Per device: integer bounds (w_lo, w_hi, n_hi) and, for Linux / Android, a bound on w - n (lo, hi)."""
    bp, L = model.b_prime, model.n_layers
    out = []
    for m, d in enumerate(devices):
        w_lo, w_hi, n_hi, diff_lo, diff_hi = 1, L, L, None, None
        so = swapout(model, d, m, k * (w_cur[m] - n_cur[m]))
        x_ram = (d.d_avail + so - _b_cio(model, m)) / (k * bp)
        x_metal = (d.d_avail_metal - _b_cio(model, m) - model.c_gpu) / (k * bp)
        s = sets[m]
        if s == 1:
            w_lo = max(w_lo, math.floor(x_ram) + 1)
        elif s == 2:
            w_lo = max(w_lo, math.floor(x_metal) + 1)
        elif s == 3:
            diff_lo = math.floor(x_ram) + 1
        elif d.os == MACOS_NO_METAL:
            w_hi = min(w_hi, math.ceil(x_ram) - 1)
        elif d.os == MACOS_METAL:
            w_hi = min(w_hi, math.ceil(x_metal) - 1)
        else:
            diff_hi = math.ceil(x_ram) - 1
        if d.gpu == "cuda":
            n_hi = min(n_hi, math.floor((d.d_avail_cuda - model.c_gpu) / (k * bp)))
        elif d.gpu == "metal":
            n_hi = min(n_hi, math.floor((d.d_avail_metal - model.c_gpu - model.b_o * (m == 0)) / (k * bp)))
        else:
            n_hi = 0
        out.append((w_lo, w_hi, max(n_hi, 0), diff_lo, diff_hi))
    return out


def solve_ilp(model: ModelProfile, devices: Sequence[DeviceProfile], sets: Sequence[int], k: int, w_cur: Sequence[int],
              n_cur: Sequence[int]) -> Optional[Tuple[List[int], List[int], float]]:
    """The integer linear program for fixed k and sets (Section 3.3, "Transform into standard ILPs"): minimise
    k (a.w + b.n + e.c) + kappa  subject to  e.w = L / k, the memory conditions of the sets, the VRAM bounds and
    0 <= n_m <= w_m.  Returns (w, n, objective) or None when the program is infeasible."""
    from scipy.optimize import Bounds, LinearConstraint, milp
    M, L = len(devices), model.n_layers
    if L % k:
        return None
    W = L // k
    a, b, c, kappa = coefficients(model, devices, sets, w_cur, n_cur, k)
    bnd = _bounds(model, devices, sets, w_cur, n_cur, k)
    lo = np.array([x[0] for x in bnd] + [0] * M, float)
    hi = np.array([x[1] for x in bnd] + [x[2] for x in bnd], float)
    if np.any(lo > hi):
        return None
    rows, lb, ub = [np.concatenate([np.ones(M), np.zeros(M)])], [W], [W]
    for m in range(M):
        r = np.zeros(2 * M); r[m] = 1; r[M + m] = -1                    # w_m - n_m
        d_lo = 0 if bnd[m][3] is None else max(0, bnd[m][3])
        d_hi = L if bnd[m][4] is None else bnd[m][4]
        if d_lo > d_hi:
            return None
        rows.append(r); lb.append(d_lo); ub.append(d_hi)
    res = milp(c=k * np.concatenate([a, b]), constraints=LinearConstraint(np.array(rows), lb, ub), integrality=np.ones(2 * M),
               bounds=Bounds(lo, hi))
    if not res.success:
        return None
    x = np.rint(res.x).astype(int)
    w, n = x[:M].tolist(), x[M:].tolist()
    return w, n, float(k * (a @ x[:M] + b @ x[M:] + c.sum()) + kappa)


# ------------------------------------------------------------------------------------------------------- Algorithm 1
@dataclass
class Plan:
    w: List[int]
    n: List[int]
    k: int
    sets: List[int]
    objective: float            # the linearised objective of the last program solved
    tpot: float                 # the written-out model evaluated at (w, n)
    devices: List[str]          # names of the devices kept, in ring order
    iterations: int


def _initial_windows(model: ModelProfile, devices: Sequence[DeviceProfile]) -> List[int]:
    """w proportional to the devices' memory budgets, summing to L (k = 1)."""
    L = model.n_layers
    mem = np.array([(d.d_avail_metal if d.os == MACOS_METAL else d.d_avail + min(d.bytes_can_swap, d.swap_avail) * (d.os == ANDROID))
                    + (d.d_avail_cuda if d.gpu == "cuda" else 0.0) for d in devices], float)
    mem = np.maximum(mem, 1.0)
    w = np.maximum(1, np.floor(L * mem / mem.sum()).astype(int))
    while w.sum() > L:
        w[int(np.argmax(w))] -= 1
    while w.sum() < L:
        w[int(np.argmax(mem / w))] += 1
    return w.tolist()


def _solve_all_k(model, devices, sets, w, n):
    best = None
    for k in [f for f in range(1, model.n_layers) if model.n_layers % f == 0]:      # the valid factors of L, excluding L
        if model.n_layers // k < len(devices):
            continue                                                                 # every device needs at least one layer
        sol = solve_ilp(model, devices, sets, k, w, n)
        if sol and (best is None or sol[2] < best[3]):
            best = (sol[0], sol[1], k, sol[2])
    return best


def halda_fixed_devices(model: ModelProfile, devices: Sequence[DeviceProfile], max_iter: int = 64) -> Optional[Plan]:
    """Algorithm 1 on a fixed ring of devices."""
    M = len(devices)
    if M == 1:
        d = devices[0]
        n_fit = 0
        if d.gpu == "cuda":
            n_fit = max(0, min(model.n_layers, math.floor((d.d_avail_cuda - model.c_gpu) / model.b_prime)))
        elif d.gpu == "metal":
            n_fit = max(0, min(model.n_layers, math.floor((d.d_avail_metal - model.c_gpu - model.b_o) / model.b_prime)))
        w, n = [model.n_layers], [n_fit]
        return Plan(w, n, 1, assign_sets(model, devices, w, n, 1), tpot(model, devices, w, n), tpot(model, devices, w, n), [d.name], 0)
    if M > model.n_layers:
        return None
    w, n = _initial_windows(model, devices), [0] * M
    forced: List[int] = []
    sets_prev: Optional[List[int]] = None
    best = None
    for it in range(1, max_iter + 1):
        W = sum(w)
        k = max(1, model.n_layers // W)
        sets = assign_sets(model, devices, w, n, k, forced)
        if sets == sets_prev and best is not None:
            return Plan(best[0], best[1], best[2], sets, best[3], tpot(model, devices, best[0], best[1]), [d.name for d in devices], it)
        sets_prev = sets
        sol = _solve_all_k(model, devices, sets, w, n)
        if sol is None:
            # the sets derived from the current point admit no feasible program: forbid overloading on the device with the slowest disk
            cand = [m for m in range(M) if sets[m] != 4 and m not in forced]
            if not cand:
                return None
            forced.append(min(cand, key=lambda m: devices[m].s_disk))
            sets_prev = None
            continue
        best = sol
        w_s, n_s, k_s, _ = sol
        # calibration: some GPU could host more layers (its VRAM is not full) while some device is overloaded
        n_hi = [x[2] for x in _bounds(model, devices, sets, w_s, n_s, k_s)]
        room = [m for m, d in enumerate(devices) if d.has_gpu and n_s[m] < min(n_hi[m], model.n_layers // k_s)]
        overloaded = [m for m in range(M) if sets[m] != 4]
        if room and overloaded:
            forced.append(min(overloaded, key=lambda m: devices[m].s_disk))
            sets_prev = None
            continue
        w, n = w_s, n_s
    return Plan(best[0], best[1], best[2], sets_prev or [], best[3], tpot(model, devices, best[0], best[1]), [d.name for d in devices], max_iter) if best else None


def halda(model: ModelProfile, devices: Sequence[DeviceProfile], keep: Sequence[str] = ()) -> Plan:
    """Halda with device selection: solve, drop the devices that got at most one layer (never the head, never one named
    in `keep`, e.g. a relay the ring cannot do without), solve again, and keep the better plan."""
    devs = list(devices)
    plan = halda_fixed_devices(model, devs)
    while plan is not None and len(devs) > 1:
        weak = [m for m in range(1, len(devs)) if plan.k * plan.w[m] <= 1 and devs[m].name not in keep]
        if not weak:
            break
        trial_devs = [d for m, d in enumerate(devs) if m not in weak]
        trial = halda_fixed_devices(model, trial_devs)
        if trial is None or trial.tpot > plan.tpot:
            break
        devs, plan = trial_devs, trial
    if plan is None:
        raise ValueError("no feasible assignment: the devices cannot hold the model under the model's constraints")
    return plan


def ring_windows(plan: Plan, n_layers: int):
    """The plan as `schedule.windows` input: window sizes per device, in ring order."""
    from . import schedule
    return schedule.windows(n_layers, plan.w)
