"""Halda and the layer-to-device assignment model (paper Section 3.2-3.3, Algorithm 1; Appendix A.3) on synthetic device
profiles: the linearised objective against the written-out latency model, each integer program against brute force,
the whole scheduler against exhaustive search on tiny instances, and the behaviours the paper reports (a small model
goes to the head's GPU alone, equal devices tie, weak devices are dropped)."""
import itertools

import numpy as np
import pytest

from paper_2504_08791_b200 import halda as H
from paper_2504_08791_b200 import schedule


def model(L=32, b=122.7e6, n_kv=1024, b_o=431e6):
    return H.ModelProfile(n_layers=L, flops_layer={"q4k": 2 * b / 0.5625, "fp32": 2e6}, flops_out={"q6k": 2 * 525e6}, b=b, b_i=295e6, b_o=b_o,
                          vocab=128256, kv_bytes_per_token=4096, n_kv=n_kv, hidden=4096, c_cpu=300e6, c_gpu=300e6)


def cpu(name, gflops, ram, disk, os=H.LINUX, comm=2e-3, **kw):
    return H.DeviceProfile(name=name, os=os, s_cpu={q: gflops * 1e9 for q in H.FORMATS}, T_cpu=20e9, s_disk=disk, d_avail=ram, t_comm=comm,
                           t_kv_cpy_cpu=2e-6, **kw)


def gpu(name, gf_cpu, gf_gpu, ram, vram, disk, comm=2e-3, kind="cuda", os=H.LINUX, **kw):
    return H.DeviceProfile(name=name, os=os, gpu=kind, uma=kind == "metal", s_cpu={q: gf_cpu * 1e9 for q in H.FORMATS},
                           s_gpu={q: gf_gpu * 1e9 for q in H.FORMATS}, T_cpu=20e9, T_gpu=400e9, s_disk=disk, d_avail=ram, d_avail_cuda=vram,
                           t_comm=comm, t_kv_cpy_cpu=2e-6, t_kv_cpy_gpu=4e-6, t_ram_vram=2e-5, t_vram_ram=2e-5, **kw)


def home_cluster():
    """Four devices in the spirit of the paper's testbed: a desktop with a mid-range GPU (head), a Mac without Metal, a laptop
    with a small GPU, a phone."""
    return [gpu("desktop", 200, 8000, 8e9, 11e9, 2e9), cpu("mac", 100, 8e9, 0.7e9, os=H.MACOS_NO_METAL), gpu("laptop", 150, 5000, 8e9, 8e9, 1.5e9),
            cpu("phone", 50, 4e9, 0.4e9, os=H.ANDROID, bytes_can_swap=1e9, swap_avail=2e9)]


def big_model():
    return model(L=80, b=481e6, b_o=862e6)


# ------------------------------------------------------------------------------------------------ model consistency
@pytest.mark.parametrize("mdl,devs", [(model(), home_cluster()), (big_model(), home_cluster()),
                                      (big_model(), [gpu("a", 100, 4000, 16e9, 24e9, 3e9), gpu("b", 100, 4000, 16e9, 24e9, 3e9)]),
                                      (model(L=48, b=300e6), [gpu("m", 120, 3000, 8e9, 0, 2e9, kind="metal", os=H.MACOS_METAL, d_avail_metal=10e9),
                                                              cpu("l", 80, 6e9, 1e9)])])
def test_linearised_objective_equals_the_written_out_model_at_the_plan(mdl, devs):
    plan = H.halda_fixed_devices(mdl, devs)
    assert plan is not None
    assert sum(plan.w) * plan.k == mdl.n_layers and all(0 <= n <= w for w, n in zip(plan.w, plan.n))
    sets = H.assign_sets(mdl, devs, plan.w, plan.n, plan.k)
    a, b, c, kappa = H.coefficients(mdl, devs, sets, plan.w, plan.n, plan.k)
    lin = plan.k * (a @ np.array(plan.w) + b @ np.array(plan.n) + c.sum()) + kappa
    assert abs(lin - H.tpot(mdl, devs, plan.w, plan.n)) <= 1e-9 * lin


def test_written_out_model_term_by_term_on_a_two_device_example():
    # one CPU-only Linux head with plenty of RAM and one CUDA device that holds its layers in VRAM: no disk term but the lookup
    mdl = model(L=4, b=100e6, n_kv=0, b_o=50e6)
    head = cpu("h", 10, 1e12, 1e9, comm=1e-3)
    dev = gpu("g", 10, 100, 1e12, 1e12, 1e9, comm=3e-3)
    w, n = [1, 1], [0, 1]                       # k = 2 rounds: two layers each
    f = sum(mdl.flops_layer.values())
    want = (2 * f / 10e9 + 2 * 525e6 / 10e9                       # head: two CPU layers + the output layer
            + 2 * 2e-6 + 2 * 100e6 / 20e9 + (295e6 / 128256 + 50e6) / 20e9 + (295e6 / 128256) / 1e9 + 2 * 1e-3
            + 2 * f / 100e9 + 2 * 4e-6 + 2 * (2e-5 + 2e-5) + 2 * 100e6 / 400e9 + 2 * 3e-3)
    assert abs(H.tpot(mdl, [head, dev], w, n) - want) < 1e-12
    assert H.device_layers(4, w, n) == ([2, 2], [0, 2], [2, 2])


# ------------------------------------------------------------------------------------- integer programs vs brute force
def _feasible(mdl, devs, sets, k, w, n):
    bnd = H._bounds(mdl, devs, sets, w, n, k)
    for m in range(len(devs)):
        w_lo, w_hi, n_hi, d_lo, d_hi = bnd[m]
        if not (w_lo <= w[m] <= w_hi and 0 <= n[m] <= min(n_hi, w[m])):
            return False
        if d_lo is not None and w[m] - n[m] < d_lo:
            return False
        if d_hi is not None and w[m] - n[m] > d_hi:
            return False
    return True


@pytest.mark.parametrize("k", [1, 2, 3])
def test_integer_program_matches_exhaustive_search(k):
    mdl = model(L=12, b=600e6, n_kv=2048)
    devs = [gpu("a", 100, 3000, 2.5e9, 2.6e9, 2e9), cpu("b", 60, 2e9, 1e9), gpu("c", 80, 1500, 1.5e9, 1.4e9, 0.5e9)]
    W = 12 // k
    for sets in ([4, 4, 4], [3, 4, 3], [3, 3, 4], [4, 3, 3]):
        ref = [1, 1, 1]                          # swapout is zero here (no Android), so the reference point does not matter
        best = None
        for w in itertools.product(range(1, W + 1), repeat=3):
            if sum(w) != W:
                continue
            for n in itertools.product(*[range(0, wi + 1) for wi in w]):
                if _feasible(mdl, devs, sets, k, w, n):
                    a, b, c, kappa = H.coefficients(mdl, devs, sets, ref, [0, 0, 0], k)
                    obj = k * (a @ np.array(w) + b @ np.array(n) + c.sum()) + kappa
                    if best is None or obj < best - 1e-15:
                        best = obj
        got = H.solve_ilp(mdl, devs, sets, k, ref, [0, 0, 0])
        if best is None:
            assert got is None
        else:
            assert got is not None and abs(got[2] - best) <= 1e-9 * abs(best)
            assert _feasible(mdl, devs, sets, k, got[0], got[1])


def _exhaustive_tpot(mdl, devs):
    L, M = mdl.n_layers, len(devs)
    best = None
    for k in [f for f in range(1, L) if L % f == 0]:
        W = L // k
        for w in itertools.product(range(1, W + 1), repeat=M):
            if sum(w) != W:
                continue
            n_hi = [x[2] for x in H._bounds(mdl, devs, [4] * M, w, [0] * M, k)]
            for n in itertools.product(*[range(0, min(wi, nh) + 1) for wi, nh in zip(w, n_hi)]):
                t = H.tpot(mdl, devs, w, n)
                if best is None or t < best[0]:
                    best = (t, w, n, k)
    return best


def test_scheduler_against_exhaustive_search_on_tiny_rings():
    mdl = model(L=12, b=600e6, n_kv=2048)
    for devs in ([gpu("a", 100, 3000, 2.5e9, 2.6e9, 2e9), cpu("b", 60, 2e9, 1e9), gpu("c", 80, 1500, 1.5e9, 1.4e9, 0.5e9)],
                 [gpu("a", 100, 3000, 9e9, 9e9, 2e9), gpu("b", 100, 3000, 9e9, 9e9, 2e9)],
                 [cpu("a", 100, 3e9, 2e9), cpu("b", 100, 3e9, 0.3e9), cpu("c", 30, 3e9, 2e9)]):
        plan = H.halda_fixed_devices(mdl, devs)
        opt = _exhaustive_tpot(mdl, devs)
        assert plan is not None and plan.tpot >= opt[0] * (1 - 1e-12)
        # the iteration over set assignments is a heuristic: it must come close to the exhaustive optimum of the written-out model
        assert plan.tpot <= 1.10 * opt[0], (plan, opt)
        # and it must beat the memory-proportional partition it starts from
        w0 = H._initial_windows(mdl, devs)
        assert plan.tpot <= H.tpot(mdl, devs, w0, [0] * len(devs)) * (1 + 1e-12)


# ------------------------------------------------------------------------------------------ behaviours the paper reports
def test_a_model_that_fits_one_gpu_goes_to_the_head_gpu_alone():
    plan = H.halda(model(), home_cluster())                      # 8B-sized: 32 layers of 123 MB fit the desktop's 11 GB of VRAM
    assert plan.devices == ["desktop"] and plan.w == [32] and plan.n == [32]


def test_equal_devices_tie_and_weak_devices_are_dropped():
    mdl = big_model()
    twins = [gpu("a", 100, 4000, 16e9, 24e9, 3e9), gpu("b", 100, 4000, 16e9, 24e9, 3e9)]
    plan = H.halda(mdl, twins)
    # the objective is a SUM of the devices' latencies (Appendix A.3 explains why not the maximum), so between equal devices
    # every split that keeps all layers in VRAM costs the same: the plan must be as good as the even split, all on the GPUs
    assert sum(plan.w) * plan.k == 80 and plan.n == plan.w
    assert plan.tpot <= H.tpot(mdl, twins, [40, 40], [40, 40]) * (1 + 1e-12)
    plan = H.halda(mdl, home_cluster())
    assert "phone" not in plan.devices and plan.devices[0] == "desktop"
    assert plan.tpot < H.tpot(mdl, home_cluster(), H._initial_windows(mdl, home_cluster()), [0, 0, 0, 0])
    # a relay the ring cannot do without is kept even if it gets a single layer
    kept = H.halda(mdl, home_cluster(), keep=("phone",))
    assert "phone" in kept.devices


def test_gpu_layers_respect_vram_and_m4_devices_are_not_overloaded():
    mdl, devs = big_model(), home_cluster()[:3]
    plan = H.halda_fixed_devices(mdl, devs)
    for m, d in enumerate(devs):
        if d.gpu == "cuda":
            assert plan.k * plan.n[m] * mdl.b_prime + mdl.c_gpu <= d.d_avail_cuda
        else:
            assert plan.n[m] == 0
        if plan.sets[m] == 4 and d.os == H.LINUX:
            assert plan.k * (plan.w[m] - plan.n[m]) * mdl.b_prime + H._b_cio(mdl, m) < d.d_avail
    ws = H.ring_windows(plan, mdl.n_layers)
    assert [w.layer_end - w.layer_begin for w in ws[:len(devs)]] == plan.w and schedule.rounds(80, plan.w) == plan.k


def test_no_feasible_assignment_is_reported():
    mdl = model(L=3)
    with pytest.raises(ValueError):
        H.halda(mdl, [cpu("a", 1, 1e9, 1e6), cpu("b", 1, 1e9, 1e6), cpu("c", 1, 1e9, 1e6), cpu("d", 1, 1e9, 1e6)])      # more devices than layers
