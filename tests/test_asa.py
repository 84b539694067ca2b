"""Host logic of the adaptive scheduling algorithm (Section III-B; Algorithm 1, profiling / estimate / solve steps):
the exact solver against brute force, the cost model's limiting cases, and the plan for a ResNet-shaped layer list."""
import itertools

import numpy as np
import pytest

from paper_2503_23186_b200 import asa, workloads as wl


def _brute(time, memory, capacity):
    L, S = time.shape
    best, arg = np.inf, None
    for pick in itertools.product(range(S), repeat=L):
        m = sum(memory[i, s] for i, s in enumerate(pick))
        if m <= capacity:
            t = sum(time[i, s] for i, s in enumerate(pick))
            if t < best - 1e-12:
                best, arg = t, pick
    return arg, best


@pytest.mark.parametrize("seed", range(12))
def test_solver_equals_brute_force(seed):
    rng = np.random.default_rng(seed)
    L = int(rng.integers(2, 8))
    time = rng.uniform(0.1, 5.0, (L, 3))
    memory = rng.integers(1, 40, (L, 3)).astype(np.float64)        # whole units: the dynamic programme is exact
    # faster strategies tend to need more memory, so the constraint binds
    order = np.argsort(time, axis=1)
    memory = np.take_along_axis(np.sort(memory, axis=1)[:, ::-1], np.argsort(order, axis=1), axis=1)
    lo, hi = memory.min(axis=1).sum(), memory.max(axis=1).sum()
    for capacity in (lo, (lo + hi) / 2, hi, hi + 10):
        pick, best = _brute(time, memory, capacity)
        choice, total, used = asa.solve(time, memory, capacity, unit=1.0)
        assert abs(total - best) <= 1e-9 and used <= capacity + 1e-9
        assert abs(sum(time[i, s] for i, s in enumerate(choice)) - total) <= 1e-9
    with pytest.raises(ValueError):
        asa.solve(time, memory, lo - 1, unit=1.0)


def test_solver_rounds_memory_up_and_stays_feasible():
    time = np.array([[1.0, 2.0, 3.0], [1.0, 5.0, 2.0]])
    memory = np.array([[10.4, 5.2, 1.1], [7.7, 1.3, 3.9]])
    choice, total, used = asa.solve(time, memory, 12.0, unit=1.0)
    assert used <= 12.0
    assert (choice, total) == ([1, 2], 4.0) or total <= 4.0   # 10.4 + 7.7 does not fit; [1, 2] needs 9.1


def test_cost_model_limits():
    c = asa.Component("conv", 1.0, 2.0, param_bytes=4e6, act_bytes=64e6, state_bytes=16e6, saved_bytes=64e6)
    one = asa.Links(devices=1, bandwidth_gbs=700.0)
    for s in asa.STRATEGIES:
        assert asa.t_comm(c, s, one) == 0.0                       # a single device communicates nothing
        assert asa.mem(c, s, one) == pytest.approx(16e6 + 64e6)
    assert asa.t_comp(c, "DP", one) == pytest.approx(3.0)
    k8 = asa.Links(devices=8, bandwidth_gbs=700.0, latency_ms=0.0)
    # data parallel: 2 (K-1)/K of the gradient bytes over the link; model parallel: the same factor on the activations
    assert asa.t_comm(c, "DP", k8) == pytest.approx(2 * 4e6 * 7 / 8 / 700e6)
    assert asa.t_comm(c, "MP", k8) == pytest.approx(2 * 64e6 * 7 / 8 / 700e6)
    assert asa.t_comm(c, "DP", k8) < asa.t_comm(c, "HP", k8) < asa.t_comm(c, "MP", k8)   # few parameters, large activations
    assert asa.mem(c, "MP", k8) == pytest.approx(16e6 / 8 + 64e6) and asa.mem(c, "DP", k8) == pytest.approx(16e6 + 64e6 / 8)
    fc = asa.Component("fc", 0.1, 0.2, param_bytes=400e6, act_bytes=0.4e6, state_bytes=1600e6, saved_bytes=0.4e6)
    assert asa.t_comm(fc, "MP", k8) < asa.t_comm(fc, "HP", k8) < asa.t_comm(fc, "DP", k8)   # many parameters, small activations
    no_param = asa.Component("pool", 0.1, 0.1, 0.0, 1e6, 0.0, 1e6)
    assert asa.t_comm(no_param, "DP", k8) == 0.0
    # a slower link makes every exchange slower, never faster
    slow = asa.Links(devices=8, bandwidth_gbs=70.0, latency_ms=0.0)
    assert all(asa.t_comm(c, s, slow) > asa.t_comm(c, s, k8) for s in asa.STRATEGIES)


def test_plan_for_a_resnet_shaped_layer_list():
    spec = wl.resnet18_spec()
    n = len(spec)
    # a made-up but shaped profile: time proportional to the layer's multiply-adds (conv) or bytes (others)
    ms = np.zeros((n, 3))
    for i, L in enumerate(spec):
        if L["kind"] == "conv":
            flops = 2.0 * 1024 * (L["H"] // L["stride"]) ** 2 * L["K"] * L["R"] ** 2 * L["C"]
            ms[i] = [flops / 0.8e12, flops / 0.8e12, flops / 0.8e12]
        elif L["kind"] == "bn":
            b = 2.0 * 1024 * L["H"] * L["W"] * L["C"]
            ms[i] = [3 * b / 5e9, 0.0, 5 * b / 5e9]
    comps = asa.components_from_spec(spec, 1024, ms)
    assert len(comps) == n and sum(c.param_bytes for c in comps) / 4 == pytest.approx(11220132 - 0, rel=1e-3)   # the net's parameter count
    links = asa.Links(devices=8, bandwidth_gbs=700.0)
    roomy = asa.select_strategies(comps, links, 180e9)
    # with memory to spare, a small convolutional net is best run data parallel throughout, and no uniform plan beats the mix
    assert roomy["time_ms"] <= min(roomy["uniform_time_ms"].values()) + 1e-9
    assert roomy["strategy"].count("DP") >= n - 4
    dp_total = sum(asa.mem(c, "DP", links) for c in comps)
    min_total = sum(min(asa.mem(c, s, links) for s in asa.STRATEGIES) for c in comps)
    assert min_total < dp_total                                        # the wide late layers hold less state when split
    tight_cap = min_total + 0.3 * (dp_total - min_total)
    tight = asa.select_strategies(comps, links, tight_cap, unit=float(1 << 14))   # fine units: every entry is rounded up to one
    assert tight["memory_bytes"] <= tight_cap and tight["time_ms"] >= roomy["time_ms"] - 1e-9
    assert any(s != "DP" for s in tight["strategy"])                  # the constraint forces some components off DP
    with pytest.raises(ValueError):
        asa.select_strategies(comps, links, 1e6)


def test_reprofile_trigger():
    a = np.array([1.0, 2.0, 3.0])
    assert not asa.needs_reprofile(a, a * 1.05)
    assert asa.needs_reprofile(a, np.array([1.0, 2.0, 5.0]))
    assert asa.needs_reprofile(a, np.array([1.0, 2.0]))
