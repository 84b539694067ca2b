"""Host logic of the paper's adaptive scheduling algorithm (Section III-B, Algorithm 1): partition the model into
components, profile each component's execution time, estimate the communication overhead of every component under
each parallelism strategy from the sizes of its activations and gradients, and solve the selection problem

    minimise   sum_i  t_comp(c_i, s_i) + t_comm(c_i, s_i)        over s_i in {DP, MP, HP}
    subject to sum_i  mem(c_i, s_i) <= M   on every device,

exactly.  (The objective is printed in the paper as a `max` over a single term, which has nothing to maximise over; it
is read here as the sum of per-component computation plus communication time, the "overall training time" of step 4
of Section III-B.  All devices are alike, so the per-device memory constraints collapse into one.)

The components are the layers of a layer list (`workloads` format), the profile comes from the library's per-layer
timing (`binding.Net.profile_read_layers`), the strategies' costs from a bandwidth / latency model of the links.  This
module only decides; executing a layer model-parallel is outside the training-step library, which runs the per-replica
step every strategy has in common.  Pure host code, numpy only.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Sequence

import numpy as np

STRATEGIES = ("DP", "MP", "HP")
BYTES_PER_PARAM_STATE = 16.0   # fp32 master, momentum and gradient sum, two bf16 copies


@dataclass
class Component:
    """One logical component c_i: measured single-device times (ms) and sizes (bytes) of one training step."""
    name: str
    t_fwd_ms: float
    t_bwd_ms: float
    param_bytes: float          # fp32 gradient bytes exchanged by data-parallel replicas
    act_bytes: float            # bf16 output activation of the whole batch (its gradient has the same size)
    state_bytes: float          # parameter state held for the component (BYTES_PER_PARAM_STATE per parameter)
    saved_bytes: float          # activations kept for the backward pass (output, mask)


@dataclass
class Links:
    """Device count and link model: a transfer of n bytes between peers costs latency_ms + n / bandwidth."""
    devices: int
    bandwidth_gbs: float        # per direction per device
    latency_ms: float = 0.005
    hp_group: int = 2           # devices that split one replica's layer under HP (data parallel across the groups)
    mp_efficiency: float = 0.85  # fraction of the ideal 1/K compute scaling a layer split across devices reaches


def components_from_spec(spec, batch: int, layer_ms: np.ndarray) -> List[Component]:
    """Partition = the layer list (Algorithm 1, "Partition model M into L logical components").  layer_ms[i] =
    (forward, parameter-gradient, data-gradient) milliseconds of layer i for one step of `batch` images."""
    comps = []
    for i, L in enumerate(spec):
        k = L["kind"]
        fwd, wg, dg = (float(v) for v in layer_ms[i])
        params = act = 0.0
        if k == "conv":
            P, Q = L["H"] // L["stride"], L["W"] // L["stride"]
            params = L["K"] * L["R"] * L["R"] * L["C"]
            act = 2.0 * batch * P * Q * L["K"]
        elif k == "bn":
            params = 2.0 * L["C"]
            act = 2.0 * batch * L["H"] * L["W"] * L["C"]
        elif k == "fc":
            params = L["K"] * L["C"] + L["K"]
            act = 4.0 * batch * L["K"]
        elif k == "avgpool":
            act = 2.0 * batch * L["C"]
        saved = act * (1.0 + (1.0 / 16.0 if k == "bn" and L.get("relu") else 0.0))
        comps.append(Component(L.get("name", f"{k}{i}"), fwd, wg + dg, 4.0 * params, act, BYTES_PER_PARAM_STATE * params, saved))
    return comps


def _xfer_ms(n_bytes: float, links: Links) -> float:
    return 0.0 if n_bytes <= 0 else links.latency_ms + n_bytes / (links.bandwidth_gbs * 1e6)


def t_comp(c: Component, s: str, links: Links) -> float:
    """Computation time of the component per step on one device under strategy s (the global batch is fixed)."""
    K = links.devices
    t = c.t_fwd_ms + c.t_bwd_ms
    if s == "DP":
        return t / K                                   # each replica takes 1/K of the images
    if s == "MP":
        return t / (K * links.mp_efficiency)           # the layer is split K ways
    m = min(links.hp_group, K)
    return t / (K * (1.0 - (1.0 - links.mp_efficiency) * (m - 1) / max(K - 1, 1)))


def t_comm(c: Component, s: str, links: Links) -> float:
    """Communication overhead per step (Section III-B step 3: from the sizes of activations and gradients).
    DP: ring reduce-scatter + all-gather of the gradients, 2 (K-1)/K of the bytes through every link.
    MP: the split layer's output is all-gathered in the forward pass and its gradient reduce-scattered in the
        backward pass, (K-1)/K of the activation bytes each way; no gradient exchange (every device owns its slice).
    HP: groups of hp_group devices split the layer, the groups are data-parallel replicas of one another."""
    K = links.devices
    if K <= 1:
        return 0.0
    if s == "DP":
        return 2.0 * _xfer_ms(c.param_bytes * (K - 1) / K, links) if c.param_bytes > 0 else 0.0
    if s == "MP":
        return 2.0 * _xfer_ms(c.act_bytes * (K - 1) / K, links)
    m = max(1, min(links.hp_group, K))
    r = K // m                                          # replicas (groups)
    t = 0.0
    if m > 1:
        t += 2.0 * _xfer_ms(c.act_bytes / r * (m - 1) / m, links)
    if r > 1 and c.param_bytes > 0:
        t += 2.0 * _xfer_ms(c.param_bytes / m * (r - 1) / r, links)
    return t


def mem(c: Component, s: str, links: Links) -> float:
    """Bytes the component occupies on one device: parameter state (replicated under DP, split under MP) plus the
    activations kept for the backward pass (split over the replicas' shares of the batch)."""
    K = links.devices
    if s == "DP":
        return c.state_bytes + c.saved_bytes / K
    if s == "MP":
        return c.state_bytes / K + c.saved_bytes       # every device holds the gathered output of all images
    m = max(1, min(links.hp_group, K))
    return c.state_bytes / m + c.saved_bytes / (K // m)


def cost_tables(comps: Sequence[Component], links: Links):
    """time[i, s] = t_comp + t_comm (ms), memory[i, s] (bytes) for every component and strategy."""
    time = np.array([[t_comp(c, s, links) + t_comm(c, s, links) for s in STRATEGIES] for c in comps])
    memory = np.array([[mem(c, s, links) for s in STRATEGIES] for c in comps])
    return time, memory


def solve(time: np.ndarray, memory: np.ndarray, capacity: float, unit: float = float(1 << 20)):
    """Exact solution of the selection problem (a multiple-choice knapsack) by dynamic programming over the memory used.
    Memory is counted in whole `unit`s, each entry rounded up, so the returned assignment always fits `capacity`; with
    entries that are multiples of `unit` the optimum is exact.  Returns (choice index per component, total time,
    total memory in bytes).  Raises ValueError if no assignment fits."""
    time = np.asarray(time, np.float64)
    L, S = time.shape
    need = np.ceil(np.asarray(memory, np.float64) / unit - 1e-9).astype(np.int64)
    cap = int(np.floor(capacity / unit + 1e-9))
    if cap < 0 or int(need.min(axis=1).sum()) > cap:
        raise ValueError("no strategy assignment fits the device memory")
    cap = min(cap, int(need.max(axis=1).sum()))          # more than the largest total is never used
    INF = np.inf
    best = np.full(cap + 1, INF)
    best[0] = 0.0
    pick = np.zeros((L, cap + 1), np.int8)
    for i in range(L):
        nxt = np.full(cap + 1, INF)
        arg = np.zeros(cap + 1, np.int8)
        for s in range(S):
            w = int(need[i, s])
            if w > cap:
                continue
            cand = np.full(cap + 1, INF)
            cand[w:] = best[:cap + 1 - w] + time[i, s]
            better = cand < nxt
            nxt = np.where(better, cand, nxt)
            arg = np.where(better, s, arg).astype(np.int8)
        best, pick[i] = nxt, arg
    u = int(np.argmin(best))
    if not np.isfinite(best[u]):
        raise ValueError("no strategy assignment fits the device memory")
    total = float(best[u])
    choice = [0] * L
    for i in range(L - 1, -1, -1):
        s = int(pick[i, u])
        choice[i] = s
        u -= int(need[i, s])
    used = float(sum(memory[i, choice[i]] for i in range(L)))
    return choice, total, used


def select_strategies(comps: Sequence[Component], links: Links, device_memory_bytes: float, unit: float = float(1 << 20)) -> Dict:
    """Steps 3-5 of Section III-B for one profile: cost model, exact selection, the plan to apply."""
    time, memory = cost_tables(comps, links)
    choice, total, used = solve(time, memory, device_memory_bytes, unit)
    per_strategy = {s: float(time[:, j].sum()) for j, s in enumerate(STRATEGIES)}
    return {"strategy": [STRATEGIES[j] for j in choice], "time_ms": total, "memory_bytes": used, "uniform_time_ms": per_strategy,
            "comm_share": float(sum(t_comm(c, STRATEGIES[j], links) for c, j in zip(comps, choice)) / total) if total > 0 else 0.0}


def needs_reprofile(old_ms: np.ndarray, new_ms: np.ndarray, threshold: float = 0.15) -> bool:
    """Algorithm 1, "if communication patterns changed significantly: re-profile and update strategy".  The paper gives
    no threshold; here: the per-component times moved by more than `threshold` of the step in total variation."""
    a, b = np.asarray(old_ms, np.float64).reshape(-1), np.asarray(new_ms, np.float64).reshape(-1)
    if a.shape != b.shape:
        return True
    denom = max(a.sum(), 1e-12)
    return float(np.abs(a - b).sum() / denom) > threshold


def profile_components(net, images, labels, n_micro: int, lr: float, momentum: float, wd: float, steps: int = 5) -> np.ndarray:
    """The profiling phase (Algorithm 1, "Profile execution time t_comp(c_i) for each component"): runs `steps` training
    steps with per-launch timing on and returns the mean (forward, parameter-gradient, data-gradient) milliseconds per
    layer.  `net` is a `binding.Net`; the parameters advance by `steps` updates."""
    net.profile_enable(True)
    for _ in range(steps):
        net.train_step(images, labels, n_micro, lr, momentum, wd, update=True)
    ms = net.profile_read_layers() / steps
    net.profile_read()
    net.profile_enable(False)
    return ms
