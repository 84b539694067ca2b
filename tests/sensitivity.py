"""How far the free-running results of one training step move when single bf16 roundings fall the other way.

The CUDA path accumulates in fp32 in an unspecified order, the oracle in fp64: for a small share of the stored bf16
elements the two sums lie on opposite sides of a rounding boundary and are stored one bf16 step apart.  Both results are
correct.  This module reruns the ORACLE with such flips injected at its storage points (a seeded random share of the
elements of a tensor takes the neighbouring bf16 value on the other side of the exact result) and measures, per
parameter tensor, how far the gradient sum, the updated parameters and the loss move.  The share per kind of tensor is
what the teacher-forced comparison of the library against the oracle shows (elements that differ at all on identical
inputs).  The spread is the yardstick for the free-running gates of tests/test_gpu_net.py."""
import numpy as np

import oracle
from oracle import net as onet

# Share of stored elements that differ between the library and the oracle on identical inputs, per kind of storage
# point (largest value seen over the layers of the ResNet-18-shaped net, rounded up): convolution outputs 2e-4..1.2e-3,
# data gradients up to 2.1e-3, BatchNorm outputs up to 3e-5, BatchNorm input gradients up to 6.5e-5, the rest 0.
DEFAULT_RATES = {"conv": 1.5e-3, "conv_dgrad": 2.5e-3, "bn": 5e-5, "bn_bwd": 1e-4}
KIND_OF_ROW = {" fwd": None, " dgrad": "conv_dgrad", " bwd dy": "bn_bwd"}   # suffixes of netcheck report rows


def flipping_round(rates, seed):
    """A stand-in for the oracle's bf16 rounding: round to nearest even, then move a random share rates[site] of the
    elements to the bf16 neighbour on the other side of the exact value."""
    rng = np.random.default_rng(seed)

    def f(x, site):
        x = np.asarray(x, np.float64)
        r = oracle.round_bf16(x)
        p = rates.get(site, 0.0)
        if p <= 0.0:
            return r
        pick = (rng.random(r.shape) < p) & (r != x)
        if not pick.any():
            return r
        with np.errstate(divide="ignore"):
            ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(r), 1e-300))) - 7.0)   # bf16 spacing in r's binade
        other = oracle.round_bf16(np.where(r > x, r - ulp, r + ulp))
        return np.where(pick, other, r)

    return f


def rel_fro(a, b):
    a, b = np.asarray(a, np.float64).reshape(-1), np.asarray(b, np.float64).reshape(-1)
    nb = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / nb) if nb > 0 else float(np.linalg.norm(a))


def step_spread(spec, params, velocity, images, labels, n_micro, lr, mu, wd, rates=None, seeds=(1, 2, 3), ref=None):
    """Reference step (plain rounding) and the largest deviation from it over `seeds` flipped reruns.
    Returns (ref, {"grads": {name: relF}, "params": {name: relF}, "loss": rel})."""
    rates = DEFAULT_RATES if rates is None else rates
    if ref is None:
        ref = onet.train_step(spec, params, velocity, images, labels, n_micro, lr, mu, wd, rounding=True)
    spread = {"grads": {k: 0.0 for k in params}, "params": {k: 0.0 for k in params}, "loss": 0.0}
    for seed in seeds:
        run = onet.train_step(spec, params, velocity, images, labels, n_micro, lr, mu, wd, rounding=flipping_round(rates, seed))
        for k in params:
            spread["grads"][k] = max(spread["grads"][k], rel_fro(run["grads"][k], ref["grads"][k]))
            spread["params"][k] = max(spread["params"][k], rel_fro(run["params"][k], ref["params"][k]))
        spread["loss"] = max(spread["loss"], abs(run["loss"] - ref["loss"]) / abs(ref["loss"]))
    return ref, spread


def rates_from_report(rep, floor=None):
    """Flip shares per kind of storage point from a teacher-forced netcheck report of the library (largest over layers)."""
    rates = dict(floor or {})
    for name, share in rep.differ.items():
        if name.endswith(" fwd") and "bn" not in name and not name.startswith(("fc", "pool")):
            kind = "conv"
        elif name.endswith(" fwd") and "bn" in name:
            kind = "bn"
        elif name.endswith(" dgrad") and not name.startswith("fc"):
            kind = "conv_dgrad"
        elif name.endswith(" bwd dy"):
            kind = "bn_bwd"
        else:
            continue
        rates[kind] = max(rates.get(kind, 0.0), share)
    return rates
