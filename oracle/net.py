"""Oracle network runner: the inner loop of Algorithm 1 over a layer list, in fp64.

TEST INFRASTRUCTURE ONLY.  For each micro-batch (a data-parallel replica's share): forward
pass, loss, backward pass; then the replicas' gradients are averaged and one SGD-momentum
update is applied.  BatchNorm statistics are taken per micro-batch, as each data-parallel
replica sees only its own share of the data.

``rounding=True`` rounds every tensor at the point where the library stores it (bf16 for
activations and activation gradients, fp32 for logits and BN statistics) so that the
comparison isolates kernel errors from storage-format errors; ``rounding=False`` is the
never-rounding definition used for the finite-difference pins.
"""
from __future__ import annotations

import numpy as np

from . import (avgpool_bwd, avgpool_fwd, bn_relu_apply, bn_relu_bwd, bn_stats, conv2d_dgrad, conv2d_fwd,
               conv2d_wgrad, round_bf16, round_f32, sgd_momentum, softmax_xent)

BN_EPS = 1e-5


def _rb(x, rounding, site=None):
    """bf16 storage point.  ``rounding`` may also be a callable ``f(x, site)`` standing in for the bf16 rounding at the
    named storage point (the tests use it to study how sensitive the step is to which way single roundings fall)."""
    if callable(rounding):
        return rounding(x, site)
    return round_bf16(x) if rounding else x


def _rf(x, rounding):
    return round_f32(x) if rounding else x


def forward(spec, params, images, labels, rounding=True, grad_scale=None):
    """Forward pass and loss.  Returns a dict with every tensor and the saved BN statistics.

    The forward/backward passes use the bf16 copy of the weights when ``rounding`` is set
    (the fp32 masters are only touched by the update)."""
    T = [np.asarray(images, np.float64)]
    saved = {}
    loss, dlogits = None, None
    for i, L in enumerate(spec):
        k = L["kind"]
        if k == "conv":
            w = _rb(params[f"w{i}"], rounding, "weights")
            T.append(_rb(conv2d_fwd(T[L["src"]], w, L["stride"], L["pad"]), rounding, "conv"))
        elif k == "bn":
            y = T[L["src"]]
            mean, var, invstd = bn_stats(y, BN_EPS)
            mean, invstd = _rf(mean, rounding), _rf(invstd, rounding)
            res = T[L["res"]] if L["res"] >= 0 else None
            a = bn_relu_apply(y, mean, invstd, params[f"gamma{i}"], params[f"beta{i}"], res, L["relu"])
            saved[i] = (mean, invstd, var)
            T.append(_rb(a, rounding, "bn"))
        elif k == "avgpool":
            T.append(_rb(avgpool_fwd(T[L["src"]]), rounding, "pool"))
        elif k == "fc":
            w = _rb(params[f"w{i}"], rounding, "weights")
            z = T[L["src"]] @ np.asarray(w, np.float64).T + np.asarray(params[f"b{i}"], np.float64)
            T.append(_rf(z, rounding))
        elif k == "xent":
            z = T[L["src"]]
            gs = (1.0 / z.shape[0]) if grad_scale is None else grad_scale
            loss, dlogits = softmax_xent(z, labels, gs)
            T.append(None)
        else:
            raise ValueError(k)
    return dict(T=T, saved=saved, loss=loss, dlogits=dlogits)


def backward(spec, params, fw, rounding=True, dout=None):
    """Backward pass.  Returns (grads dict keyed like params, activation-gradient lists).

    ``dout``: upstream gradient of the last tensor when the list has no loss layer."""
    T, saved = fw["T"], fw["saved"]
    contrib = [[] for _ in T]  # gradient contributions per tensor (a BN output has at most two consumers)
    grads = {}
    if dout is not None:
        contrib[len(T) - 1].append(np.asarray(dout, np.float64))
    for i in reversed(range(len(spec))):
        L = spec[i]
        k = L["kind"]
        out_t = i + 1
        if k == "xent":
            contrib[L["src"]].append(_rb(fw["dlogits"], rounding, "dlogits"))
            continue
        if not contrib[out_t]:
            raise RuntimeError(f"layer {i} output has no gradient")
        if k == "fc":
            dz = contrib[out_t][0]
            w = np.asarray(_rb(params[f"w{i}"], rounding, "weights"), np.float64)
            grads[f"w{i}"] = dz.T @ T[L["src"]]
            grads[f"b{i}"] = dz.sum(axis=0)
            contrib[L["src"]].append(_rb(dz @ w, rounding, "fc_dgrad"))
        elif k == "avgpool":
            contrib[L["src"]].append(_rb(avgpool_bwd(contrib[out_t][0], L["H"], L["W"]), rounding, "pool_bwd"))
        elif k == "bn":
            c = contrib[out_t]
            assert len(c) <= 2
            mean, invstd, _ = saved[i]
            dy, dres, dgamma, dbeta = bn_relu_bwd(c[0], c[1] if len(c) == 2 else None, T[L["src"]], T[out_t],
                                                  params[f"gamma{i}"], mean, invstd, L["relu"], L["res"] >= 0)
            grads[f"gamma{i}"], grads[f"beta{i}"] = dgamma, dbeta
            contrib[L["src"]].append(_rb(dy, rounding, "bn_bwd"))
            if L["res"] >= 0:
                contrib[L["res"]].append(_rb(dres, rounding, "bn_bwd_res"))
        elif k == "conv":
            dy = contrib[out_t][0]
            assert len(contrib[out_t]) == 1
            x = T[L["src"]]
            grads[f"w{i}"] = conv2d_wgrad(dy, x, L["R"], L["R"], L["stride"], L["pad"])
            if L["src"] != 0:  # the image batch needs no gradient
                w = _rb(params[f"w{i}"], rounding, "weights")
                contrib[L["src"]].append(_rb(conv2d_dgrad(dy, w, x.shape, L["stride"], L["pad"]), rounding, "conv_dgrad"))
    return grads, contrib


def train_step(spec, params, velocity, images, labels, n_micro, lr, mu, wd, rounding=True):
    """One optimiser step over n_micro micro-batches (replicas).  Returns dict with loss (mean
    over all images), summed gradients, new params and new velocity (all fp64 numpy)."""
    n = images.shape[0] // n_micro
    gsum = {k: np.zeros(v.shape) for k, v in params.items()}
    loss = 0.0
    logits = []
    for m in range(n_micro):
        fw = forward(spec, params, images[m * n:(m + 1) * n], labels[m * n:(m + 1) * n], rounding)
        g, _ = backward(spec, params, fw, rounding)
        for k in gsum:
            gsum[k] += g[k]
        loss += fw["loss"] / n_micro
        logits.append(fw["T"][-2])
    new_p, new_v = {}, {}
    for k in params:
        new_p[k], new_v[k] = sgd_momentum(params[k], velocity[k], gsum[k], 1.0 / n_micro, lr, mu, wd)
    return dict(loss=loss, grads=gsum, params=new_p, velocity=new_v, logits=np.concatenate(logits))
