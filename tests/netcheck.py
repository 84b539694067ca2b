"""Teacher-forced, layer-by-layer check of one training step: after the library has run a
micro-batch, every layer's actual device inputs (activations and gradient buffers left in the
workspace) are fed to the oracle and the layer's device outputs are compared with the oracle's.
Each kernel is thus judged on identical inputs with the per-kernel tolerances, on the real data
distribution of the network, with no amplification of legitimate rounding differences through
ill-conditioned sums further down the chain.

With ``sample`` set, convolution outputs / data gradients / weight gradients are checked on a
random subset of elements computed one by one from the definition (for full-size workloads)."""
import numpy as np
import torch

import oracle
from parity import MAX_REL, REL_FRO, errors, host


def _shape(spec, t, n, net):
    """Stored shape of tensor t (as laid out in the workspace)."""
    if t == 0:
        L = spec[0]
        return (n, L["H"], L["W"], net.image_c_pad)
    L = spec[t - 1]
    k = L["kind"]
    if k == "conv":
        return (n, L["H"] // L["stride"], L["W"] // L["stride"], L["K"])
    if k == "bn":
        return (n, L["H"], L["W"], L["C"])
    if k == "avgpool":
        return (n, L["C"])
    if k == "fc":
        return (n, -(-L["K"] // 64) * 64)
    return None


def grad_slots(spec):
    """(src_slot, res_slot) per layer: which gradient buffer of its input tensors a layer writes.
    Buffers are handed out in backward order, one per consumer."""
    count = [0] * (len(spec) + 1)
    slots = {}
    for i in reversed(range(len(spec))):
        L = spec[i]
        s = r = -1
        if L["kind"] != "conv" or L["src"] != 0:
            s = count[L["src"]]; count[L["src"]] += 1
            if L["kind"] == "bn" and L["res"] >= 0:
                r = count[L["res"]]; count[L["res"]] += 1
        slots[i] = (s, r)
    return slots, count


class Report:
    def __init__(self):
        self.rows = []
        self.differ = {}

    def add(self, name, got, ref, rel_fro=REL_FRO, max_rel=MAX_REL):
        rel, mx = errors(got, ref)
        self.rows.append((name, rel, mx, rel <= rel_fro and mx <= max_rel and bool(np.all(np.isfinite(got)))))
        # share of elements that differ at all: for tensors stored in bf16 these are the roundings that fell the other way
        self.differ[name] = float(np.mean(np.asarray(got, np.float64).reshape(-1) != np.asarray(ref, np.float64).reshape(-1)))

    def failures(self):
        return [r for r in self.rows if not r[3]]

    def worst(self):
        return max(self.rows, key=lambda r: r[1])

    def assert_ok(self):
        bad = self.failures()
        assert not bad, "\n".join(f"{n}: relF={a:.3e} max={b:.3e}" for n, a, b, _ in bad[:20])


def _conv_samples(rng, x, w, y_shape, stride, pad, count):
    """Forward convolution at `count` random output positions, one by one from the definition."""
    N, P, Q, K = y_shape
    idx = np.stack([rng.integers(0, d, count) for d in (N, P, Q, K)], 1)
    H, W = x.shape[1:3]
    R = w.shape[1]
    out = np.zeros(count)
    for j, (n, p, q, k) in enumerate(idx):
        acc = 0.0
        for r in range(R):
            h = p * stride + r - pad
            if h < 0 or h >= H:
                continue
            for s in range(R):
                ww = q * stride + s - pad
                if 0 <= ww < W:
                    acc += float(np.dot(x[n, h, ww, :], w[k, r, s, :]))
        out[j] = acc
    return idx, out


def _dgrad_samples(rng, dy, w, x_shape, stride, pad, count):
    N, H, W, C = x_shape
    idx = np.stack([rng.integers(0, d, count) for d in (N, H, W, C)], 1)
    P, Q = dy.shape[1:3]
    R = w.shape[1]
    out = np.zeros(count)
    for j, (n, h, ww, c) in enumerate(idx):
        acc = 0.0
        for r in range(R):
            ph = h + pad - r
            if ph % stride or not (0 <= ph // stride < P):
                continue
            for s in range(R):
                qw = ww + pad - s
                if qw % stride or not (0 <= qw // stride < Q):
                    continue
                acc += float(np.dot(dy[n, ph // stride, qw // stride, :], w[:, r, s, c]))
        out[j] = acc
    return idx, out


def _wgrad_samples(rng, dy, x, R, stride, pad, count):
    N, H, W, C = x.shape
    P, Q, K = dy.shape[1:]
    idx = np.stack([rng.integers(0, d, count) for d in (K, R, R, C)], 1)
    out = np.zeros(count)
    xp = np.zeros((N, H + 2 * pad, W + 2 * pad), np.float64)
    for j, (k, r, s, c) in enumerate(idx):
        xp[:] = 0.0
        xp[:, pad:pad + H, pad:pad + W] = x[..., c]
        win = xp[:, r:r + stride * P:stride, s:s + stride * Q:stride]
        out[j] = float(np.vdot(dy[..., k], win))
    return idx, out


def check_step(net, spec, images, labels, n, n_micro_scale=1, sample=None, seed=0, groups=1, lowmem=False):
    """Checks the micro-batch whose state is in the workspace (run train_step with n_micro=1, update=False
    first).  `images` are the logical (unpadded) images of that pass: `groups` micro-batches side by side, each
    with its own BatchNorm statistics (n = total images).  Returns a Report.

    lowmem: for full-size workloads.  Host copies are fp32 (exact for bf16 data), fetched from the device each time a
    layer needs them and dropped afterwards, so the host holds one layer's tensors at a time; every element is still
    compared, against the same oracle functions."""
    rep = Report()
    rng = np.random.default_rng(seed)
    rb, rf = oracle.round_bf16, oracle.round_f32
    wq = net.unpack(net.w_bf16)                     # bf16 weights actually used by forward/backward
    wm = net.unpack(net.w)                          # fp32 masters (BN parameters, bias)
    g = net.unpack(net.g)
    slots, n_contrib = grad_slots(spec)

    def to_host(t):
        return t.detach().float().cpu().numpy() if lowmem else host(t)

    def act(t):
        if t == 0:
            return np.asarray(images, np.float32 if lowmem else np.float64)
        shp = _shape(spec, t, n, net)
        dt = torch.float32 if spec[t - 1]["kind"] == "fc" else torch.bfloat16
        return to_host(net.tensor_view(t, shp, dt))

    def grad(t, slot):
        return to_host(net.tensor_view(t, _shape(spec, t, n, net), torch.bfloat16, True, slot))

    cache = {}

    def A(t):
        if lowmem:
            return act(t)
        if t not in cache:
            cache[t] = act(t)
        return cache[t]

    saved = {}
    for i, L in enumerate(spec):
        k, name = L["kind"], L.get("name", str(i))
        if k == "conv":
            x, w, y = A(L["src"]), wq[f"w{i}"].astype(np.float64), A(i + 1)
            if sample:
                idx, ref = _conv_samples(rng, x, w, y.shape, L["stride"], L["pad"], sample)
                rep.add(f"{name} fwd (sampled)", y[tuple(idx.T)], rb(ref), 2 * REL_FRO, MAX_REL * np.max(np.abs(y)) / max(np.max(np.abs(ref)), 1e-30))
            else:
                rep.add(f"{name} fwd", y, rb(oracle.conv2d_fwd(x, w, L["stride"], L["pad"])))
        elif k == "bn":
            y = A(L["src"])
            res = A(L["res"]) if L["res"] >= 0 else None
            per, saved[i], outs = n // groups, [], []
            for gi in range(groups):
                sl = slice(gi * per, (gi + 1) * per)
                mean, var, invstd = oracle.bn_stats(y[sl], 1e-5)
                mean, invstd = rf(mean), rf(invstd)
                saved[i].append((mean, invstd))
                outs.append(oracle.bn_relu_apply(y[sl], mean, invstd, wm[f"gamma{i}"], wm[f"beta{i}"], None if res is None else res[sl], L["relu"]))
            rep.add(f"{name} fwd", A(i + 1), rb(np.concatenate(outs)))
        elif k == "avgpool":
            rep.add(f"{name} fwd", A(i + 1), rb(oracle.avgpool_fwd(A(L["src"]))))
        elif k == "fc":
            z = A(L["src"]) @ wq[f"w{i}"].astype(np.float64).T + wm[f"b{i}"].astype(np.float64)
            rep.add(f"{name} fwd", A(i + 1)[:, :L["K"]], z)
        elif k == "xent":
            z = A(L["src"])[:, :L["K"]]
            loss, dz = oracle.softmax_xent(z, labels, float(groups) / n)
            rep.add("loss", np.array([net.loss.item() * n_micro_scale]), np.array([loss]), 1e-5, 1e-5)
            rep.add("dlogits", grad(L["src"], slots[i][0])[:, :L["K"]], rb(dz))
    for i in reversed(range(len(spec))):
        L = spec[i]
        k, name = L["kind"], L.get("name", str(i))
        s_slot, r_slot = slots[i]
        if k == "fc":
            dz = grad(i + 1, 0)
            rep.add(f"{name} wgrad", g[f"w{i}"], dz[:, :L["K"]].T @ A(L["src"]))
            rep.add(f"{name} bias grad", g[f"b{i}"], dz[:, :L["K"]].sum(0), 1e-4, 1e-4)
            rep.add(f"{name} dgrad", grad(L["src"], s_slot), rb(dz[:, :L["K"]] @ wq[f"w{i}"].astype(np.float64)))
        elif k == "avgpool":
            rep.add(f"{name} bwd", grad(L["src"], s_slot), rb(oracle.avgpool_bwd(grad(i + 1, 0), L["H"], L["W"])))
        elif k == "bn":
            two = n_contrib[i + 1] == 2
            per, parts = n // groups, []
            g1, g2 = grad(i + 1, 0), (grad(i + 1, 1) if two else None)
            y_in, a_out = A(L["src"]), A(i + 1)
            for gi in range(groups):
                sl = slice(gi * per, (gi + 1) * per)
                mean, invstd = saved[i][gi]
                parts.append(oracle.bn_relu_bwd(g1[sl], None if g2 is None else g2[sl], y_in[sl], a_out[sl], wm[f"gamma{i}"], mean, invstd,
                                                L["relu"], L["res"] >= 0))
            del g1, g2, y_in, a_out
            dy = np.concatenate([q[0] for q in parts])
            dres = np.concatenate([q[1] for q in parts]) if L["res"] >= 0 else None
            dg, db = sum(q[2] for q in parts), sum(q[3] for q in parts)
            rep.add(f"{name} bwd dy", grad(L["src"], s_slot), rb(dy))
            if L["res"] >= 0:
                rep.add(f"{name} bwd dres", grad(L["res"], r_slot), rb(dres))
            rep.add(f"{name} dgamma", g[f"gamma{i}"], dg)
            rep.add(f"{name} dbeta", g[f"beta{i}"], db)
        elif k == "conv":
            dy, x, w = grad(i + 1, 0), A(L["src"]), wq[f"w{i}"].astype(np.float64)
            if sample:
                idx, ref = _wgrad_samples(rng, dy, x, L["R"], L["stride"], L["pad"], min(sample, 64))
                got = g[f"w{i}"][tuple(idx.T)]
                rep.add(f"{name} wgrad (sampled)", got, ref, 2 * REL_FRO, MAX_REL * np.max(np.abs(g[f"w{i}"])) / max(np.max(np.abs(ref)), 1e-30))
                if L["src"] != 0:
                    dx = grad(L["src"], s_slot)
                    idx, ref = _dgrad_samples(rng, dy, w, x.shape, L["stride"], L["pad"], sample)
                    rep.add(f"{name} dgrad (sampled)", dx[tuple(idx.T)], rb(ref), 2 * REL_FRO, MAX_REL * np.max(np.abs(dx)) / max(np.max(np.abs(ref)), 1e-30))
            else:
                rep.add(f"{name} wgrad", g[f"w{i}"], oracle.conv2d_wgrad(dy, x, L["R"], L["R"], L["stride"], L["pad"]))
                if L["src"] != 0:
                    rep.add(f"{name} dgrad", grad(L["src"], s_slot), rb(oracle.conv2d_dgrad(dy, w, x.shape, L["stride"], L["pad"])))
    return rep


def check_step_sampled(net, spec, images, labels, n, groups=1, samples=128, bn_channels=4, seed=0):
    """Full-size variant of check_step: every layer of the pass left in the workspace is checked against the oracle
    on its own device inputs, but only on what the oracle can compute one by one at this size -- `samples` random
    outputs per convolution (forward, data gradient) and a few filter entries (weight gradient), `bn_channels` whole
    channels per BatchNorm (statistics, outputs, both gradients), and the small head in full.  Host copies are fp32
    (exact for bf16 data) and fetched on demand, so the largest workloads fit in host memory."""
    rep = Report()
    rng = np.random.default_rng(seed)
    rb, rf = oracle.round_bf16, oracle.round_f32
    wq, wm, g = net.unpack(net.w_bf16), net.unpack(net.w), net.unpack(net.g)
    slots, n_contrib = grad_slots(spec)
    per = n // groups

    def host32(t):
        return t.detach().float().cpu().numpy()

    def act(t):
        if t == 0:
            return np.asarray(images, np.float32)
        dt = torch.float32 if spec[t - 1]["kind"] == "fc" else torch.bfloat16
        return host32(net.tensor_view(t, _shape(spec, t, n, net), dt))

    def grad(t, slot):
        return host32(net.tensor_view(t, _shape(spec, t, n, net), torch.bfloat16, True, slot))

    def cols(a, chs):   # selected channels as a contiguous fp64 [rows, len(chs)] array per group
        return np.ascontiguousarray(a.reshape(groups, -1, a.shape[-1])[:, :, chs], dtype=np.float64)

    def tol(full, ref):
        return MAX_REL * float(np.max(np.abs(full))) / max(float(np.max(np.abs(ref))), 1e-30)

    for i, L in enumerate(spec):
        k, name = L["kind"], L.get("name", str(i))
        if k == "conv":
            x, w, y = act(L["src"]), wq[f"w{i}"].astype(np.float64), act(i + 1)
            idx, ref = _conv_samples(rng, x, w, y.shape, L["stride"], L["pad"], samples)
            rep.add(f"{name} fwd (sampled)", y[tuple(idx.T)], rb(ref), 2 * REL_FRO, tol(y, ref))
            dy = grad(i + 1, 0)
            idx, ref = _wgrad_samples(rng, dy, x, L["R"], L["stride"], L["pad"], max(8, samples // 8))
            rep.add(f"{name} wgrad (sampled)", g[f"w{i}"][tuple(idx.T)], ref, 2 * REL_FRO, tol(g[f"w{i}"], ref))
            if L["src"] != 0:
                dx = grad(L["src"], slots[i][0])
                idx, ref = _dgrad_samples(rng, dy, w, x.shape, L["stride"], L["pad"], samples)
                rep.add(f"{name} dgrad (sampled)", dx[tuple(idx.T)], rb(ref), 2 * REL_FRO, tol(dx, ref))
        elif k == "bn":
            C = L["C"]
            chs = np.sort(rng.choice(C, size=min(bn_channels, C), replace=False))
            y, a = cols(act(L["src"]), chs), cols(act(i + 1), chs)
            res = cols(act(L["res"]), chs) if L["res"] >= 0 else None
            g1 = cols(grad(i + 1, 0), chs)
            g2 = cols(grad(i + 1, 1), chs) if n_contrib[i + 1] == 2 else None
            gam, bet = wm[f"gamma{i}"][chs], wm[f"beta{i}"][chs]
            a_ref, dy_ref, dres_ref, dg, db = [], [], [], 0.0, 0.0
            for gi in range(groups):
                mean, var, invstd = oracle.bn_stats(y[gi], 1e-5)
                mean, invstd = rf(mean), rf(invstd)
                a_ref.append(oracle.bn_relu_apply(y[gi], mean, invstd, gam, bet, None if res is None else res[gi], L["relu"]))
                q = oracle.bn_relu_bwd(g1[gi], None if g2 is None else g2[gi], y[gi], a[gi], gam, mean, invstd, L["relu"], L["res"] >= 0)
                dy_ref.append(q[0]); dres_ref.append(q[1]); dg = dg + q[2]; db = db + q[3]
            rep.add(f"{name} fwd (channels)", a, rb(np.stack(a_ref)))
            rep.add(f"{name} bwd dy (channels)", cols(grad(L["src"], slots[i][0]), chs), rb(np.stack(dy_ref)))
            if L["res"] >= 0:
                rep.add(f"{name} bwd dres (channels)", cols(grad(L["res"], slots[i][1]), chs), rb(np.stack(dres_ref)))
            rep.add(f"{name} dgamma (channels)", g[f"gamma{i}"][chs], dg)
            rep.add(f"{name} dbeta (channels)", g[f"beta{i}"][chs], db)
        elif k == "avgpool":
            rep.add(f"{name} fwd", act(i + 1), rb(oracle.avgpool_fwd(act(L["src"]))))
            rep.add(f"{name} bwd", grad(L["src"], slots[i][0]), rb(oracle.avgpool_bwd(grad(i + 1, 0), L["H"], L["W"])))
        elif k == "fc":
            pooled, dz = act(L["src"]).astype(np.float64), grad(i + 1, 0).astype(np.float64)
            z = pooled @ wq[f"w{i}"].astype(np.float64).T + wm[f"b{i}"].astype(np.float64)
            rep.add(f"{name} fwd", act(i + 1)[:, :L["K"]], z)
            rep.add(f"{name} wgrad", g[f"w{i}"], dz[:, :L["K"]].T @ pooled)
            rep.add(f"{name} bias grad", g[f"b{i}"], dz[:, :L["K"]].sum(0), 1e-4, 1e-4)
            rep.add(f"{name} dgrad", grad(L["src"], slots[i][0]), rb(dz[:, :L["K"]] @ wq[f"w{i}"].astype(np.float64)))
        elif k == "xent":
            z = act(L["src"])[:, :L["K"]].astype(np.float64)
            loss, dz = oracle.softmax_xent(z, labels, 1.0 / per)
            rep.add("loss", np.array([net.loss.item()]), np.array([loss]), 1e-5, 1e-5)
            rep.add("dlogits", grad(L["src"], slots[i][0])[:, :L["K"]], rb(dz))
    return rep
