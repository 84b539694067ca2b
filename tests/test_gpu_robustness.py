"""Robustness of the CUDA path beyond parity: guard bands around every output and scratch buffer (the stand-in for a
memory checker: a store that strays outside its buffer lands on a sentinel), every kernel-variant switch off and on
against the oracle, and the wind-down of every kernel with bounded waits when a wait's budget runs out (a budget of one
poll on a healthy launch: the status word reports the time-out, the context stays usable, the next call is correct)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_23186_b200 import workloads as wl
from parity import assert_close, dev_bf16, dev_f32, host

pytestmark = pytest.mark.gpu

GUARD = 4096   # bytes of sentinel on both sides


class Guarded:
    """A device tensor of the given shape and dtype with GUARD bytes of 0xC3 before and after it."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256
        self.raw = torch.full((GUARD + n + pad + GUARD,), 0xC3, dtype=torch.uint8, device="cuda")
        self.n = n
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, name):
        before, after = self.raw[:GUARD], self.raw[GUARD + self.n:]
        assert bool((before == 0xC3).all()) and bool((after == 0xC3).all()), f"{name}: bytes outside the buffer were written"


def _desc(N, H, W, C, K, R, stride):
    from paper_2503_23186_b200 import binding
    return binding.conv_desc(N, H, W, C, K, R, stride)


def _dgrad_weights(ctx, w):
    K, R, S, C = w.shape
    src = dev_bf16(w).reshape(-1)
    dst = Guarded((src.numel(),), torch.bfloat16)
    ctx.weight_pack_dgrad([(0, K, R * S, C)], src, dst.t)
    dst.check("dgrad weight layout")
    return dst.t


GUARD_SHAPES = [(8, 32, 32, 64, 64, 3, 1), (3, 8, 8, 32, 32, 3, 1), (4, 16, 16, 128, 256, 3, 1), (8, 32, 32, 64, 128, 3, 2), (6, 4, 4, 128, 64, 3, 1),
                (2, 32, 32, 16, 160, 1, 1), (130, 1, 1, 512, 128, 1, 1)]


@pytest.fixture(scope="module")
def ctx():
    from paper_2503_23186_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


@pytest.mark.parametrize("shape", GUARD_SHAPES, ids=lambda s: "n{}h{}w{}c{}k{}r{}s{}".format(*s))
def test_convolutions_stay_inside_their_buffers(ctx, shape):
    N, H, W, C, K, R, st = shape
    x, w, g = wl.conv_problem(30, *shape)
    P = H // st
    y = Guarded((N, P, P, K), torch.bfloat16, float("nan"))
    stats = Guarded((2 * K,), torch.float64, 0.0)
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y.t, ch_stats=stats.t)
    dx = Guarded((N, H, W, C), torch.bfloat16, float("nan"))
    ctx.conv2d_dgrad(_desc(*shape), dev_bf16(g), _dgrad_weights(ctx, w), dx.t)
    dw = Guarded((K, R, R, C), torch.float32, float("nan"))
    ctx.conv2d_wgrad(_desc(*shape), dev_bf16(g), dev_bf16(x), dw.t, accumulate=False)
    assert ctx.device_status() == 0
    for buf, name in ((y, "y"), (stats, "channel statistics"), (dx, "dx"), (dw, "dw")):
        buf.check(name)
    assert_close(y.t, oracle.conv2d_fwd(x, w, st, (R - 1) // 2), "y")
    assert_close(dx.t, oracle.conv2d_dgrad(g, w, x.shape, st, (R - 1) // 2), "dx")
    assert_close(dw.t, oracle.conv2d_wgrad(g, x, R, R, st, (R - 1) // 2), "dw")


@pytest.mark.parametrize("shape", [(8, 32, 32, 64), (3, 8, 8, 160), (33, 31, 32, 64), (20, 32, 33, 160)], ids=lambda s: "x".join(map(str, s)))
def test_batchnorm_and_small_kernels_stay_inside_their_buffers(ctx, shape):
    N, H, W, C = shape
    M = N * H * W
    r = wl.rng_for(31, f"guard{shape}")
    y = wl.to_bf16_grid(r.standard_normal(shape) + 0.5)
    res = wl.to_bf16_grid(r.standard_normal(shape))
    da1, da2 = wl.to_bf16_grid(r.standard_normal(shape)), wl.to_bf16_grid(r.standard_normal(shape))
    gamma, beta = dev_f32(1.0 + 0.1 * r.standard_normal(C)), dev_f32(0.1 * r.standard_normal(C))
    a = Guarded(shape, torch.bfloat16, float("nan"))
    stats = Guarded((2 * C,), torch.float64, 3.0)
    sm, si = Guarded((C,), torch.float32), Guarded((C,), torch.float32)
    rm, rv = Guarded((C,), torch.float32, 0.0), Guarded((C,), torch.float32, 1.0)
    mask = Guarded((M * C // 8,), torch.uint8, 0)
    ctx.bn_relu_fwd(N, H, W, C, dev_bf16(y), stats.t, False, gamma, beta, dev_bf16(res), True, 1e-5, a.t, sm.t, si.t, rm.t, rv.t, 0.1, relu_mask=mask.t)
    dy, dres = Guarded(shape, torch.bfloat16, float("nan")), Guarded(shape, torch.bfloat16, float("nan"))
    dg, db = Guarded((C,), torch.float32, 0.0), Guarded((C,), torch.float32, 0.0)
    ws = Guarded((ctx.bn_relu_bwd_workspace_bytes(C),), torch.uint8)
    ctx.bn_relu_bwd(N, H, W, C, dev_bf16(da1), dev_bf16(da2), dev_bf16(y), None, gamma, sm.t, si.t, True, dy.t, dres.t, dg.t, db.t, False, ws.t,
                    relu_mask=mask.t)
    if (M * (C // 8)) % 16 == 0:
        wsg = Guarded((ctx.bn_relu_bwd_groups_workspace_bytes(C, 1),), torch.uint8)
        dy2 = Guarded(shape, torch.bfloat16, float("nan"))
        ctx.bn_relu_bwd_groups(1, M, C, dev_bf16(da1), dev_bf16(da2), dev_bf16(y), gamma, sm.t, si.t, True, dy2.t, dres.t, dg.t, db.t, False, mask.t, wsg.t)
        wsg.check("grouped backward scratch"); dy2.check("dy (grouped)")
        assert_close(dy2.t, host(dy.t), "dy grouped vs two-pass", 1e-5, 1e-2)
    pooled = Guarded((N, C), torch.bfloat16, float("nan"))
    ctx.avgpool_fwd(N, H * W, C, a.t, pooled.t)
    dpool = Guarded(shape, torch.bfloat16, float("nan"))
    ctx.avgpool_bwd(N, H * W, C, pooled.t, dpool.t)
    assert ctx.device_status() == 0
    for buf, name in ((a, "a"), (stats, "stats"), (sm, "mean"), (si, "invstd"), (rm, "running mean"), (rv, "running var"), (mask, "mask"), (dy, "dy"),
                      (dres, "dres"), (dg, "dgamma"), (db, "dbeta"), (ws, "scratch"), (pooled, "pooled"), (dpool, "pool gradient")):
        buf.check(name)
    assert np.all(np.isfinite(host(a.t))) and np.all(np.isfinite(host(dy.t)))


def test_loss_update_and_padding_stay_inside_their_buffers(ctx):
    r = wl.rng_for(32, "guard-small")
    n, classes, pitch = 130, 100, 128
    z = dev_f32((r.standard_normal((n, pitch)) * 2).astype(np.float32))
    labels = torch.from_numpy(r.integers(0, classes, n).astype(np.int32)).cuda()
    loss, dz = Guarded((1,), torch.float32, 0.0), Guarded((n, pitch), torch.bfloat16, float("nan"))
    ctx.softmax_xent_fwd_bwd(n, classes, z, pitch, labels, 1.0 / n, 1.0 / n, loss.t, dz.t, pitch)
    db = Guarded((classes,), torch.float32, 0.0)
    ctx.bias_grad(n, classes, pitch, dz.t, db.t, False)
    count = 4 * 1000 + 4
    w, v, g = (Guarded((count,), torch.float32, 0.5) for _ in range(3))
    wb = Guarded((count,), torch.bfloat16, 0.0)
    ctx.grad_accum_sgd_momentum(count, w.t, v.t, g.t, 0.125, 0.1, 0.9, 5e-4, wb.t, True)
    x = dev_bf16(wl.to_bf16_grid(r.standard_normal((7, 5, 5, 3))))
    xp, xc = Guarded((7, 5, 5, 16), torch.bfloat16, float("nan")), Guarded((7, 5, 5, 32), torch.bfloat16, float("nan"))
    ctx.pad_channels(7 * 25, 3, 16, x, xp.t)
    ctx.im2col_3x3(7, 5, 5, 3, 32, x, xc.t)
    assert ctx.device_status() == 0
    for buf, name in ((loss, "loss"), (dz, "dlogits"), (db, "bias gradient"), (w, "w"), (v, "v"), (g, "g"), (wb, "bf16 copy"), (xp, "padded"), (xc, "patches")):
        buf.check(name)


# ------------------------------------------------------------------------------ kernel-variant switches off and on
SWITCHES = [("B2C_ISSUE_SPLIT", "0"), ("B2C_ISSUE_SPLIT", "1"), ("B2C_WGRAD_FRAME", "0"), ("B2C_WGRAD_FRAME", "1"), ("B2C_WGRAD_ISSUERS", "1"),
            ("B2C_WGRAD_ISSUERS", "2"), ("B2C_PDL", "0"), ("B2C_PDL", "1"), ("B2C_CTA_PAIRS", "3"), ("B2C_CTA_PAIRS", "1"), ("B2C_HMERGE", "0"), ("B2C_HMERGE", "1"),
            ("B2C_GROUP_KBLOCKS", "0"), ("B2C_GROUP_KBLOCKS", "1")]


@pytest.mark.parametrize("name,value", SWITCHES, ids=lambda v: str(v))
def test_kernel_switches_off_and_on(name, value, monkeypatch):
    """Each switch of b2c_create in both positions: forward, data gradient and weight gradient of layers that reach the
    switched path (256-channel tiles, 3x3 stride-1 layers with 8- and 32-pixel rows, 64 output channels, stride-2 and 1x1 layers
    whose short k-blocks share ring slots, with an even and an odd number of k-blocks, with one and with two issuing threads per unit)
    against the oracle."""
    from paper_2503_23186_b200 import binding
    monkeypatch.setenv(name, value)
    c = binding.Context(0)
    try:
        # (the 64-output-channel layers are large enough for merged horizontal taps: at least two tiles per SM, rows of 32 / 16 / 8 pixels)
        for shape in [(4, 16, 16, 128, 256, 3, 1), (4, 8, 8, 512, 512, 3, 1), (40, 32, 32, 64, 64, 3, 1), (160, 16, 16, 64, 64, 3, 1), (600, 8, 8, 128, 64, 3, 1),
                      (16, 8, 8, 128, 128, 3, 1), (8, 32, 32, 64, 128, 3, 2), (8, 16, 16, 256, 64, 1, 1), (8, 16, 16, 192, 64, 1, 1), (4, 16, 16, 160, 320, 3, 2)]:
            N, H, W, C, K, R, st = shape
            x, w, g = wl.conv_problem(33, *shape)
            P = H // st
            pad = (R - 1) // 2
            y = torch.full((N, P, P, K), float("nan"), dtype=torch.bfloat16, device="cuda")
            c.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y)
            assert_close(y, oracle.conv2d_fwd(x, w, st, pad), f"y {shape} {name}={value}")
            dx = torch.full(x.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            c.conv2d_dgrad(_desc(*shape), dev_bf16(g), _dgrad_weights(c, w), dx)
            assert_close(dx, oracle.conv2d_dgrad(g, w, x.shape, st, pad), f"dx {shape} {name}={value}")
            dw = torch.full(w.shape, float("nan"), dtype=torch.float32, device="cuda")
            c.conv2d_wgrad(_desc(*shape), dev_bf16(g), dev_bf16(x), dw, accumulate=False)
            assert_close(dw, oracle.conv2d_wgrad(g, x, R, R, st, pad), f"dw {shape} {name}={value}")
            assert c.device_status() == 0
    finally:
        c.close()


@pytest.mark.parametrize("name,value", [("B2C_FUSE_WIDE", "0"), ("B2C_FUSE_WIDE", "1"), ("B2C_FUSE_BN_STATS", "0"), ("B2C_FUSE_BN_STATS", "1"),
                                        ("B2C_BN_GROUPED", "1"), ("B2C_BN_GROUPED", "0")], ids=lambda v: str(v))
def test_step_plan_switches_off_and_on(name, value, monkeypatch):
    """The switches b2c_net_create / b2c_train_step read: where the BatchNorm statistics are taken, and the grouped BatchNorm
    backward.  One pass of four micro-batches side by side, every layer against the oracle on its own device inputs."""
    from paper_2503_23186_b200 import binding
    from netcheck import check_step
    monkeypatch.setenv(name, value)
    c = binding.Context(0)
    try:
        spec = wl.tiny_net_spec(classes=10, hw=16, c=3, width=64, width2=128)
        params = wl.perturb_bn_params(wl.init_params(spec, 34), 34)
        images, labels = wl.image_batch(34, 4 * 8, hw=16, c=3, classes=10)
        net = binding.Net(c, spec, 8, n_concurrent=4)
        net.load_params(params)
        net.train_step(dev_bf16(images), torch.from_numpy(labels).cuda(), 4, 0.1, 0.9, 5e-4, update=False)
        assert c.device_status() == 0
        check_step(net, spec, images, labels, 32, groups=4).assert_ok()
        net.close()
    finally:
        c.close()


# ------------------------------------------------------------------------------ bounded waits run out: wind-down and recovery
def _expect_timeout_then_recover(ctx, run, check):
    ctx.set_spin_limit(1)
    try:
        run()
        status = ctx.device_status()
    finally:
        ctx.set_spin_limit(1 << 22)
    assert status == 7   # B2C_ERR_DEVICE_TIMEOUT
    run()
    assert ctx.device_status() == 0
    check()


@pytest.mark.parametrize("shape", [(16, 16, 16, 128, 128, 3, 1), (8, 8, 8, 256, 256, 3, 1), (8, 32, 32, 64, 128, 3, 2)], ids=lambda s: "n{}h{}w{}c{}k{}r{}s{}".format(*s))
def test_forward_variants_wind_down_on_timeout(ctx, shape):
    """CTA pairs (128- and 256-channel tiles, the latter with two issuing threads per unit) and a stride-2 layer."""
    N, H, W, C, K, R, st = shape
    x, w, _ = wl.conv_problem(35, *shape)
    P = H // st
    y = torch.zeros((N, P, P, K), dtype=torch.bfloat16, device="cuda")
    X, Wt = dev_bf16(x), dev_bf16(w)
    _expect_timeout_then_recover(ctx, lambda: ctx.conv2d_fwd(_desc(*shape), X, Wt, y),
                                 lambda: assert_close(y, oracle.conv2d_fwd(x, w, st, 1), "y after recovery"))


@pytest.mark.parametrize("shape", [(8, 32, 32, 64, 64, 3, 1), (4, 8, 8, 512, 512, 3, 1), (8, 32, 32, 64, 128, 1, 2)], ids=lambda s: "n{}h{}w{}c{}k{}r{}s{}".format(*s))
def test_weight_gradient_winds_down_on_timeout(ctx, shape):
    N, H, W, C, K, R, st = shape
    x, _, g = wl.conv_problem(36, *shape)
    dw = torch.zeros((K, R, R, C), dtype=torch.float32, device="cuda")
    X, G = dev_bf16(x), dev_bf16(g)
    _expect_timeout_then_recover(ctx, lambda: ctx.conv2d_wgrad(_desc(*shape), G, X, dw, accumulate=False),
                                 lambda: assert_close(dw, oracle.conv2d_wgrad(g, x, R, R, st, (R - 1) // 2), "dw after recovery"))


@pytest.mark.parametrize("grouped", [False, True], ids=["two-pass", "grouped"])
def test_staged_batchnorm_backward_winds_down_on_timeout(ctx, grouped):
    """The bulk-copy ring of the BatchNorm backward (two launches, or one cooperative launch with its grid-wide barrier)."""
    G, M, C = 2, 32768, 64   # enough rows per block for the two-pass launcher to choose the staged kernels
    r = wl.rng_for(37, "bn-timeout")
    y = wl.to_bf16_grid(r.standard_normal((G, M, C)))
    da = wl.to_bf16_grid(r.standard_normal((G, M, C)))
    gamma = np.ones(C, np.float32)
    means, invstds, dy_ref = [], [], []
    for gi in range(G):
        mean, _, invstd = oracle.bn_stats(y[gi], 1e-5)
        mean, invstd = oracle.round_f32(mean), oracle.round_f32(invstd)
        q = oracle.bn_relu_bwd(da[gi], None, y[gi], y[gi], gamma, mean, invstd, False, False)
        means.append(mean); invstds.append(invstd); dy_ref.append(q[0])
    dy = torch.zeros((G, M, C), dtype=torch.bfloat16, device="cuda")
    dg, db = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda")
    DA, Y, GM = dev_bf16(da), dev_bf16(y), dev_f32(gamma)
    if grouped:
        ws = torch.zeros(ctx.bn_relu_bwd_groups_workspace_bytes(C, G), dtype=torch.uint8, device="cuda")
        run = lambda: ctx.bn_relu_bwd_groups(G, M, C, DA, None, Y, GM, dev_f32(np.stack(means)), dev_f32(np.stack(invstds)), False, dy, None, dg, db, False, None, ws)
        check = lambda: assert_close(dy, np.stack(dy_ref), "dy after recovery")
    else:
        ws = torch.zeros(ctx.bn_relu_bwd_workspace_bytes(C), dtype=torch.uint8, device="cuda")
        run = lambda: ctx.bn_relu_bwd(1, M, 1, C, DA[0], None, Y[0], None, GM, dev_f32(means[0]), dev_f32(invstds[0]), False, dy[0], None, dg, db, False, ws)
        check = lambda: assert_close(dy[0], dy_ref[0], "dy after recovery")
    _expect_timeout_then_recover(ctx, run, check)


def test_stall_counters_report_wait_cycles(ctx):
    """b2c_set_stall_counters: the convolution kernels add their roles' wait cycles and lifetime to a caller-owned array."""
    shape = (16, 32, 32, 64, 64, 3, 1)
    x, w, g = wl.conv_problem(38, *shape)
    y = torch.empty((16, 32, 32, 64), dtype=torch.bfloat16, device="cuda")
    cnt = torch.zeros(8, dtype=torch.int64, device="cuda")
    ctx.set_stall_counters(cnt)
    try:
        ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y)
        torch.cuda.synchronize()
        fwd = cnt.cpu().numpy().copy()
        cnt.zero_()
        dw = torch.zeros((64, 3, 3, 64), dtype=torch.float32, device="cuda")
        ctx.conv2d_wgrad(_desc(*shape), dev_bf16(g), dev_bf16(x), dw, accumulate=False)
        torch.cuda.synchronize()
        wg = cnt.cpu().numpy().copy()
    finally:
        ctx.set_stall_counters(None)
    assert fwd[4] > 0 and all(0 <= fwd[i] <= 2 * fwd[4] for i in range(4))   # waits are parts of the CTAs' lifetime (two issuing threads add into [1], [2])
    assert wg[4] > 0 and wg[7] > 0 and wg[6] > 0
    assert_close(y, oracle.conv2d_fwd(x, w, 1, 1), "y with diagnostics on")
    assert ctx.device_status() == 0
