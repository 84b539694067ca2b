"""Per-kernel parity (teacher-forced): every C-ABI entry point against the fp64 oracle on the same
seeded bf16-rounded inputs.  Sizes span several tiles, ragged tails and every supported layout path."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_23186_b200 import workloads as wl
from parity import SGD_REL, assert_close, dev_bf16, dev_f32, errors, host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2503_23186_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def _desc(N, H, W, C, K, R, stride):
    from paper_2503_23186_b200 import binding
    return binding.conv_desc(N, H, W, C, K, R, stride)


# (N, H, W, C, K, R, stride): 128-byte / 64-byte / 32-byte swizzle paths, stride 2, 1x1, ragged batch,
# several channel tiles, tiles spanning several images, WRN widths.
CONV_SHAPES = [
    (8, 32, 32, 64, 64, 3, 1),
    (8, 32, 32, 16, 16, 3, 1),      # config 1
    (3, 8, 8, 32, 32, 3, 1),        # 1.5 tiles: ragged batch, 64-byte rows
    (4, 16, 16, 128, 256, 3, 1),
    (4, 16, 16, 256, 128, 3, 1),
    (8, 32, 32, 64, 128, 3, 2),
    (8, 32, 32, 64, 128, 1, 2),
    (5, 16, 16, 32, 64, 3, 2),
    (6, 4, 4, 128, 64, 3, 1),       # 8 images per tile, ragged
    (2, 16, 16, 160, 160, 3, 1),    # WRN width
    (2, 32, 32, 160, 160, 3, 1),    # WRN width at full image size (framed weight-gradient stages with 32-channel boxes)
    (4, 8, 8, 512, 512, 3, 1),      # two channel tiles of 256, long reduction
    (2, 32, 32, 16, 160, 1, 1),
    (130, 1, 1, 512, 128, 1, 1),    # classifier-shaped
]


def _ids(s):
    return "n{}h{}w{}c{}k{}r{}s{}".format(*s)


@pytest.mark.parametrize("shape", CONV_SHAPES, ids=_ids)
def test_conv2d_fwd(ctx, shape):
    N, H, W, C, K, R, st = shape
    x, w, _ = wl.conv_problem(0, N, H, W, C, K, R, st)
    ref = oracle.conv2d_fwd(x, w, st, (R - 1) // 2)
    y = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    stats = torch.zeros(2 * K, dtype=torch.float64, device="cuda")
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y, ch_stats=stats)
    assert ctx.device_status() == 0
    assert_close(y, ref, "y")
    # fused BatchNorm statistics are those of the values as stored
    ys = host(y).reshape(-1, K)
    s = host(stats)
    np.testing.assert_allclose(s[:K], ys.sum(0), rtol=1e-5, atol=1e-3 * np.sqrt(ys.shape[0]))
    np.testing.assert_allclose(s[K:], (ys * ys).sum(0), rtol=1e-5)


def test_conv2d_fwd_f32_bias(ctx):
    shape = (130, 1, 1, 512, 128, 1, 1)
    N, H, W, C, K, R, st = shape
    x, w, _ = wl.conv_problem(1, *shape)
    bias = wl.rng_for(1, "bias").standard_normal(K).astype(np.float32)
    ref = oracle.conv2d_fwd(x, w, st, 0) + bias.astype(np.float64)
    y = torch.full(ref.shape, float("nan"), dtype=torch.float32, device="cuda")
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y, bias=dev_f32(bias))
    assert ctx.device_status() == 0
    assert_close(y, ref, "logits")


def test_conv2d_fwd_delta_and_shift_exact(ctx):
    # identity / shift filters reproduce the input bit for bit (checks orientation and padding corners)
    N, H, W, C = 2, 16, 16, 64
    x = wl.normal_bf16(2, "x", (N, H, W, C))
    for (r, s) in [(1, 1), (0, 0), (2, 1), (1, 2)]:
        w = np.zeros((C, 3, 3, C), np.float32)
        w[np.arange(C), r, s, np.arange(C)] = 1.0
        y = torch.empty((N, H, W, C), dtype=torch.bfloat16, device="cuda")
        ctx.conv2d_fwd(_desc(N, H, W, C, C, 3, 1), dev_bf16(x), dev_bf16(w), y)
        ref = oracle.conv2d_fwd(x, w, 1, 1)
        assert np.array_equal(host(y), ref), (r, s)


def _dgrad_weights(ctx, w):
    """[k,r,s,c] bf16 -> the [c,r,s,k] tap-flipped layout, produced by the library's own kernel."""
    K, R, S, C = w.shape
    src = dev_bf16(w).reshape(-1)
    dst = torch.empty_like(src)
    ctx.weight_pack_dgrad([(0, K, R * S, C)], src, dst)
    return dst


@pytest.mark.parametrize("shape", CONV_SHAPES, ids=_ids)
def test_conv2d_dgrad(ctx, shape):
    N, H, W, C, K, R, st = shape
    x, w, g = wl.conv_problem(0, *shape)
    ref = oracle.conv2d_dgrad(g, w, x.shape, st, (R - 1) // 2)
    wd = _dgrad_weights(ctx, w)
    expect = np.ascontiguousarray(np.flip(w, (1, 2)).transpose(3, 1, 2, 0))
    assert np.array_equal(host(wd).reshape(expect.shape), expect)
    dx = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.conv2d_dgrad(_desc(*shape), dev_bf16(g), wd, dx)
    assert ctx.device_status() == 0
    assert_close(dx, ref, "dx")
    # adjoint identity on the GPU results: <conv(x;w), g> = <x, dgrad(g;w)>
    y = torch.empty(g.shape, dtype=torch.bfloat16, device="cuda")
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y)
    lhs, rhs = np.vdot(host(y), g), np.vdot(x, host(dx))
    scale = np.linalg.norm(host(y)) * np.linalg.norm(g)
    assert abs(lhs - rhs) <= 2e-3 * scale


@pytest.mark.parametrize("shape", CONV_SHAPES, ids=_ids)
def test_conv2d_wgrad(ctx, shape):
    N, H, W, C, K, R, st = shape
    x, w, g = wl.conv_problem(0, *shape)
    ref = oracle.conv2d_wgrad(g, x, R, R, st, (R - 1) // 2)
    dw = torch.full(ref.shape, float("nan"), dtype=torch.float32, device="cuda")
    ctx.conv2d_wgrad(_desc(*shape), dev_bf16(g), dev_bf16(x), dw, accumulate=False)
    assert ctx.device_status() == 0
    assert_close(dw, ref, "dw")
    # accumulate: a second call adds the same sum again (micro-batch accumulation)
    ctx.conv2d_wgrad(_desc(*shape), dev_bf16(g), dev_bf16(x), dw, accumulate=True)
    assert_close(dw, 2 * ref, "dw accumulated")


def test_conv_rejects_bad_arguments(ctx):
    from paper_2503_23186_b200 import binding
    x = torch.zeros(8 * 32 * 32 * 64, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros_like(x)
    w = torch.zeros(64 * 9 * 64, dtype=torch.bfloat16, device="cuda")
    for bad, code in [((8, 32, 32, 60, 64, 3, 1), 2), ((8, 24, 24, 64, 64, 3, 1), 2), ((8, 32, 32, 64, 64, 5, 1), 2),
                      ((8, 31, 32, 64, 64, 3, 2), 2), ((0, 32, 32, 64, 64, 3, 1), 1)]:
        with pytest.raises(binding.B2CError) as e:
            ctx.conv2d_fwd(_desc(*bad), x, w, y)
        assert e.value.status == code, bad
    with pytest.raises(binding.B2CError) as e:
        ctx.conv2d_fwd(_desc(8, 32, 32, 64, 64, 3, 1), x[1:], w, y)   # 2-byte offset
    assert e.value.status == 3
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------ BatchNorm
# the last two are large enough for the bulk-copy ring of the backward kernels (with a ragged last chunk; 160 channels
# leave 16 threads of a block without a channel group)
BN_SHAPES = [(8, 32, 32, 64), (3, 8, 8, 160), (128, 4, 4, 512), (5, 16, 16, 8), (2, 16, 16, 640), (33, 31, 32, 64), (20, 32, 33, 160)]


@pytest.mark.parametrize("shape", BN_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("relu,use_res", [(True, False), (True, True), (False, False)])
def test_bn_relu_fwd_bwd(ctx, shape, relu, use_res):
    N, H, W, C = shape
    M = N * H * W
    r = wl.rng_for(3, f"bn{shape}")
    y = wl.to_bf16_grid(r.standard_normal(shape) * (0.5 + r.random(C)) + 2.0 * r.standard_normal(C))
    res = wl.to_bf16_grid(r.standard_normal(shape)) if use_res else None
    gamma = (1.0 + 0.3 * r.standard_normal(C)).astype(np.float32)
    beta = (0.2 * r.standard_normal(C)).astype(np.float32)
    da1 = wl.to_bf16_grid(r.standard_normal(shape))
    da2 = wl.to_bf16_grid(r.standard_normal(shape)) if use_res else None

    mean, var, invstd = oracle.bn_stats(y, 1e-5)
    mean32, invstd32 = oracle.round_f32(mean), oracle.round_f32(invstd)
    a_ref = oracle.round_bf16(oracle.bn_relu_apply(y, mean32, invstd32, gamma, beta, res, relu))

    dy_, a = dev_bf16(y), torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    stats = torch.full((2 * C,), 7.0, dtype=torch.float64, device="cuda")   # stale contents must not matter
    sm, si = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    rm, rv = torch.zeros(C, device="cuda"), torch.ones(C, device="cuda")
    mask = torch.full((M * C // 8,), 0xAA, dtype=torch.uint8, device="cuda")
    ctx.bn_relu_fwd(N, H, W, C, dy_, stats, False, dev_f32(gamma), dev_f32(beta), None if res is None else dev_bf16(res), relu, 1e-5, a, sm, si,
                    rm, rv, 0.1, relu_mask=mask)
    if relu:   # bit i of byte j says whether stored output 8j+i is positive
        bits = np.unpackbits(mask.cpu().numpy(), bitorder="little").astype(bool)
        assert np.array_equal(bits, host(a).reshape(-1) > 0)
    assert_close(sm, mean, "mean", 1e-5, 1e-5)
    assert_close(si, invstd, "invstd", 1e-4, 1e-4)
    assert_close(a, a_ref, "a")
    assert_close(rm, 0.1 * mean, "running mean", 1e-5, 1e-5)
    assert_close(rv, 0.9 + 0.1 * var * M / (M - 1), "running var", 1e-4, 1e-4)

    # backward, teacher-forced with the oracle's stored forward output as the ReLU mask
    dy_ref, dres_ref, dg_ref, db_ref = oracle.bn_relu_bwd(da1, da2, y, a_ref, gamma, mean32, invstd32, relu, use_res)
    dyo = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    dres = torch.empty(shape, dtype=torch.bfloat16, device="cuda") if use_res else None
    dg, db = torch.full((C,), 1.0, device="cuda"), torch.full((C,), -2.0, device="cuda")
    ws = torch.empty(ctx.bn_relu_bwd_workspace_bytes(C), dtype=torch.uint8, device="cuda")
    ctx.bn_relu_bwd(N, H, W, C, dev_bf16(da1), None if da2 is None else dev_bf16(da2), dy_, dev_bf16(a_ref), dev_f32(gamma), dev_f32(mean32),
                    dev_f32(invstd32), relu, dyo, dres, dg, db, True, ws)
    assert_close(dyo, dy_ref, "dy")
    assert_close(dg, dg_ref + 1.0, "dgamma (accumulated)", 2e-3, 2e-3)
    assert_close(db, db_ref - 2.0, "dbeta (accumulated)", 2e-3, 2e-3)
    if use_res:
        assert_close(dres, oracle.round_bf16(dres_ref), "dres", 1e-6, 1e-6)
    if relu:
        # the same backward pass reading the bit mask of the oracle's stored output instead of the output tensor
        mask_ref = torch.from_numpy(np.packbits((a_ref.reshape(-1) > 0), bitorder="little")).cuda()
        dyo2 = torch.empty_like(dyo)
        dg2, db2 = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda")
        ctx.bn_relu_bwd(N, H, W, C, dev_bf16(da1), None if da2 is None else dev_bf16(da2), dy_, None, dev_f32(gamma), dev_f32(mean32),
                        dev_f32(invstd32), relu, dyo2, None, dg2, db2, False, ws, relu_mask=mask_ref)
        assert_close(dyo2, host(dyo), "dy (mask)", 1e-5, 1e-2)   # same arithmetic; the channel sums differ in summation order only
        assert_close(dg2, dg_ref, "dgamma (mask)", 2e-3, 2e-3)
    assert ctx.device_status() == 0


# (groups, rows per group, channels): ragged tails, more groups than fit the look-ahead, one chunk per block at most,
# idle threads at 160 channels, and a 64-channel case whose groups are large enough to be taken one at a time
BN_GROUP_SHAPES = [(4, 2048, 64), (3, 1000, 160), (8, 96, 512), (1, 4096, 128), (5, 16 * 1024, 64), (2, 640, 8)]


@pytest.mark.parametrize("shape", BN_GROUP_SHAPES, ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("relu,use_res", [(True, False), (True, True), (False, False)])
def test_bn_relu_bwd_groups(ctx, shape, relu, use_res):
    """Several statistics groups (micro-batches) back to back, each differentiated with its own statistics, both passes
    in one cooperative launch: every group against the oracle, the parameter gradients against the sum over groups."""
    G, M, C = shape
    r = wl.rng_for(14, f"bng{shape}{relu}{use_res}")
    y = wl.to_bf16_grid(r.standard_normal((G, M, C)) * (0.5 + r.random(C)) + 1.5 * r.standard_normal((G, 1, C)))
    da1 = wl.to_bf16_grid(r.standard_normal((G, M, C)))
    da2 = wl.to_bf16_grid(r.standard_normal((G, M, C))) if use_res else None
    gamma = (1.0 + 0.3 * r.standard_normal(C)).astype(np.float32)
    beta = (0.2 * r.standard_normal(C)).astype(np.float32)
    means, invstds, a_ref, dy_ref, dres_ref = [], [], [], [], []
    dg_ref, db_ref = np.zeros(C), np.zeros(C)
    for g in range(G):
        mean, _, invstd = oracle.bn_stats(y[g], 1e-5)
        mean, invstd = oracle.round_f32(mean), oracle.round_f32(invstd)
        a = oracle.round_bf16(oracle.bn_relu_apply(y[g], mean, invstd, gamma, beta, None, relu))
        q = oracle.bn_relu_bwd(da1[g], None if da2 is None else da2[g], y[g], a, gamma, mean, invstd, relu, use_res)
        means.append(mean); invstds.append(invstd); a_ref.append(a); dy_ref.append(q[0]); dres_ref.append(q[1])
        dg_ref += q[2]; db_ref += q[3]
    mask = torch.from_numpy(np.packbits(np.stack(a_ref).reshape(-1) > 0, bitorder="little")).cuda() if relu else None
    dyo = torch.full((G, M, C), float("nan"), dtype=torch.bfloat16, device="cuda")
    dres = torch.full((G, M, C), float("nan"), dtype=torch.bfloat16, device="cuda") if use_res else None
    dg, db = torch.full((C,), 1.0, device="cuda"), torch.full((C,), -2.0, device="cuda")
    ws = torch.full((ctx.bn_relu_bwd_groups_workspace_bytes(C, G),), 0x5A, dtype=torch.uint8, device="cuda")   # stale contents must not matter
    args = (G, M, C, dev_bf16(da1), None if da2 is None else dev_bf16(da2), dev_bf16(y), dev_f32(gamma), dev_f32(np.stack(means)),
            dev_f32(np.stack(invstds)), relu, dyo, dres, dg, db)
    ctx.bn_relu_bwd_groups(*args, True, mask, ws)
    assert ctx.device_status() == 0
    assert_close(dyo, np.stack(dy_ref), "dy")
    if use_res:
        assert_close(dres, oracle.round_bf16(np.stack(dres_ref)), "dres", 1e-6, 1e-6)
    assert_close(dg, dg_ref + 1.0, "dgamma (accumulated)", 2e-3, 2e-3)
    assert_close(db, db_ref - 2.0, "dbeta (accumulated)", 2e-3, 2e-3)
    # overwrite mode, and a second call on the same workspace
    ctx.bn_relu_bwd_groups(*args, False, mask, ws)
    assert ctx.device_status() == 0
    assert_close(dg, dg_ref, "dgamma", 2e-3, 2e-3)
    assert_close(db, db_ref, "dbeta", 2e-3, 2e-3)
    assert_close(dyo, np.stack(dy_ref), "dy (second call)")


def test_bn_large_mean_small_spread(ctx):
    # |mean| ~ 50x the spread: E[y^2] - E[y]^2 must not lose the variance
    N, H, W, C = 8, 16, 16, 16
    k = wl.rng_for(4, "k").integers(-4, 5, size=(N, H, W, C))
    y = (16.0 + k / 8.0).astype(np.float32)   # exactly representable in bf16
    mean, var, invstd = oracle.bn_stats(y, 1e-5)
    a = torch.empty((N, H, W, C), dtype=torch.bfloat16, device="cuda")
    stats = torch.zeros(2 * C, dtype=torch.float64, device="cuda")
    sm, si = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    ctx.bn_relu_fwd(N, H, W, C, dev_bf16(y), stats, False, dev_f32(np.ones(C)), dev_f32(np.zeros(C)), None, False, 1e-5, a, sm, si)
    assert_close(si, invstd, "invstd", 1e-4, 1e-4)
    assert_close(a, oracle.bn_relu_apply(y, mean, invstd, np.ones(C), np.zeros(C), None, False), "a")


def test_bn_with_conv_fused_statistics(ctx):
    shape = (8, 32, 32, 64, 64, 3, 1)
    N, H, W, C, K, R, st = shape
    x, w, _ = wl.conv_problem(5, *shape)
    y = torch.empty((N, H, W, K), dtype=torch.bfloat16, device="cuda")
    stats = torch.zeros(2 * K, dtype=torch.float64, device="cuda")
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y, ch_stats=stats)
    a = torch.empty_like(y)
    sm, si = torch.empty(K, device="cuda"), torch.empty(K, device="cuda")
    ctx.bn_relu_fwd(N, H, W, K, y, stats, True, dev_f32(np.ones(K)), dev_f32(np.zeros(K)), None, True, 1e-5, a, sm, si)
    yh = host(y)
    mean, var, invstd = oracle.bn_stats(yh, 1e-5)
    assert_close(si, invstd, "invstd", 1e-4, 1e-4)
    assert_close(a, oracle.bn_relu_apply(yh, mean, invstd, np.ones(K), np.zeros(K), None, True), "a")


# ------------------------------------------------------------------------------ small kernels
def test_avgpool_pad_bias(ctx):
    r = wl.rng_for(6, "pool")
    a = wl.to_bf16_grid(r.standard_normal((5, 4, 4, 64)))
    pooled = torch.empty((5, 64), dtype=torch.bfloat16, device="cuda")
    ctx.avgpool_fwd(5, 16, 64, dev_bf16(a), pooled)
    assert_close(pooled, oracle.avgpool_fwd(a), "pooled")
    g = wl.to_bf16_grid(r.standard_normal((5, 64)))
    da = torch.empty((5, 4, 4, 64), dtype=torch.bfloat16, device="cuda")
    ctx.avgpool_bwd(5, 16, 64, dev_bf16(g), da)
    assert np.array_equal(host(da), oracle.round_bf16(oracle.avgpool_bwd(g, 4, 4)))
    x = wl.to_bf16_grid(r.standard_normal((7, 5, 5, 3)))
    xp = torch.full((7, 5, 5, 16), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.pad_channels(7 * 25, 3, 16, dev_bf16(x), xp)
    assert np.array_equal(host(xp)[..., :3], x) and np.all(host(xp)[..., 3:] == 0)
    # patch matrix of the 3x3 / pad 1 window: column (r*3+s)*3 + ch holds x[h+r-1, w+s-1, ch]
    xc = torch.full((7, 5, 5, 32), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.im2col_3x3(7, 5, 5, 3, 32, dev_bf16(x), xc)
    xpad = np.zeros((7, 7, 7, 3), np.float32)
    xpad[:, 1:6, 1:6, :] = x
    ref = np.zeros((7, 5, 5, 32), np.float32)
    for rr in range(3):
        for ss in range(3):
            ref[..., (rr * 3 + ss) * 3:(rr * 3 + ss) * 3 + 3] = xpad[:, rr:rr + 5, ss:ss + 5, :]
    assert np.array_equal(host(xc), ref)
    dz = wl.to_bf16_grid(r.standard_normal((130, 128)))
    db = torch.ones(100, device="cuda")
    ctx.bias_grad(130, 100, 128, dev_bf16(dz), db, True)
    assert_close(db, 1.0 + dz[:, :100].astype(np.float64).sum(0), "db", 1e-5, 1e-5)


@pytest.mark.parametrize("n,classes,pitch", [(128, 100, 128), (7, 10, 16), (256, 100, 104)])
def test_softmax_xent(ctx, n, classes, pitch):
    r = wl.rng_for(7, f"sm{n}")
    z = (r.standard_normal((n, pitch)) * 3).astype(np.float32)
    labels = r.integers(0, classes, n).astype(np.int32)
    loss_ref, dz_ref = oracle.softmax_xent(z[:, :classes], labels, 1.0 / n)
    loss = torch.zeros(1, device="cuda")
    dz = torch.full((n, pitch), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.softmax_xent_fwd_bwd(n, classes, dev_f32(z), pitch, torch.from_numpy(labels).cuda(), 1.0 / n, 1.0 / n, loss, dz, pitch)
    assert abs(loss.item() - loss_ref) <= 1e-5 * abs(loss_ref)
    assert_close(dz[:, :classes], dz_ref, "dlogits")
    assert np.all(host(dz)[:, classes:] == 0)
    assert ctx.device_status() == 0


def test_softmax_xent_hand_values_and_bad_label(ctx):
    z = torch.zeros((4, 104), device="cuda")
    labels = torch.tensor([0, 7, 50, 99], dtype=torch.int32, device="cuda")
    loss = torch.zeros(1, device="cuda")
    dz = torch.empty((4, 104), dtype=torch.bfloat16, device="cuda")
    ctx.softmax_xent_fwd_bwd(4, 100, z, 104, labels, 0.25, 1.0, loss, dz, 104)
    assert abs(loss.item() - np.log(100.0)) < 1e-5
    d = host(dz)
    assert d[1, 7] == oracle.round_bf16(np.array([-0.99]))[0] and d[1, 8] == oracle.round_bf16(np.array([0.01]))[0]
    assert ctx.device_status() == 0
    labels[2] = 100
    ctx.softmax_xent_fwd_bwd(4, 100, z, 104, labels, 0.25, 1.0, loss, dz, 104)
    assert ctx.device_status() == 8       # B2C_ERR_BAD_LABEL, then cleared
    assert ctx.device_status() == 0


def test_sgd_momentum(ctx):
    count = 1000 * 4 + 4
    r = wl.rng_for(8, "sgd")
    w = r.standard_normal(count).astype(np.float32)
    v = (0.1 * r.standard_normal(count)).astype(np.float32)
    g = (8 * 0.05 * r.standard_normal(count)).astype(np.float32)
    w_ref, v_ref = oracle.sgd_momentum(w, v, g, 1.0 / 8, 0.1, 0.9, 5e-4)
    dw, dv, dg = dev_f32(w), dev_f32(v), dev_f32(g)
    wb = torch.empty(count, dtype=torch.bfloat16, device="cuda")
    ctx.grad_accum_sgd_momentum(count, dw, dv, dg, 1.0 / 8, 0.1, 0.9, 5e-4, wb, True)
    rel_w, _ = errors(host(dw), w_ref)
    rel_v, _ = errors(host(dv), v_ref)
    assert rel_w <= SGD_REL and rel_v <= SGD_REL, (rel_w, rel_v)
    assert torch.equal(wb, dw.to(torch.bfloat16))       # bf16 copy = RNE of the new master, bit exact
    assert torch.count_nonzero(dg).item() == 0
    # hand value
    one = lambda x: torch.full((4,), x, device="cuda")
    w1, v1, g1 = one(1.0), one(0.5), one(0.2)
    ctx.grad_accum_sgd_momentum(4, w1, v1, g1, 1.0, 0.1, 0.9, 5e-4, None, False)
    assert abs(v1[0].item() - 0.6505) < 1e-6 and abs(w1[0].item() - 0.93495) < 1e-6 and abs(g1[0].item() - 0.2) < 1e-7


def test_bounded_wait_reports_timeout(ctx):
    # A spin budget of one poll cannot outlast a TMA round trip: the kernel must wind down, report
    # B2C_ERR_DEVICE_TIMEOUT and leave the context usable.  Nothing hangs: every wait is bounded.
    shape = (8, 32, 32, 64, 64, 3, 1)
    x, w, _ = wl.conv_problem(9, *shape)
    y = torch.zeros((8, 32, 32, 64), dtype=torch.bfloat16, device="cuda")
    ctx.set_spin_limit(1)
    try:
        ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y)
        status = ctx.device_status()
    finally:
        ctx.set_spin_limit(1 << 22)
    assert status == 7
    ctx.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y)
    assert ctx.device_status() == 0
    assert_close(y, oracle.conv2d_fwd(x, w, 1, 1), "y after recovery")


@pytest.mark.parametrize("mode", ["0", "1"])
def test_conv_full_halo_on_and_off(mode, monkeypatch):
    """3x3 stride-1 layers large enough for full-halo stages (one framed 8x16 tile per channel block serves all nine
    taps; single CTAs at 64 channels, CTA pairs at 128), with the mode switched off and on: same results."""
    from paper_2503_23186_b200 import binding
    monkeypatch.setenv("B2C_FULL_HALO", mode)
    c = binding.Context(0)
    try:
        for shape in [(64, 32, 32, 64, 64, 3, 1), (160, 16, 16, 128, 128, 3, 1), (40, 16, 32, 64, 64, 3, 1)]:
            N, H, W, C, K, R, st = shape
            x, w, g = wl.conv_problem(13, *shape)
            ref = oracle.conv2d_fwd(x, w, st, 1)
            y = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            stats = torch.zeros(2 * K, dtype=torch.float64, device="cuda")
            c.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y, ch_stats=stats)
            assert c.device_status() == 0
            assert_close(y, ref, f"y {shape} full_halo={mode}")
            ys = host(y).reshape(-1, K)
            np.testing.assert_allclose(host(stats)[:K], ys.sum(0), rtol=1e-5, atol=1e-3 * np.sqrt(ys.shape[0]))
            np.testing.assert_allclose(host(stats)[K:], (ys * ys).sum(0), rtol=1e-4)
            dx = torch.full(x.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            c.conv2d_dgrad(_desc(*shape), dev_bf16(g), _dgrad_weights(c, w), dx)
            assert c.device_status() == 0
            assert_close(dx, oracle.conv2d_dgrad(g, w, x.shape, st, 1), f"dx {shape} full_halo={mode}")
    finally:
        c.close()


@pytest.mark.parametrize("mode", ["0", "2"])
def test_conv_cta_pairs_forced_on_and_off(mode, monkeypatch):
    """The forward / data-gradient kernel on single CTAs only (0) and on CTA pairs wherever possible (2): same results."""
    from paper_2503_23186_b200 import binding
    monkeypatch.setenv("B2C_CTA_PAIRS", mode)
    c = binding.Context(0)
    try:
        for shape in [(8, 32, 32, 64, 64, 3, 1), (4, 16, 16, 128, 256, 3, 1), (4, 16, 16, 256, 128, 3, 1), (8, 32, 32, 64, 128, 3, 2),
                      (2, 16, 16, 160, 160, 3, 1), (6, 4, 4, 128, 64, 3, 1)]:
            N, H, W, C, K, R, st = shape
            x, w, g = wl.conv_problem(11, *shape)
            ref = oracle.conv2d_fwd(x, w, st, (R - 1) // 2)
            y = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            stats = torch.zeros(2 * K, dtype=torch.float64, device="cuda")
            c.conv2d_fwd(_desc(*shape), dev_bf16(x), dev_bf16(w), y, ch_stats=stats)
            assert c.device_status() == 0
            assert_close(y, ref, f"y {shape} pairs={mode}")
            ys = host(y).reshape(-1, K)
            np.testing.assert_allclose(host(stats)[:K], ys.sum(0), rtol=1e-5, atol=1e-3 * np.sqrt(ys.shape[0]))
            dx = torch.full(x.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            c.conv2d_dgrad(_desc(*shape), dev_bf16(g), _dgrad_weights(c, w), dx)
            assert c.device_status() == 0
            assert_close(dx, oracle.conv2d_dgrad(g, w, x.shape, st, (R - 1) // 2), f"dx {shape} pairs={mode}")
    finally:
        c.close()
