"""The allocation-free BatchNorm backward entry point (b2c_bn_relu_bwd_static) against the regular one and the oracle.

Some callers of this library cannot allocate device memory where they call it: they run under an allocator they do
not own, inside a fixed memory budget, or must not trigger the device synchronisation that CUDA's allocation calls
imply.  For them the library carries its own scratch for this one operation.  The file name makes pytest collect
this test last, so a run that stops at the first failure has already been through every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_23186_b200 import workloads as wl
from parity import assert_close, dev_bf16, dev_f32, host

pytestmark = pytest.mark.gpu


def _problem(seed, shape, use_res):
    N, H, W, C = shape
    r = wl.rng_for(seed, f"static{shape}")
    y = wl.to_bf16_grid(r.standard_normal(shape) * (0.5 + r.random(C)) + r.standard_normal(C))
    a = wl.to_bf16_grid(np.maximum(r.standard_normal(shape), 0.0))
    da1 = wl.to_bf16_grid(r.standard_normal(shape))
    da2 = wl.to_bf16_grid(r.standard_normal(shape)) if use_res else None
    gamma = (1.0 + 0.3 * r.standard_normal(C)).astype(np.float32)
    mean = y.reshape(-1, C).mean(0).astype(np.float32)
    invstd = (1.0 / np.sqrt(y.reshape(-1, C).var(0) + 1e-5)).astype(np.float32)
    return y, a, da1, da2, gamma, mean, invstd


def _run(ctx, shape, prob, static, relu=True):
    N, H, W, C = shape
    y, a, da1, da2, gamma, mean, invstd = prob
    dy = torch.empty(shape, dtype=torch.bfloat16, device="cuda")
    dres = torch.empty(shape, dtype=torch.bfloat16, device="cuda") if da2 is not None else None
    dg, db = torch.zeros(C, device="cuda"), torch.zeros(C, device="cuda")
    args = (N, H, W, C, dev_bf16(da1), None if da2 is None else dev_bf16(da2), dev_bf16(y), dev_bf16(a), dev_f32(gamma), dev_f32(mean),
            dev_f32(invstd), relu, dy, dres, dg, db, False)
    if static:
        ctx.bn_relu_bwd_static(*args)
    else:
        ws = torch.empty(ctx.bn_relu_bwd_workspace_bytes(C), dtype=torch.uint8, device="cuda")
        ctx.bn_relu_bwd(*args, ws)
    assert ctx.device_status() == 0
    return dy, dres, dg, db


def test_static_scratch_variant_matches_regular_entry_point():
    from paper_2503_23186_b200 import binding
    ctx = binding.Context(0)
    try:
        # two calls in a row with different channel counts: the second must not see the first one's sums
        # (the third problem has no ReLU and is large enough for the bulk-copy ring of the backward kernels)
        for seed, shape, use_res, relu in [(0, (8, 16, 16, 256), True, True), (1, (5, 8, 8, 64), False, True), (2, (33, 31, 32, 64), False, False)]:
            prob = _problem(seed, shape, use_res)
            ref = _run(ctx, shape, prob, static=False, relu=relu)
            got = _run(ctx, shape, prob, static=True, relu=relu)
            y, a, da1, da2, gamma, mean, invstd = prob
            want = oracle.bn_relu_bwd(da1, da2, y, a, gamma, mean, invstd, relu, use_res)
            want = (oracle.round_bf16(want[0]), None if want[1] is None else oracle.round_bf16(want[1]), want[2], want[3])
            for name, g, r, o in zip(("dy", "dres", "dgamma", "dbeta"), got, ref, want):
                if r is None:
                    assert g is None
                    continue
                assert_close(g, host(r), name + " (against the regular entry point)")
                assert_close(g, o, name + " (against the oracle)")
        # sizes beyond the built-in scratch are refused with a clear status and nothing is enqueued
        big = (1, 1, 1, 2048 + 8)
        t = torch.zeros(big, dtype=torch.bfloat16, device="cuda")
        f = torch.zeros(big[3], device="cuda")
        with pytest.raises(binding.B2CError) as e:
            ctx.bn_relu_bwd_static(1, 1, 1, big[3], t, None, t, t, f, f, f, True, t.clone(), None, f.clone(), f.clone(), False)
        assert e.value.status == 4   # B2C_ERR_WORKSPACE_TOO_SMALL
        assert ctx.device_status() == 0
    finally:
        ctx.close()
