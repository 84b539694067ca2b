"""World-size-2 run of the data-parallel driver on CPU (gloo): two replicas, each with its own shard, must end with
the parameters a single process obtains from the whole batch.  The replicas compute with the oracle (a stand-in with
the interface of binding.Net); what is tested is the host logic: sharding, the gradient exchange and the averaging."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import net as onet
from paper_2503_23186_b200 import data_parallel as dp
from paper_2503_23186_b200 import workloads as wl

LR, MU, WD = 0.1, 0.9, 5e-4


class OracleNet:
    """binding.Net look-alike backed by the fp64 oracle, with the library's flat-array layout: filter banks in layer
    order (each starting on a multiple of 8 elements), then the remaining parameters; `w` (master), `v`, `g` and the
    derived copy `w_bf16` the forward and backward passes read (kept in fp64 here: the host logic is what is tested)."""

    def __init__(self, spec, params):
        self.spec = spec
        weights = [f"w{i}" for i, L in enumerate(spec) if L["kind"] in ("conv", "fc")]
        self.names = weights + sorted(k for k in params if k not in weights)
        self.shapes = {k: params[k].shape for k in self.names}
        self.offsets, off = {}, 0
        for k in self.names:
            self.offsets[k] = off
            off += -(-params[k].size // 8) * 8
        self.param_count = off
        self._weights = weights
        self.w = torch.zeros(off, dtype=torch.float64)
        for k in self.names:
            self.w[self.offsets[k]:self.offsets[k] + params[k].size] = torch.from_numpy(params[k].astype(np.float64).reshape(-1))
        self.v = torch.zeros_like(self.w)
        self.g = torch.zeros_like(self.w)
        self.w_bf16 = self.w.clone()

    def weight_layer_ranges(self):
        return [(self.offsets[k], self.offsets[k] + int(np.prod(self.shapes[k]))) for k in self._weights]

    def _dict(self, flat):
        a = flat.numpy()
        return {k: a[self.offsets[k]:self.offsets[k] + int(np.prod(self.shapes[k]))].reshape(self.shapes[k]).copy() for k in self.names}

    @property
    def params(self):
        return self._dict(self.w)

    def train_step(self, images, labels, n_micro, lr, mu, wd, update=True):
        n = images.shape[0] // n_micro
        loss = 0.0
        used = self._dict(self.w_bf16)          # forward and backward read the derived copy, never the masters
        sums = {k: np.zeros(self.shapes[k]) for k in self.names}
        for m in range(n_micro):
            fw = onet.forward(self.spec, used, images[m * n:(m + 1) * n], labels[m * n:(m + 1) * n], rounding=False)
            gr, _ = onet.backward(self.spec, used, fw, rounding=False)
            for k in sums:
                sums[k] += gr[k]
            loss += fw["loss"] / n_micro
        for k in self.names:
            self.g[self.offsets[k]:self.offsets[k] + sums[k].size] += torch.from_numpy(sums[k].reshape(-1))
        if update:
            self.apply_update(n_micro, lr, mu, wd)
        return loss

    def apply_update_range(self, begin, end, n_avg, lr, mu, wd):
        import oracle
        w, v = oracle.sgd_momentum(self.w[begin:end].numpy(), self.v[begin:end].numpy(), self.g[begin:end].numpy(), 1.0 / n_avg, lr, mu, wd)
        self.w[begin:end] = torch.from_numpy(w)
        self.v[begin:end] = torch.from_numpy(v)
        self.g[begin:end] = 0.0
        self.w_bf16[begin:end] = self.w[begin:end]

    def apply_update(self, n_avg, lr, mu, wd):
        self.apply_update_range(0, self.param_count, n_avg, lr, mu, wd)

    def refresh_derived_weights(self):
        pass


def _problem(n_images=16):
    spec = wl.tiny_net_spec(classes=10, hw=8, c=4, width=4, width2=8)
    params = wl.perturb_bn_params(wl.init_params(spec, 7), 7)
    images, labels = wl.image_batch(7, n_images, hw=8, c=4, classes=10)
    return spec, params, images.astype(np.float64), labels


def _replica(rank, world, port, out):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec, params, images, labels = _problem()
        b, e = dp.shard_bounds(images.shape[0], rank, world)
        net = OracleNet(spec, params)
        dp.dp_train_step(net, images[b:e], labels[b:e], 2, LR, MU, WD)     # 2 micro-batches of 4 per replica
        out[rank] = {k: v.copy() for k, v in net.params.items()}
    finally:
        dist.destroy_process_group()


def test_two_replicas_match_single_process():
    spec, params, images, labels = _problem()
    ref = onet.train_step(spec, {k: v.astype(np.float64) for k, v in params.items()}, {k: np.zeros(v.shape) for k, v in params.items()},
                          images, labels, 4, LR, MU, WD, rounding=False)    # 4 micro-batches of 4 in one process
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_replica, args=(2, port, out), nprocs=2, join=True)
        got = {r: out[r] for r in (0, 1)}
    for k in params:
        np.testing.assert_allclose(got[0][k], ref["params"][k], rtol=1e-10, atol=1e-12)
        np.testing.assert_array_equal(got[0][k], got[1][k])                 # replicas stay in lock step


def test_shard_bounds():
    assert dp.shard_bounds(1024, 3, 8) == (384, 512)
    with pytest.raises(ValueError):
        dp.shard_bounds(10, 0, 3)


def test_single_replica_uses_fused_step():
    spec, params, images, labels = _problem()
    net = OracleNet(spec, params)
    dp.dp_train_step(net, images, labels, 4, LR, MU, WD)
    ref = onet.train_step(spec, {k: v.astype(np.float64) for k, v in params.items()}, {k: np.zeros(v.shape) for k, v in params.items()},
                          images, labels, 4, LR, MU, WD, rounding=False)
    for k in params:
        np.testing.assert_allclose(net.params[k], ref["params"][k], rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------------------------------------------------------
# gradient synchronisation fused with the update: reduce-scatter, update of the replica's own slice, all-gather
# ------------------------------------------------------------------------------------------------------------------
def _replica_sharded(rank, world, port, out, steps, n_buckets):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        spec, params, images, labels = _problem(24)
        b, e = dp.shard_bounds(images.shape[0], rank, world)
        plain, sharded = OracleNet(spec, params), OracleNet(spec, params)
        buckets = dp.bucket_plan(sharded.param_count, sharded.weight_layer_ranges(), n_buckets)
        n_micro = 2
        for _ in range(steps):
            # the replicated update on the same reduced gradients: the sum over replicas taken bucket by bucket, so that
            # the collective adds in the same order as in the sharded form (with three or more replicas the order in
            # which a ring all-reduce adds depends on where an element falls in the message)
            plain.train_step(images[b:e], labels[b:e], n_micro, LR, MU, WD, update=False)
            for lo, hi, _ in buckets:
                dist.all_reduce(plain.g[lo:hi])
            plain.apply_update(n_micro * world, LR, MU, WD)
            dp.dp_train_step_sharded(sharded, images[b:e], labels[b:e], n_micro, LR, MU, WD, buckets)
        copy_before_gather = sharded.w_bf16.clone()
        stale = float((sharded.w - plain.w).abs().max())      # masters outside the owned slices are not kept current
        dp.gather_masters(sharded, buckets)
        out[rank] = dict(plain_w=plain.w.numpy().copy(), plain_v=plain.v.numpy().copy(), copy=copy_before_gather.numpy().copy(),
                         w=sharded.w.numpy().copy(), v=sharded.v.numpy().copy(), g=float(sharded.g.abs().max()), stale=stale,
                         buckets=buckets)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,n_buckets", [(2, 3), (3, 2), (3, 1)])
def test_sharded_update_equals_replicated_update(world, n_buckets):
    """Two optimiser steps with the exchange fused with the update (bucketed reduce-scatter, update of the own slice,
    all-gather of the derived copy) leave every replica with exactly the weights the all-reduce form produces, bit for
    bit in fp64, and, once gathered, the same masters and momentum; both agree with one process on the whole batch."""
    port = 31500 + (os.getpid() % 2000) + 7 * world + n_buckets
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_replica_sharded, args=(world, port, out, 2, n_buckets), nprocs=world, join=True)
        got = {r: out[r] for r in range(world)}
    for r in range(world):
        np.testing.assert_array_equal(got[r]["copy"], got[r]["plain_w"])      # the copy every replica computes with
        np.testing.assert_array_equal(got[r]["w"], got[r]["plain_w"])         # masters and momentum after the gather
        np.testing.assert_array_equal(got[r]["v"], got[r]["plain_v"])
        np.testing.assert_array_equal(got[r]["w"], got[0]["w"])
        assert got[r]["g"] == 0.0
    assert max(got[r]["stale"] for r in range(world)) > 0.0                   # the state really was sharded
    assert len(got[0]["buckets"]) == min(n_buckets, 3) + 1                      # weight buckets + the tail
    # one process on the whole batch: the same numbers up to the order of the sum over replicas
    spec, params, images, labels = _problem(24)
    p = {k: v.astype(np.float64) for k, v in params.items()}
    vel = {k: np.zeros(v.shape) for k, v in params.items()}
    for _ in range(2):
        ref = onet.train_step(spec, p, vel, images, labels, 2 * world, LR, MU, WD, rounding=False)
        p, vel = ref["params"], ref["velocity"]
    probe = OracleNet(spec, params)
    flat = got[0]["w"]
    for k in params:
        off = probe.offsets[k]
        np.testing.assert_allclose(flat[off:off + params[k].size].reshape(params[k].shape), p[k], rtol=1e-10, atol=1e-12)


def test_bucket_plan_and_slices():
    ranges = [(0, 1000), (1000, 5000), (5000, 5800), (5808, 9000)]
    b = dp.bucket_plan(9100, ranges, 3)
    assert b == [(5808, 9000, 3), (1000, 5808, 1), (0, 1000, 0), (9000, 9100, 0)]
    assert dp.bucket_plan(9100, ranges, 1) == [(0, 9000, 0), (9000, 9100, 0)]
    # buckets tile the arrays exactly, in completion order of the backward pass (last layer first, the tail last)
    covered = sorted((x, y) for x, y, _ in b)
    assert covered[0][0] == 0 and covered[-1][1] == 9100 and all(l[1] == r[0] for l, r in zip(covered, covered[1:]))
    for world in (1, 2, 3, 8):
        for begin, end, _ in b:
            sl = [dp.slice_of(begin, end, r, world) for r in range(world)]
            assert sl[0][0] == begin and sl[-1][1] == end and all(l[1] == r[0] for l, r in zip(sl, sl[1:]))
            assert all((s0 - begin) % dp.ALIGN == 0 for s0, s1 in sl if s1 > s0)   # every non-empty slice starts aligned
    with pytest.raises(ValueError):
        dp.bucket_plan(9100, [(4, 1000)], 2)
