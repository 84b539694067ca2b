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
    """binding.Net look-alike backed by the fp64 oracle: flat gradient tensor `g`, train_step, apply_update."""

    def __init__(self, spec, params):
        self.spec = spec
        self.params = {k: v.astype(np.float64) for k, v in params.items()}
        self.vel = {k: np.zeros_like(v) for k, v in self.params.items()}
        self.names = sorted(self.params)
        self.g = torch.zeros(sum(self.params[k].size for k in self.names), dtype=torch.float64)

    def train_step(self, images, labels, n_micro, lr, mu, wd, update=True):
        n = images.shape[0] // n_micro
        flat, loss = [], 0.0
        sums = {k: np.zeros_like(v) for k, v in self.params.items()}
        for m in range(n_micro):
            fw = onet.forward(self.spec, self.params, images[m * n:(m + 1) * n], labels[m * n:(m + 1) * n], rounding=False)
            gr, _ = onet.backward(self.spec, self.params, fw, rounding=False)
            for k in sums:
                sums[k] += gr[k]
            loss += fw["loss"] / n_micro
        for k in self.names:
            flat.append(sums[k].reshape(-1))
        self.g += torch.from_numpy(np.concatenate(flat))
        if update:
            self.apply_update(n_micro, lr, mu, wd)
        return loss

    def apply_update(self, n_avg, lr, mu, wd):
        import oracle
        off, g = 0, self.g.numpy()
        for k in self.names:
            sz = self.params[k].size
            w, v = oracle.sgd_momentum(self.params[k], self.vel[k], g[off:off + sz].reshape(self.params[k].shape), 1.0 / n_avg, lr, mu, wd)
            self.params[k], self.vel[k] = w, v
            off += sz
        self.g.zero_()


def _problem():
    spec = wl.tiny_net_spec(classes=10, hw=8, c=4, width=4, width2=8)
    params = wl.perturb_bn_params(wl.init_params(spec, 7), 7)
    images, labels = wl.image_batch(7, 16, hw=8, c=4, classes=10)
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
