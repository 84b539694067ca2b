"""Data-parallel driver of the training step: one process per GPU, replicas exchange gradient sums once per update.

Algorithm 1: every replica runs forward, loss and backward on its own share of the mini-batch, gradients are
synchronised across devices (mean over all replicas and micro-batches), and every replica applies the same update.
The exchange is a sum all-reduce of the flat fp32 gradient array; the division by the number of micro-batches of
all replicas happens inside the fused update kernel.  Host logic only: `net` is any object with the interface of
`binding.Net` (train_step / apply_update / g).
"""
from __future__ import annotations


def shard_bounds(total: int, rank: int, world: int):
    """[begin, end) of the images replica `rank` processes; every replica gets the same count."""
    if total % world:
        raise ValueError("the global batch must divide evenly over the replicas")
    per = total // world
    return rank * per, (rank + 1) * per


def dp_train_step(net, images, labels, n_micro, lr, momentum, wd, group=None):
    """One optimiser step on this replica's shard (images/labels already local).  Without an initialised process
    group (or with one replica) this is the library's fused single-call step."""
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if world == 1:
        return net.train_step(images, labels, n_micro, lr, momentum, wd, update=True)
    loss = net.train_step(images, labels, n_micro, lr, momentum, wd, update=False)
    dist.all_reduce(net.g, group=group)                      # sum of the replicas' gradient sums
    net.apply_update(n_micro * world, lr, momentum, wd)      # mean over all micro-batches of all replicas
    return loss
