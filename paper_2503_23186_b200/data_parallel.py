"""Data-parallel driver of the training step: one process per GPU, replicas exchange gradient sums once per update.

Algorithm 1: every replica runs forward, loss and backward on its own share of the mini-batch, gradients are
synchronised across devices (mean over all replicas and micro-batches), and the parameters are updated.  Two forms of
the exchange are implemented, both host logic over `torch.distributed` collectives (NCCL on GPUs, gloo in the CPU tests):

* `dp_train_step`: a sum all-reduce of the whole flat fp32 gradient array, then the same fused update on every replica.
* `dp_train_step_sharded`: gradient synchronisation fused with the update.  The flat parameter arrays are cut into
  buckets in reverse layer order (the order in which the backward pass finishes them); each bucket is reduce-scattered
  as soon as its gradients are final, so the exchange of the late layers overlaps the backward pass of the early ones;
  every replica then updates only its own 1/world slice of each bucket (fp32 master, momentum: the optimiser state is
  sharded), and the slices of the bf16 weight copy are all-gathered, which moves half the bytes of the fp32 masters.
  A replica's fp32 masters and momentum are current only inside the slices it owns; `gather_masters` collects them.

`net` is any object with the interface of `binding.Net` (train_step / apply_update / apply_update_range /
refresh_derived_weights and the flat tensors g, w_bf16); the CPU tests pass an oracle-backed stand-in.
"""
from __future__ import annotations

ALIGN = 8   # elements: slices of the flat arrays start on 32-byte (fp32) / 16-byte (bf16) boundaries


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


# ------------------------------------------------------------------------------------------------------------------
# gradient synchronisation fused with the update
# ------------------------------------------------------------------------------------------------------------------
def bucket_plan(param_count: int, layer_ranges, n_buckets: int):
    """Cuts the flat parameter arrays [0, param_count) into buckets, listed in the order the backward pass completes them.

    layer_ranges: [(begin, end)] element ranges of the filter banks of successive weight layers (layer order = array
    order; begins are multiples of ALIGN).  The weight region is cut at filter-bank starts into at most n_buckets
    pieces of roughly equal size, taken from the last layer backwards.  Everything behind the last filter bank
    (BatchNorm scale / shift of every layer, the classifier bias) is final only when the whole backward pass is: it
    forms one more bucket at the end of the list.  Returns [(begin, end, first_layer)]: first_layer = index into
    layer_ranges of the earliest layer with parameters in the bucket, whose backward pass completes the bucket."""
    if n_buckets < 1 or param_count < 1 or not layer_ranges:
        raise ValueError("bad bucket plan arguments")
    ranges = [(int(b), int(e)) for b, e in layer_ranges]
    if ranges[0][0] != 0 or any(b % ALIGN for b, _ in ranges) or any(r[0] < l[1] for l, r in zip(ranges, ranges[1:])):
        raise ValueError("layer ranges must start at 0, ascend without overlap and begin on multiples of ALIGN")
    w_end = -(-ranges[-1][1] // ALIGN) * ALIGN
    if w_end > param_count:
        raise ValueError("layer ranges exceed the parameter count")
    target = w_end / n_buckets
    buckets, end, acc = [], w_end, 0
    for idx in range(len(ranges) - 1, 0, -1):
        acc = end - ranges[idx][0]
        if acc >= target and len(buckets) < n_buckets - 1:
            buckets.append((ranges[idx][0], end, idx))
            end = ranges[idx][0]
    buckets.append((0, end, 0))
    if w_end < param_count:
        buckets.append((w_end, param_count, 0))
    return buckets


def slice_of(begin: int, end: int, rank: int, world: int):
    """Replica `rank`'s slice [b, e) of bucket [begin, end): equal slices of ceil(len / world) rounded up to ALIGN, the
    last ones possibly shorter or empty."""
    n = end - begin
    per = -(-n // world)
    per = -(-per // ALIGN) * ALIGN
    b = min(begin + rank * per, end)
    e = min(b + per, end)
    return b, e


def _reduce_scatter_sum(flat_bucket, rank, world, group):
    """Sum over replicas of a bucket; on return this replica's slice of `flat_bucket` holds the total (other slices are
    unspecified).  NCCL: reduce-scatter over padded equal slices; backends without reduce-scatter (gloo): all-reduce."""
    import torch
    import torch.distributed as dist
    n = flat_bucket.numel()
    per = slice_of(0, n, 0, world)[1]
    backend = dist.get_backend(group)
    if backend == "nccl" and per * world == n:
        out = flat_bucket[rank * per:(rank + 1) * per]
        dist.reduce_scatter_tensor(out, flat_bucket, op=dist.ReduceOp.SUM, group=group)
        return
    if backend == "nccl":
        padded = torch.zeros(per * world, dtype=flat_bucket.dtype, device=flat_bucket.device)
        padded[:n] = flat_bucket
        out = torch.empty(per, dtype=flat_bucket.dtype, device=flat_bucket.device)
        dist.reduce_scatter_tensor(out, padded, op=dist.ReduceOp.SUM, group=group)
        b, e = slice_of(0, n, rank, world)
        flat_bucket[b:e] = out[:e - b]
        return
    dist.all_reduce(flat_bucket, op=dist.ReduceOp.SUM, group=group)


def _all_gather_slices(flat_bucket, rank, world, group):
    """Every replica contributes its slice of the bucket; on return the whole bucket is current everywhere."""
    import torch
    import torch.distributed as dist
    n = flat_bucket.numel()
    per = slice_of(0, n, 0, world)[1]
    if per * world == n:
        dist.all_gather_into_tensor(flat_bucket, flat_bucket[rank * per:(rank + 1) * per].clone(), group=group)
        return
    mine = torch.zeros(per, dtype=flat_bucket.dtype, device=flat_bucket.device)
    b, e = slice_of(0, n, rank, world)
    mine[:e - b] = flat_bucket[b:e]
    gathered = torch.empty(per * world, dtype=flat_bucket.dtype, device=flat_bucket.device)
    dist.all_gather_into_tensor(gathered, mine, group=group)
    flat_bucket.copy_(gathered[:n])


def dp_train_step_sharded(net, images, labels, n_micro, lr, momentum, wd, buckets, group=None, comm_stream=None):
    """One optimiser step with the gradient exchange fused with the update (see the module docstring).

    buckets: bucket_plan(...) for this net and world size.  comm_stream (GPU only): a torch stream for the collectives;
    with it and a net that records per-bucket gradient-ready events (`net.set_buckets(buckets)`), bucket k's reduce-scatter
    starts as soon as the backward pass has finished the bucket's first layer, while the backward pass continues."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    rank = dist.get_rank(group) if world > 1 else 0
    if world == 1:
        return net.train_step(images, labels, n_micro, lr, momentum, wd, update=True)
    events = getattr(net, "bucket_events", None)
    use_stream = comm_stream is not None and events is not None
    loss = net.train_step(images, labels, n_micro, lr, momentum, wd, update=False)
    n_avg = n_micro * world
    for k, (begin, end, _first_layer) in enumerate(buckets):
        ctx = torch.cuda.stream(comm_stream) if use_stream else _null()
        with ctx:
            if use_stream:
                net.bucket_wait(k, comm_stream)                        # the bucket's gradients are final on the compute stream
            _reduce_scatter_sum(net.g[begin:end], rank, world, group)   # this replica's slice now holds the sum over replicas
            b, e = slice_of(begin, end, rank, world)
            if e > b:
                net.apply_update_range(b, e, n_avg, lr, momentum, wd)   # fp32 master + momentum of the owned slice; bf16 copy of it
            net.g[begin:end].zero_()                                    # the other replicas' slices carry stale partial sums
            _all_gather_slices(net.w_bf16[begin:end], rank, world, group)
    if use_stream:
        torch.cuda.current_stream().wait_stream(comm_stream)
    net.refresh_derived_weights()                                       # the data-gradient layout of the bf16 copy
    return loss


def gather_masters(net, buckets, group=None):
    """Collects the fp32 masters and momentum of all replicas' slices (for a checkpoint or an evaluation): after it
    every replica holds the full current arrays."""
    import torch.distributed as dist
    world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if world == 1:
        return
    rank = dist.get_rank(group)
    for begin, end, _ in buckets:
        _all_gather_slices(net.w[begin:end], rank, world, group)
        _all_gather_slices(net.v[begin:end], rank, world, group)


class _null:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False
