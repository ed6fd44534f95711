"""Intra-group data parallelism of one stage (Asteroid Section 3.2, Eq. 5), host side.

The devices of a group hold replicas of the stage.  Every device runs its share y_d of each micro-batch of B samples
through its own replica (forward, backward, accumulate, through the C ABI as in a single-device round); before the update
the accumulated gradients are synchronised: device d scales its arena by y_d / B and the group sums the arenas, so that
every replica applies the gradient of the whole micro-batch mean and the replicas stay identical.  (BatchNorm statistics
are then those of a device's own share, as in any data-parallel run without synchronised BatchNorm.)

The library does no communication: this module does the scaling and the AllReduce with torch.distributed (NCCL on GPUs),
on the stream torch uses, over a tensor view of the arena that `asteroid_stage_grad_buffer` returns.
"""
import torch
import torch.distributed as dist


def group_shares(batch, weights):
    """Split a micro-batch of `batch` samples over the devices of a group in proportion to `weights` (for instance the
    inverse of their measured step times): integer shares that sum to `batch`, largest remainders first, every
    device at least one sample when batch >= len(weights)."""
    n = len(weights)
    if n < 1 or batch < 0 or any(w <= 0 for w in weights):
        raise ValueError("weights must be positive")
    tot = float(sum(weights))
    raw = [batch * w / tot for w in weights]
    y = [int(r) for r in raw]
    if batch >= n:
        y = [max(1, v) for v in y]
    order = sorted(range(n), key=lambda i: (-(raw[i] - int(raw[i])), i))
    k = 0
    while sum(y) < batch:
        y[order[k % n]] += 1
        k += 1
    order = sorted(range(n), key=lambda i: (-y[i], i))
    k = 0
    while sum(y) > batch:
        i = order[k % n]
        if y[i] > (1 if batch >= n else 0):
            y[i] -= 1
        k += 1
    return y


def allreduce_weighted(t, share, batch, group=None):
    """In place: t <- sum over the group's ranks of t_rank * share_rank / batch.  Works on any tensor torch.distributed
    can reduce (CUDA tensors over NCCL, CPU tensors over gloo)."""
    t.mul_(float(share) / float(batch))
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t


class _DeviceFloats:
    """A float32 device array given by address and length, presented through the CUDA array interface."""

    def __init__(self, ptr, n):
        self.__cuda_array_interface__ = {"shape": (int(n),), "typestr": "<f4", "data": (int(ptr), False), "version": 2}


def grad_tensor(handle):
    """torch view (no copy) of a stage's accumulated-gradient arena."""
    from . import binding
    ptr, n = binding.asteroid_stage_grad_buffer(handle)
    return torch.as_tensor(_DeviceFloats(ptr, n), device="cuda")


def allreduce_gradients(handle, share, batch, group=None):
    """Gradient synchronisation of a data-parallel group member: call between the last `asteroid_stage_accumulate` of a
    round and `asteroid_stage_step`, on the torch stream whose handle the stage calls were given."""
    return allreduce_weighted(grad_tensor(handle), share, batch, group)
