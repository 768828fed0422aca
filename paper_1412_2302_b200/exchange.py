"""The paper's exchange between replicas when every replica lives in its own process and GPU ("Data parallelism"
section and its figure): after each replica's update on its own minibatch, weights, biases and momentum are exchanged
and averaged, so that all replicas are equal again.

Across R processes that is an all-reduce(sum) of the parameter and momentum arrays followed by a multiplication by
1/R.  The collective is torch.distributed's (NCCL over NVLink on GPUs, gloo on CPU); the arrays are views into the
library's own device memory (AlexNet.param_views), so nothing is copied, and the multiplication, the bf16 copies and
the transposed filters are the library's scale-and-refresh kernel.

Two forms, equal in exact arithmetic for replicas that start the step identical (the paper's closing remark in that
section; checked to 1e-5 in the tests):

  exchange_and_average(rep)            after train_step: all-reduce w and v (8 bytes per parameter on the wire)
  exchange_then_average(rep)           after train_step, the paper's own two steps: every rank receives the other ranks'
                                       w and v into buffers of its own (all-gather), then averages them with its own
  allreduce_gradients_and_update(rep)  after forward_backward: all-reduce g (4 bytes per parameter), then one update
                                       with the mean gradient

  allreduce_gradients_overlapped_and_update(rep, comm_stream)
                                       the gradient form with the all-reduce of the FC weight gradients (96% of the
                                       bytes) issued from a second stream as soon as they exist, under the convolution
                                       layers' backward pass; only the rest is exchanged after the pass

`rep` is anything with param_views() -> (w, v, g) torch tensors, scale_and_refresh(scale) and apply_update(scale):
LocalReplica adapts an AlexNet handle; the CPU tests pass a stand-in that holds host tensors.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class LocalReplica:
    """Replica `replica` of an AlexNet handle as the exchange functions see it.  Collectives are queued behind the
    handle's compute stream, and the library's kernels behind the collectives."""

    def __init__(self, net, replica=0):
        self.net, self.replica = net, replica
        self._views = net.param_views(replica)

    def param_views(self):
        return self._views

    def stream(self):
        return torch.cuda.stream(self.net.compute_stream)

    def scale_and_refresh(self, scale):
        self.net.scale_and_refresh(self.replica, scale)

    def apply_update(self, grad_scale):
        self.net.apply_update(self.replica, grad_scale)

    def average_received(self, recv_w, recv_v, self_rank):
        self.net.average_received(self.replica, recv_w, recv_v, self_rank)

    def fc_range(self):
        return self.net.fc_range()

    def stream_wait_fc_gradients(self, stream):
        self.net.stream_wait_fc_gradients(stream)

    def wait_stream(self, stream):
        self.net.compute_stream.wait_stream(stream)


class _NoStream:
    def __enter__(self):
        return self

    def __exit__(self, *a):
        return False


def _initialised():
    return dist.is_available() and dist.is_initialized()


def _world(group):
    return dist.get_world_size(group) if _initialised() else 1


def exchange_and_average(rep, group=None):
    """Steps 2 and 3 of the paper's data-parallel figure over all ranks of `group`: every rank ends with the mean of
    all ranks' parameters and momenta (bitwise the same on every rank: the all-reduce delivers one sum to all)."""
    world = _world(group)
    w, v, _ = rep.param_views()
    with (rep.stream() if hasattr(rep, "stream") else _NoStream()):
        if _initialised():           # also with one rank: the collective then runs as a self-check of the plumbing
            dist.all_reduce(w, op=dist.ReduceOp.SUM, group=group)
            dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)
        rep.scale_and_refresh(1.0 / world)


def exchange_then_average(rep, group=None, buffers=None):
    """The figure's steps as drawn: (2) every replica's weights, biases and momentum are copied to all others, into receive
    buffers on the receiving GPU; (3) every GPU averages what it holds.  buffers = (list of w buffers, list of v buffers),
    one per rank, kept by the caller between steps (allocated here when None).  Returns the buffers."""
    world = _world(group)
    rank = dist.get_rank(group) if _initialised() else 0
    w, v, _ = rep.param_views()
    if buffers is None:
        buffers = ([torch.empty_like(w) for _ in range(world)], [torch.empty_like(v) for _ in range(world)])
    with (rep.stream() if hasattr(rep, "stream") else _NoStream()):
        if _initialised():
            dist.all_gather(buffers[0], w, group=group)
            dist.all_gather(buffers[1], v, group=group)
        rep.average_received(buffers[0], buffers[1], rank)
    return buffers


def allreduce_gradients_and_update(rep, group=None):
    """The gradient form: sum the pending gradients of all ranks, then every rank applies one update with the mean
    gradient.  Half the bytes of exchange_and_average on the wire; the replicas stay identical by construction."""
    world = _world(group)
    _, _, g = rep.param_views()
    with (rep.stream() if hasattr(rep, "stream") else _NoStream()):
        if _initialised():
            dist.all_reduce(g, op=dist.ReduceOp.SUM, group=group)
        rep.apply_update(1.0 / world)


def allreduce_gradients_overlapped_and_update(rep, comm_stream, group=None):
    """Call right after forward_backward has been issued.  The all-reduce of the FC weight gradients is queued on
    comm_stream behind a device-side wait for those gradients and runs beside the rest of the backward pass; the
    convolution and bias gradients are all-reduced from the compute stream after the pass; then one update with the mean
    gradient.  Every rank issues the same collectives in the same order."""
    world = _world(group)
    _, _, g = rep.param_views()
    b, e = rep.fc_range()
    rep.stream_wait_fc_gradients(comm_stream)
    with (torch.cuda.stream(comm_stream) if comm_stream is not None else _NoStream()):
        if _initialised():
            dist.all_reduce(g[b:e], op=dist.ReduceOp.SUM, group=group)
    with (rep.stream() if hasattr(rep, "stream") else _NoStream()):
        if _initialised():
            dist.all_reduce(g[:b], op=dist.ReduceOp.SUM, group=group)
            dist.all_reduce(g[e:], op=dist.ReduceOp.SUM, group=group)
        rep.wait_stream(comm_stream)
        rep.apply_update(1.0 / world)


def barrier(world: int) -> None:
    if world > 1:
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Maximum of a per-rank scalar (the timed milliseconds) over all ranks."""
    if world <= 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
