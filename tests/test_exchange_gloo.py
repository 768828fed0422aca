"""The exchange between replicas in separate processes, on CPU: two gloo ranks run the same Python entry points the
GPU ranks run (paper_1412_2302_b200.exchange) on host tensors, and the result is compared with the oracle's
exchange-and-average of two replicas that each took an update on their own gradient.  Also the timing plumbing of the
bench (maximum over ranks)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import oracle as O
from paper_1412_2302_b200 import exchange

N = 4099          # parameters of the stand-in replica (odd, so that nothing relies on a vector width)
LR, MU, WD = 0.01, 0.9, 5e-4


class HostReplica:
    """What exchange.* needs of a replica, held in host memory: (w, v, g) views, the scale-and-refresh step and the
    update rule (fp32, the arithmetic of the device's update kernel).  refreshed counts the rebuilds of the bf16 copy."""

    def __init__(self, w, v, g):
        self.w, self.v, self.g = (torch.from_numpy(np.array(t, np.float32)) for t in (w, v, g))
        self.refreshed = 0
        self.pending = True

    def param_views(self):
        return self.w, self.v, self.g

    def scale_and_refresh(self, scale):
        self.w.mul_(scale); self.v.mul_(scale)
        self.refreshed += 1

    def average_received(self, recv_w, recv_v, self_rank):
        n = len(recv_w)
        sw, sv = torch.zeros_like(self.w), torch.zeros_like(self.v)
        for r in range(n):                              # rank order, the own arrays at the own rank
            sw += self.w if r == self_rank else recv_w[r]
            sv += self.v if r == self_rank else recv_v[r]
        self.w.copy_(sw * (1.0 / n)); self.v.copy_(sv * (1.0 / n))
        self.refreshed += 1

    def fc_range(self):
        return 1000, 3500                               # any split of the vector into three ranges

    def stream_wait_fc_gradients(self, stream):
        pass

    def wait_stream(self, stream):
        pass

    def apply_update(self, grad_scale):
        assert self.pending
        self.v.mul_(MU).add_(self.w, alpha=-LR * WD).add_(self.g * grad_scale, alpha=-LR)
        self.w.add_(self.v)
        self.pending = False


def inputs(rank):
    rng = np.random.default_rng(100)
    w = rng.standard_normal(N) * 0.05               # both ranks start identical (after the previous exchange)
    v = rng.standard_normal(N) * 0.01
    g = np.random.default_rng(200 + rank).standard_normal(N) * 0.1      # each rank's own minibatch gradient
    return w, v, g


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, v, g = inputs(rank)
        # parameter form: update on the own gradient, then exchange and average weights and momentum
        a = HostReplica(w, v, g)
        a.apply_update(1.0)
        exchange.exchange_and_average(a)
        # gradient form: all-reduce the gradients, one update with their mean
        b = HostReplica(w, v, g)
        exchange.allreduce_gradients_and_update(b)
        # the gradient form with the large range exchanged apart (on a GPU: from a second stream, under the backward pass)
        d = HostReplica(w, v, g)
        exchange.allreduce_gradients_overlapped_and_update(d, None)
        assert torch.equal(d.w, b.w) and torch.equal(d.v, b.v)
        # the figure's own two steps: receive the other replica's arrays, then average
        c = HostReplica(w, v, g)
        c.apply_update(1.0)
        exchange.exchange_then_average(c)
        assert torch.equal(c.w, a.w) and torch.equal(c.v, a.v)          # two replicas: the same sum, the same halving
        exchange.barrier(world)
        ms = exchange.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
        out.put((rank, a.w.numpy().copy(), a.v.numpy().copy(), b.w.numpy().copy(), b.v.numpy().copy(), a.refreshed, ms))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_exchange_matches_the_oracle():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((out.get(timeout=120) for _ in range(2)), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, aw0, av0, bw0, bv0, n0, ms0), (_, aw1, av1, bw1, bv1, n1, ms1) = res
    # every rank holds the same replica afterwards, bit for bit
    assert np.array_equal(aw0, aw1) and np.array_equal(av0, av1) and np.array_equal(bw0, bw1) and np.array_equal(bv0, bv1)
    assert n0 == n1 == 1
    # the oracle: two replicas, one update each on its own gradient, then exchange-and-average
    mask = np.ones(N)
    reps = []
    for r in range(2):
        w, v, g = inputs(r)
        reps.append(O.sgd_momentum(w.astype(np.float32).astype(np.float64), v.astype(np.float32).astype(np.float64),
                                   g.astype(np.float32).astype(np.float64), LR, MU, WD, mask))
    wm = O.replica_average(reps[0][0], reps[1][0])[0]
    vm = O.replica_average(reps[0][1], reps[1][1])[0]

    def rel(x, y):
        return np.linalg.norm(x - y) / np.linalg.norm(y)
    assert rel(aw0, wm) < 1e-5 and rel(av0, vm) < 1e-5            # parameter form
    assert rel(bw0, wm) < 1e-5 and rel(bv0, vm) < 1e-5            # gradient form: the same replica (the paper's equivalence)
    assert ms0 == ms1 == 15.0                                      # both ranks agree on the maximum


def test_single_process_exchange_is_the_identity_average():
    w, v, g = inputs(0)
    a = HostReplica(w, v, g)
    before = a.w.clone()
    exchange.exchange_and_average(a)                 # no process group: one replica, scale 1
    assert torch.equal(a.w, before) and a.refreshed == 1
    assert exchange.max_over_ranks(3.5, 1) == 3.5
