"""The multi-rank plumbing of the bench on CPU: two gloo ranks take different data streams, the job time is the
maximum over ranks, and the job throughput counts the images of all ranks."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1412_2302_b200 import multi, synth


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
        img = synth.images(synth.BASE_SEED, multi.rank_stream(rank), 0, 2)
        multi.barrier(world)
        ms = multi.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
        out.put((rank, int(img[:, :8, :8].astype(np.int64).sum()), ms, multi.job_throughput(128, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_distinct_streams():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, ms0, t0), (r1, s1, ms1, t1) = res
    assert (r0, r1) == (0, 1)
    assert s0 != s1                                   # different minibatches per rank
    assert ms0 == ms1 == 15.0                         # both ranks agree on the maximum
    assert t0 == t1 == 2 * 128 / 15e-3                # whole-job images per second


def test_single_rank_needs_no_process_group():
    assert multi.max_over_ranks(3.5, 1) == 3.5
    assert multi.job_throughput(128, 1, 2.0) == 64000.0
