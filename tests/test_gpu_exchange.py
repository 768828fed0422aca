"""The exchange between replicas in separate processes, on one GPU: a one-rank NCCL group runs the collectives of
paper_1412_2302_b200.exchange on the views of the library's own parameter arrays, behind the compute stream.  With one
rank the all-reduce returns its input, so the results must equal the plain single-replica paths bit for bit; what is
exercised is the plumbing the N-GPU bench relies on (views into the arena, stream order between NCCL and the
library's kernels, the scale-and-refresh and deferred-update entry points)."""
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

from paper_1412_2302_b200 import exchange, synth

pytestmark = pytest.mark.gpu


@pytest.fixture()
def nccl_group():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    yield
    dist.destroy_process_group()


def test_one_rank_nccl_exchange_equals_local_paths(nccl_group):
    from paper_1412_2302_b200.alexnet import AlexNet
    seed, B = synth.BASE_SEED + 13, 4
    w = synth.init_params(seed, variance_preserving=True)

    def run(mode):
        net = AlexNet(batch=B, seed=seed, mean_image=synth.mean_image(seed))
        net.set_params(w)
        rep = exchange.LocalReplica(net, 0)
        losses, state = [], {}
        for step in range(3):
            img = torch.from_numpy(synth.images(seed, 0, step, B)).pin_memory()
            lab = torch.from_numpy(synth.labels(seed, 0, step, B)).pin_memory()
            net.load_batch_async(0, img, lab, step)
            if mode == "plain":
                losses.append(net.train_step(0, want_loss=True))
            elif mode == "params":
                losses.append(net.train_step(0, want_loss=True))
                exchange.exchange_and_average(rep)
            elif mode == "overlap":
                losses.append(None)
                net.forward_backward(0)
                exchange.allreduce_gradients_overlapped_and_update(rep, state.setdefault("comm", torch.cuda.Stream()))
                buf = state.setdefault("loss", torch.zeros(1).pin_memory())
                net.loss_async(0, buf); net.sync()
                losses[-1] = float(buf[0])
            elif mode == "gather":
                losses.append(net.train_step(0, want_loss=True))
                state["buffers"] = exchange.exchange_then_average(rep, buffers=state.get("buffers"))
            else:
                losses.append(net.forward_backward(0, want_loss=True))
                exchange.allreduce_gradients_and_update(rep)
        net.sync()
        out = (losses, net.get_params(0, 0), net.get_params(0, 1))
        net.close()
        return out

    plain, params, grads, gather, overlap = run("plain"), run("params"), run("grads"), run("gather"), run("overlap")
    for other in (params, grads, gather, overlap):
        assert other[0] == plain[0]
        assert np.array_equal(other[1], plain[1]) and np.array_equal(other[2], plain[2])
    assert not np.array_equal(plain[1], w)
