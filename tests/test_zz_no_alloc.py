"""The allocation-free bias-gradient entry point against the bias gradient the
step's own backward-weight operation produces, on two calls in a row (the
second with other sizes, so that stale scratch contents would show)."""
import numpy as np
import pytest
import torch

from paper_1412_2302_b200 import synth

pytestmark = pytest.mark.gpu


def test_bias_grad_noalloc_matches_step_operation_twice():
    from paper_1412_2302_b200 import alexnet as A
    B, seed = 3, synth.BASE_SEED + 7
    net = A.AlexNet(batch=B, seed=seed)
    off = {"conv5.b": (2333824, 256), "conv4.b": (1891072, 384)}
    for call, (op, tdy, tin, key, C) in enumerate([("CONV5_BWD_WEIGHT", "DA5", "A4", "conv5.b", 256),
                                                   ("CONV4_BWD_WEIGHT", "DA4", "A3", "conv4.b", 384)]):
        dy = synth.bf16_grid(seed, 100 + call, (B, C, 13, 13), -1, 1)
        net.set_tensor(tdy, dy)
        net.set_tensor(tin, synth.bf16_grid(seed, 200 + call, (B, 384, 13, 13), -1, 1))
        net.run_op(op)
        net.sync()
        o, n = off[key]
        want = net.get_params(0, 2)[o:o + n]                     # the existing path
        rows = torch.from_numpy(dy.transpose(0, 2, 3, 1).reshape(-1, C).copy()).to(torch.bfloat16).cuda()
        db = torch.full((C,), float("nan"), device="cuda")
        A.bias_grad_noalloc(rows, db)
        torch.cuda.synchronize()
        got = db.cpu().numpy()
        assert np.isfinite(got).all()
        assert np.linalg.norm(got - want) <= 1e-5 * np.linalg.norm(want), call
    # sizes beyond the fixed scratch are refused with a message, nothing is launched
    big = torch.zeros(4, 8192, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(A.AlexNetError) as e:
        A.bias_grad_noalloc(big, torch.zeros(8192, device="cuda"))
    assert e.value.code == A.ERR_ARG and "4096" in str(e.value)
    net.close()
