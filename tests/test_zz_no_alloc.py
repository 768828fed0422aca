"""The allocation-free bias-gradient entry point (alexnet_bias_grad_noalloc).

Some users of the library cannot call cudaMalloc when they need a bias
gradient: a loop in the middle of overlapped steps (an allocation synchronises
the device and would serialise the loader stream with the compute stream), or a
process that has handed all free HBM to the arena.  For them the entry point
keeps its scratch in a fixed 1 MiB array inside the library image.

Checked here: its output against the existing path's (the bias gradient the
step's own backward-weight operation produces) on two calls in a row, and
against a column sum computed on the host in fp64, over sizes that use one
split, several splits with a ragged last one, and the cap of 64 splits at the
largest channel count the scratch holds; calls of different shapes follow one
another, so that contents a previous call left in the scratch would show."""
import numpy as np
import pytest
import torch

from paper_1412_2302_b200 import synth

pytestmark = pytest.mark.gpu


def host_colsum(rows_bf16):
    return rows_bf16.to(torch.float32).cpu().numpy().astype(np.float64).sum(axis=0)


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
        assert np.linalg.norm(got - host_colsum(rows)) <= 1e-5 * np.linalg.norm(want), call
    # sizes beyond the fixed scratch are refused with a message, nothing is launched
    big = torch.zeros(4, 8192, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(A.AlexNetError) as e:
        A.bias_grad_noalloc(big, torch.zeros(8192, device="cuda"))
    assert e.value.code == A.ERR_ARG and "4096" in str(e.value)
    net.close()


# (rows, channels): splits = clamp(rows / 256, 1, 64), the scratch is laid out [split][channels]
CASES = [(20000, 4096),     # 64 splits (capped from 78) at the largest channel count: the whole 1 MiB scratch
         (300, 4096),       # 1 split right after: only row 0 of the scratch may be read
         (5000, 4096),      # 19 splits, last one ragged
         (1000, 8),         # 3 splits of 334 rows, the last with 332; the smallest channel count
         (21632, 256),      # 64 splits (capped from 84): conv5's gradient at batch 128
         (777, 72),         # 3 splits; channels not a multiple of 64 (the second column block is partial), rows % 32 != 0
         (1, 4096)]         # a single row


def test_bias_grad_noalloc_against_host_column_sums():
    from paper_1412_2302_b200 import alexnet as A
    rng = np.random.default_rng(23)
    st = torch.cuda.Stream()
    for rows, C in CASES:
        x = torch.from_numpy((rng.integers(-64, 65, size=(rows, C)) / 64.0).astype(np.float32)).to(torch.bfloat16).cuda()
        want = host_colsum(x)
        db = torch.full((C,), float("nan"), device="cuda")
        torch.cuda.synchronize()
        A.bias_grad_noalloc(x, db, stream=st)
        st.synchronize()
        got = db.cpu().numpy().astype(np.float64)
        assert np.isfinite(got).all(), (rows, C)
        # bf16 multiples of 1/64, fp32 accumulation: sums of up to 20000 such values are exact in fp32
        assert np.abs(got - want).max() <= 1e-5 * max(1.0, np.abs(want).max()), (rows, C, np.abs(got - want).max())
    for bad_rows, bad_c, word in ((0, 64, "rows"), (16, 12, "multiple of 8"), (16, 4104, "4096")):
        x = torch.zeros(max(bad_rows, 1), bad_c, dtype=torch.bfloat16, device="cuda")
        msg = __import__("ctypes").create_string_buffer(256)
        rc = A.load_library().alexnet_bias_grad_noalloc(A._ptr(x), bad_rows, bad_c, A._ptr(torch.zeros(bad_c, device="cuda")), None, msg, 256)
        assert rc == A.ERR_ARG and word in msg.value.decode(), (bad_rows, bad_c, msg.value)
