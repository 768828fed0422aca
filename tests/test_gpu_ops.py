"""Kernel-level parity: every operation of the step, run in isolation through
the C ABI on inputs that are exactly representable in bf16, against the fp64
oracle.  Integer artefacts (crop/flip, argmax, dropout masks) must match bit
for bit; floating point within rel-L2 2e-2 (bf16 operands, fp32 accumulate),
1e-5 for the fp32 update / average pass."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_1412_2302_b200 import synth

pytestmark = pytest.mark.gpu

SEED = synth.BASE_SEED + 5
TOL = 2e-2


def tag(name):
    return sum(map(ord, name))


def rel(a, b):
    a, b = np.asarray(a, np.float64).ravel(), np.asarray(b, np.float64).ravel()
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)


# every operation runs at batch 3 (ragged: no grid is a multiple of the 128-row tile, one or two tiles per kernel, split
# counts at their maximum) three times: tile shapes from the cost model, convolutions on single CTAs only, and
# convolutions on CTA pairs (cta_group::2) only; and once more at batch 40, where the persistent kernels walk several
# rounds of their tile lists with a partial last round (conv1: 1016 row tiles, conv2: 263 per group, conv3-5: 62 with a
# ragged last one) and the split counts follow from the batch
@pytest.fixture(scope="module", params=[(0, 3), (16, 3), (32, 3), (0, 40)], ids=["auto", "single-cta", "cta-pairs", "auto-batch40"])
def net(request):
    from paper_1412_2302_b200.alexnet import AlexNet
    flags, batch = request.param
    n = AlexNet(batch=batch, replicas=2, seed=SEED, mean_image=synth.mean_image(SEED), flags=flags)
    yield n
    n.close()


@pytest.fixture(scope="module")
def params(net):
    """bf16-representable parameters (multiples of 1/256 in [-0.25, 0.25]), biases too."""
    rng = np.random.default_rng(11)
    w = (rng.integers(-64, 65, size=net.param_count) / 256.0).astype(np.float32)
    net.set_params(w, 0, 0)
    return O.unpack(w.astype(np.float64))


CONVS = [("conv1", "X0", "A1", (3, 227, 227)), ("conv2", "P1", "A2", (96, 27, 27)), ("conv3", "P2", "A3", (256, 13, 13)),
         ("conv4", "A3", "A4", (384, 13, 13)), ("conv5", "A4", "A5", (384, 13, 13))]


@pytest.mark.parametrize("name,tin,tout,shp", CONVS)
def test_conv_forward(net, params, name, tin, tout, shp):
    B = net.batch
    x = synth.bf16_grid(SEED, tag(name), (B,) + shp, -1, 1)
    if name == "conv1":
        x = x * 4
    net.set_tensor(tin, x)
    net.run_op(name.upper() + "_FWD")
    net.sync()
    c = O.CONV[name]
    ref = np.maximum(O.conv_fwd(x, params[name + ".W"], params[name + ".b"], c["s"], c["p"], c["g"]), 0)
    got = net.get_tensor(tout).reshape(ref.shape)
    assert rel(got, ref) < TOL, rel(got, ref)
    assert (got >= 0).all()


# conv1's data gradient (the gradient with respect to the image) is not part of the training step; the per-layer sweep
# runs it, in the space-to-depth layout of conv1's input
BWD = [("conv1", "DA1", "DX0", None, (3, 227, 227)), ("conv2", "DA2", "DP1", None, (96, 27, 27)), ("conv3", "DA3", "DP2", None, (256, 13, 13)),
       ("conv4", "DA4", "DA3", "A3", (384, 13, 13)), ("conv5", "DA5", "DA4", "A4", (384, 13, 13))]


@pytest.mark.parametrize("name,tdy,tdx,tmask,shp", BWD)
def test_conv_backward_data(net, params, name, tdy, tdx, tmask, shp):
    B = net.batch
    c = O.CONV[name]
    ho = 55 if name == "conv1" else shp[1]
    dy = synth.bf16_grid(SEED, 7 + tag(name), (B, c["cout"], ho, ho), -1, 1)
    net.set_tensor(tdy, dy)
    ref = O.conv_bwd_data(dy, params[name + ".W"], (B,) + shp, c["s"], c["p"], c["g"])
    if tmask:
        m = synth.bf16_grid(SEED, 9 + tag(name), (B,) + shp, -1, 1)
        m = np.maximum(m, 0)
        net.set_tensor(tmask, m)
        ref = ref * (m > 0)
    net.run_op(name.upper() + "_BWD_DATA")
    net.sync()
    got = net.get_tensor(tdx).reshape(ref.shape)
    assert rel(got, ref) < TOL, rel(got, ref)


WG = [("conv1", "X0", "DA1", (3, 227, 227), 55), ("conv2", "P1", "DA2", (96, 27, 27), 27), ("conv3", "P2", "DA3", (256, 13, 13), 13),
      ("conv4", "A3", "DA4", (384, 13, 13), 13), ("conv5", "A4", "DA5", (384, 13, 13), 13)]


@pytest.mark.parametrize("name,tin,tdy,shp,ho", WG)
def test_conv_backward_weight_and_bias(net, params, name, tin, tdy, shp, ho):
    B = net.batch
    c = O.CONV[name]
    x = synth.bf16_grid(SEED, 21 + tag(name), (B,) + shp, -1, 1)
    dy = synth.bf16_grid(SEED, 22 + tag(name), (B, c["cout"], ho, ho), -1, 1)
    net.set_tensor(tin, x)
    net.set_tensor(tdy, dy)
    net.run_op(name.upper() + "_BWD_WEIGHT")
    net.sync()
    dw, db = O.conv_bwd_weight(x, dy, params[name + ".W"].shape, c["s"], c["p"], c["g"])
    g = net.get_params(0, 2)
    off, _ = O.param_offsets()
    o, n, _ = off[name + ".W"]
    assert rel(g[o:o + n], dw) < 1e-3, rel(g[o:o + n], dw)     # fp32 output, exact products: only summation order
    o, n, _ = off[name + ".b"]
    assert rel(g[o:o + n], db) < 1e-3


FCS = [("fc6", "P5", "F6", "M6", 2), ("fc7", "F6", "F7", "M7", 3), ("fc8", "F7", "Z", None, None)]


@pytest.mark.parametrize("name,tin,tout,tm,stream", FCS)
def test_fc_forward_with_dropout(net, params, name, tin, tout, tm, stream):
    B = net.batch
    K, N = O.FC[name]
    x = synth.bf16_grid(SEED, 31 + tag(name), (B, K), -1, 1)
    xin = x.reshape(B, 256, 6, 6) if name == "fc6" else x
    net.set_tensor(tin, xin)
    net.run_op(name.upper() + "_FWD")
    net.sync()
    ref = O.fc_fwd(x, params[name + ".W"], params[name + ".b"])
    if tm:
        keep = O.dropout_mask(SEED, stream, 0, 0, B, N, 0.5)
        assert np.array_equal(net.get_tensor(tm).reshape(B, N).astype(np.uint8), keep)   # bit exact
        ref = np.maximum(ref, 0) * keep
    got = net.get_tensor(tout).reshape(B, N)
    assert rel(got, ref) < (TOL if tm else 1e-4), rel(got, ref)


FCB = [("fc6", "DF6", "DP5", None), ("fc7", "DF7", "DF6", "F6"), ("fc8", "DZ", "DF7", "F7")]


@pytest.mark.parametrize("name,tdy,tdx,tmask", FCB)
def test_fc_backward_data(net, params, name, tdy, tdx, tmask):
    B = net.batch
    K, N = O.FC[name]
    dy = synth.bf16_grid(SEED, 41 + tag(name), (B, N), -1, 1)
    net.set_tensor(tdy, dy)
    ref = dy.astype(np.float64) @ params[name + ".W"]
    if tmask:
        m = np.maximum(synth.bf16_grid(SEED, 42 + tag(name), (B, K), -1, 1), 0)
        net.set_tensor(tmask, m)
        ref = ref * (m > 0)
    net.run_op(name.upper() + "_BWD_DATA")
    net.sync()
    got = net.get_tensor(tdx).reshape(B, -1)
    if name == "fc6":
        ref = ref.reshape(B, 256, 6, 6).reshape(B, -1)
    assert rel(got, ref) < TOL, rel(got, ref)


FCW = [("fc6", "P5", "DF6"), ("fc7", "F6", "DF7"), ("fc8", "F7", "DZ")]


@pytest.mark.parametrize("name,tin,tdy", FCW)
def test_fc_backward_weight_and_bias(net, params, name, tin, tdy):
    B = net.batch
    K, N = O.FC[name]
    x = synth.bf16_grid(SEED, 51 + tag(name), (B, K), -1, 1)
    dy = synth.bf16_grid(SEED, 52 + tag(name), (B, N), -1, 1)
    net.set_tensor(tin, x.reshape(B, 256, 6, 6) if name == "fc6" else x)
    net.set_tensor(tdy, dy)
    net.run_op(name.upper() + "_BWD_WEIGHT")
    net.sync()
    _, dw, db = O.fc_bwd(x, params[name + ".W"], dy)
    g = net.get_params(0, 2)
    off, _ = O.param_offsets()
    o, n, _ = off[name + ".W"]
    assert rel(g[o:o + n], dw) < 1e-5
    o, n, _ = off[name + ".b"]
    assert rel(g[o:o + n], db) < 1e-5


@pytest.mark.parametrize("which,ta,tn,tdn,tda,shp", [(1, "A1", "N1", "DN1", "DA1", (96, 55, 55)), (2, "A2", "N2", "DN2", "DA2", (256, 27, 27))])
def test_lrn_forward_backward(net, which, ta, tn, tdn, tda, shp):
    B = net.batch
    a = np.maximum(synth.bf16_grid(SEED, 60 + which, (B,) + shp, -1, 1) * 64, 0)   # post-ReLU range up to 64
    g = synth.bf16_grid(SEED, 62 + which, (B,) + shp, -1, 1)
    net.set_tensor(ta, a)
    net.set_tensor(tdn, g)
    net.run_op(f"LRN{which}_FWD")
    net.run_op(f"LRN{which}_BWD")
    net.sync()
    assert rel(net.get_tensor(tn), O.lrn_fwd(a)) < 4e-3
    ref = O.lrn_bwd(a, g) * (a > 0)
    assert rel(net.get_tensor(tda), ref) < 4e-3


POOLS = [(1, "N1", "P1", "ARG1", "DP1", "DN1", None, (96, 55, 55)), (2, "N2", "P2", "ARG2", "DP2", "DN2", None, (256, 27, 27)),
         (5, "A5", "P5", "ARG5", "DP5", "DA5", "A5", (256, 13, 13))]


@pytest.mark.parametrize("which,tx,ty,targ,tdy,tdx,trelu,shp", POOLS)
def test_pool_forward_backward(net, which, tx, ty, targ, tdy, tdx, trelu, shp):
    B = net.batch
    x = np.maximum(synth.bf16_grid(SEED, 70 + which, (B,) + shp, -1, 1), 0)   # many exact ties at 0 and on the grid
    net.set_tensor(tx, x)
    net.run_op(f"POOL{which}_FWD")
    net.sync()
    y, arg = O.pool_fwd(x)
    assert np.array_equal(net.get_tensor(ty).reshape(y.shape), y.astype(np.float32))
    assert np.array_equal(net.get_tensor(targ).reshape(arg.shape).astype(np.uint8), arg)     # bit exact
    dy = synth.bf16_grid(SEED, 75 + which, y.shape, -1, 1)
    net.set_tensor(tdy, dy)
    net.run_op(f"POOL{which}_BWD")
    net.sync()
    ref = O.pool_bwd(dy, arg, x.shape)
    if trelu:
        ref = ref * (x > 0)
    assert rel(net.get_tensor(tdx), ref) < 4e-3


def tie_heavy(seed, tag, shape, block=3, scale=8.0):
    """Post-ReLU activations full of exact ties: piecewise constant over block x block pixels (so that the pixels of a
    pooling window often hold identical channel vectors, whose normalised values are then identical bit for bit), about
    half of the blocks zero."""
    Bn, C, H, W = shape
    hb, wb = (H + block - 1) // block, (W + block - 1) // block
    coarse = np.maximum(synth.bf16_grid(seed, tag, (Bn, C, hb, wb), -1, 1) * scale, 0)
    return np.repeat(np.repeat(coarse, block, axis=2), block, axis=3)[:, :, :H, :W].copy()


FUSED = [(1, "A1", "N1", "P1", "ARG1", "DP1", "DA1", (96, 55, 55)), (2, "A2", "N2", "P2", "ARG2", "DP2", "DA2", (256, 27, 27))]


@pytest.mark.parametrize("which,ta,tn,tp,targ,tdp,tda,shp", FUSED)
@pytest.mark.parametrize("block", [3, 2, 1])
def test_fused_lrn_pool_forward_argmax_bit_exact(net, which, ta, tn, tp, targ, tdp, tda, shp, block):
    """The kernel the training step runs for LRN + pooling (integer-key maximum).  The normalised tensor it pools is the
    one the single-operation LRN kernel writes (same device function), so pooling THAT tensor with the oracle gives the
    exact expectation: values and argmax codes bit for bit, on inputs where most windows hold exact ties (zeros and
    repeated non-zero values), so that any tie rule but first-maximum-in-scan-order fails."""
    B = net.batch
    a = tie_heavy(SEED, 90 + which + 10 * block, (B,) + shp, block)
    net.set_tensor(ta, a)
    net.run_op(f"LRN{which}_FWD")
    net.sync()
    n_gpu = net.get_tensor(tn).reshape((B,) + shp)
    assert rel(n_gpu, O.lrn_fwd(a)) < 4e-3
    y, arg = O.pool_fwd(n_gpu.astype(np.float64))
    # the input must really exercise the tie rule: in many windows the maximum occurs more than once
    cnt = sum((n_gpu[:, :, ky:ky + 2 * y.shape[2] - 1:2, kx:kx + 2 * y.shape[3] - 1:2] == y).astype(np.int32)
              for ky in range(3) for kx in range(3))
    assert (cnt >= 2).mean() > (0.3 if block > 1 else 0.01)
    net.set_tensor(tp, np.full(y.shape, -1.0, np.float32))
    net.set_tensor(targ, np.full(arg.shape, 9, np.float32))
    net.run_op(f"LRN{which}_POOL{which}_FWD")
    net.sync()
    assert np.array_equal(net.get_tensor(tp).reshape(y.shape), y.astype(np.float32))
    assert np.array_equal(net.get_tensor(targ).reshape(arg.shape).astype(np.uint8), arg)     # bit exact


@pytest.mark.parametrize("which,ta,tn,tp,targ,tdp,tda,shp", FUSED)
def test_fused_pool_lrn_backward(net, which, ta, tn, tp, targ, tdp, tda, shp):
    """The fused backward kernel of the step (pooling gradient scattered in shared memory, LRN gradient, ReLU mask)
    against the oracle's pool_bwd followed by lrn_bwd, with argmax codes that send several windows to one pixel."""
    B = net.batch
    a = tie_heavy(SEED, 95 + which, (B,) + shp, 2)
    y, arg = O.pool_fwd(O.lrn_fwd(a))
    rng = np.random.default_rng(17 + which)
    arg = np.where(rng.random(arg.shape) < 0.5, arg, rng.integers(0, 9, size=arg.shape)).astype(np.uint8)   # any valid code
    dp = synth.bf16_grid(SEED, 97 + which, y.shape, -1, 1)
    net.set_tensor(ta, a)
    net.set_tensor(targ, arg.astype(np.float32))
    net.set_tensor(tdp, dp)
    net.run_op(f"POOL{which}_LRN{which}_BWD")
    net.sync()
    dn = O.round_bf16(O.pool_bwd(dp, arg, a.shape))          # the kernel rounds the pooled gradient to bf16, as the unfused path stores it
    ref = O.lrn_bwd(a, dn) * (a > 0)
    got = net.get_tensor(tda).reshape(ref.shape)
    assert rel(got, ref) < 4e-3, rel(got, ref)
    assert (got[a <= 0] == 0).all()


def test_softmax_xent(net):
    B = net.batch
    z = synth.normal(SEED, 80, (B, 1000), 3.0)
    lab = synth.labels(SEED, 0, 0, B)
    img = synth.images(SEED, 0, 0, B)
    import torch
    net.load_batch_async(0, torch.from_numpy(img), torch.from_numpy(lab), 0)   # brings the labels to the device
    net.sync()
    net.set_tensor("Z", z)
    net.run_op("SOFTMAX")
    net.sync()
    p, L, dz = O.softmax_xent(z, lab)
    assert rel(net.get_tensor("DZ"), dz) < 4e-3
    ln = net.get_tensor("LOSS")
    assert abs(ln.mean() - L) < 1e-5 * abs(L)
    # the slot stays loaded; consume it so that later tests start clean
    net.train_step(0)
    net.sync()


def test_preprocess_crop_flip_bit_exact(net):
    B = net.batch
    import torch
    for step in (5, 6):
        img = synth.images(SEED, 1, step, B)
        lab = synth.labels(SEED, 1, step, B)
        net.load_batch_async(1, torch.from_numpy(img), torch.from_numpy(lab), step)
        net.train_step(1)
        net.sync()
        cf = O.crop_flip(SEED, 1, step, B)
        assert np.array_equal(net.get_tensor("CROPFLIP", 1).reshape(B, 3).astype(np.int32), cf)
        x0 = O.preprocess(img, synth.mean_image(SEED), cf)
        got = net.get_tensor("X0", 1).reshape(x0.shape)
        # identical source pixels: only the bf16 rounding of (u8 - mean) differs
        assert np.array_equal(got, O.round_bf16(x0.astype(np.float32)).astype(np.float32))


def test_update_and_average_fp32(net):
    B = net.batch
    rng = np.random.default_rng(3)
    n = net.param_count
    w0 = rng.standard_normal(n).astype(np.float32) * 0.05
    v0 = rng.standard_normal(n).astype(np.float32) * 0.01
    net.set_params(w0, 0, 0); net.set_params(v0, 0, 1)
    g = net.get_params(0, 2).astype(np.float64)         # whatever gradient the last step left
    net.run_op("UPDATE", 0)
    net.sync()
    w1, v1 = O.sgd_momentum(w0.astype(np.float64), v0.astype(np.float64), g, 0.01, 0.9, 5e-4, O.decay_mask())
    assert rel(net.get_params(0, 1), v1) < 1e-5 and rel(net.get_params(0, 0), w1) < 1e-5
    assert np.abs(net.get_params(0, 1) - v1).max() < 1e-5 * np.abs(v1).max() + 1e-9
    # average with a different replica
    wb = rng.standard_normal(n).astype(np.float32) * 0.05
    vb = rng.standard_normal(n).astype(np.float32) * 0.01
    net.set_params(wb, 1, 0); net.set_params(vb, 1, 1)
    wa, va = net.get_params(0, 0), net.get_params(0, 1)
    net.replica_average()
    net.sync()
    ga, gb = net.get_params(0, 0), net.get_params(1, 0)
    assert np.array_equal(ga, gb) and np.array_equal(net.get_params(0, 1), net.get_params(1, 1))   # bitwise equal
    assert rel(ga, O.replica_average(wa.astype(np.float64), wb.astype(np.float64))[0]) < 1e-5
    assert rel(net.get_params(0, 1), O.replica_average(va.astype(np.float64), vb.astype(np.float64))[0]) < 1e-5
    before = ga.copy()
    net.replica_average()                                 # identical replicas: bitwise identity
    net.sync()
    assert np.array_equal(net.get_params(0, 0), before) and np.array_equal(net.get_params(1, 0), before)


def test_preprocess_intensity_augmentation(net):
    """The augmentation the paper's experiments leave out, as an option of the preprocessing gather: per-image RGB offsets
    from the hash (fp32 Box-Muller on the device, fp64 in the oracle: the bf16 result may differ by one rounding step in a
    few places), never at evaluation, and switched off again the gather is bit-exact as before."""
    import torch
    B = net.batch
    th = 0.6
    eigvec = np.array([[np.cos(th), -np.sin(th), 0.0], [np.sin(th), np.cos(th), 0.0], [0.0, 0.0, 1.0]]) @ np.array(
        [[1.0, 0.0, 0.0], [0.0, np.cos(0.3), -np.sin(0.3)], [0.0, np.sin(0.3), np.cos(0.3)]])
    eigval = np.array([55.0, 5.0, 1.2])                     # spread of the three components, in pixel units
    step = 9
    img, lab = synth.images(SEED, 0, step, B), synth.labels(SEED, 0, step, B)
    net.set_color_augmentation(eigvec, eigval, 0.1)
    net.load_batch_async(0, torch.from_numpy(img), torch.from_numpy(lab), step)
    net.sync()
    cf = O.crop_flip(SEED, 0, step, B)
    assert np.array_equal(net.get_tensor("CROPFLIP").reshape(B, 3).astype(np.int32), cf)
    shift = O.color_shift(SEED, 0, step, B, eigvec.astype(np.float32), eigval.astype(np.float32), 0.1)
    assert np.abs(shift).max() > 1.0                        # a visible offset
    ref = O.preprocess(img, synth.mean_image(SEED), cf, shift)
    got = net.get_tensor("X0").reshape(ref.shape).astype(np.float64)
    plain = O.preprocess(img, synth.mean_image(SEED), cf)
    assert rel(got, ref) < 2.5e-3 and rel(got, plain) > 10 * rel(got, ref)
    want = O.round_bf16(ref.astype(np.float32))
    off = got != want
    # one bf16 rounding step, or, where pixel - mean + offset nearly cancels, the fp32 rounding of terms of size 256
    assert off.mean() < 0.01 and (np.abs(got - want)[off] <= np.abs(want[off]) * 2.0 ** -7 + 2e-4).all()
    net.train_step(0); net.sync()
    # evaluation never augments; and with sigma = 0 the training gather is bit-exact again
    net.eval_batch(0, torch.from_numpy(img), torch.from_numpy(lab))       # (the parameters are whatever earlier tests left: only X0 matters)
    x_eval = net.get_tensor("X0").reshape(ref.shape)
    centre = O.preprocess(img, synth.mean_image(SEED), np.tile(np.array([[14, 14, 0]], np.int32), (B, 1)))
    assert np.array_equal(x_eval, O.round_bf16(centre.astype(np.float32)).astype(np.float32))
    net.set_color_augmentation(sigma=0.0)
    net.load_batch_async(0, torch.from_numpy(img), torch.from_numpy(lab), step)
    net.sync()
    assert np.array_equal(net.get_tensor("X0").reshape(ref.shape), O.round_bf16(plain.astype(np.float32)).astype(np.float32))
    net.train_step(0); net.sync()
