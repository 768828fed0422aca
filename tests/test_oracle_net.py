"""Pins of the oracle's whole-network composition: an independent autograd
model built from PyTorch CPU fp64 library ops, a directional finite
difference, the ln(1000) first-loss closed form and the two-replica algebra."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import oracle as O
from paper_1412_2302_b200 import synth

SEED = synth.BASE_SEED + 2


def torch_loss(wflat, X, labels, m6, m7):
    P = {k: torch.from_numpy(v.copy()).requires_grad_() for k, v in O.unpack(wflat).items()}
    x = torch.from_numpy(X)
    lrn = lambda t: F.local_response_norm(t, 5, alpha=5e-4, beta=0.75, k=2.0)   # torch divides alpha by n
    x = F.max_pool2d(lrn(F.relu(F.conv2d(x, P["conv1.W"], P["conv1.b"], stride=4))), 3, 2)
    x = F.max_pool2d(lrn(F.relu(F.conv2d(x, P["conv2.W"], P["conv2.b"], padding=2, groups=2))), 3, 2)
    x = F.relu(F.conv2d(x, P["conv3.W"], P["conv3.b"], padding=1))
    x = F.relu(F.conv2d(x, P["conv4.W"], P["conv4.b"], padding=1, groups=2))
    x = F.max_pool2d(F.relu(F.conv2d(x, P["conv5.W"], P["conv5.b"], padding=1, groups=2)), 3, 2)
    x = x.reshape(x.shape[0], -1)
    x = F.relu(F.linear(x, P["fc6.W"], P["fc6.b"])) * torch.from_numpy(m6.astype(np.float64))
    x = F.relu(F.linear(x, P["fc7.W"], P["fc7.b"])) * torch.from_numpy(m7.astype(np.float64))
    z = F.linear(x, P["fc8.W"], P["fc8.b"])
    return F.cross_entropy(z, torch.from_numpy(labels.astype(np.int64))), P


def test_whole_net_gradients_match_independent_autograd_model_and_fd():
    B = 2
    w = synth.init_params(SEED, variance_preserving=True, bias=0.1).astype(np.float64)
    img, lab, mean = synth.images(SEED, 0, 3, B), synth.labels(SEED, 0, 3, B), synth.mean_image(SEED)
    net = O.OracleNet(O.OracleConfig(seed=SEED), w)
    T = net.forward_backward(img, lab, mean, step=3)
    loss_t, P = torch_loss(w, T["x0"], lab, T["m6"], T["m7"])
    loss_t.backward()
    assert abs(T["loss"] - loss_t.item()) < 1e-10
    off, _ = O.param_offsets()
    for k, (o, n, shp) in off.items():
        ref = P[k].grad.numpy().ravel()
        got = T["g"][o:o + n]
        assert np.linalg.norm(got - ref) <= 1e-9 * max(np.linalg.norm(ref), 1e-30), k
        assert np.linalg.norm(ref) > 0, k
    # directional central difference of the loss along a random direction over all parameters
    d = np.random.default_rng(0).standard_normal(w.size) * np.abs(w).mean()
    h = 1e-7
    Lp = O.OracleNet(O.OracleConfig(seed=SEED), w + h * d).forward_backward(img, lab, mean, 3)["loss"]
    Lm = O.OracleNet(O.OracleConfig(seed=SEED), w - h * d).forward_backward(img, lab, mean, 3)["loss"]
    fd, an = (Lp - Lm) / (2 * h), float(T["g"] @ d)
    assert abs(fd - an) < 1e-5 * abs(an) + 1e-9


def test_first_loss_is_ln1000_and_two_replica_step_equals_double_batch():
    cfg = O.OracleConfig(seed=SEED)
    w = synth.init_params(SEED).astype(np.float64)          # N(0, 0.01^2), zero biases
    mean = synth.mean_image(SEED)
    ia, la = synth.images(SEED, 0, 0, 1), synth.labels(SEED, 0, 0, 1)
    ib, lb = synth.images(SEED, 1, 0, 1), synth.labels(SEED, 1, 0, 1)
    a = O.OracleNet(cfg, w, replica=0)
    b = O.OracleNet(cfg, w, replica=1)
    Ta = a.train_step(ia, la, mean, 0)
    Tb = b.train_step(ib, lb, mean, 0)
    assert abs(Ta["loss"] - math.log(1000)) < 2e-2 and abs(Tb["loss"] - math.log(1000)) < 2e-2
    assert (Ta["cf"] != Tb["cf"]).any() and (Ta["m6"] != Tb["m6"]).any()   # replicas draw different streams
    assert not np.array_equal(a.w, b.w)
    O.average_replicas(a, b)
    assert np.array_equal(a.w, b.w) and np.array_equal(a.v, b.v)
    # equals one momentum step from (w, 0) with the mean of the two gradients
    g = 0.5 * (Ta["g"] + Tb["g"])
    wm, vm = O.sgd_momentum(w, np.zeros_like(w), g, cfg.lr, cfg.momentum, cfg.weight_decay, O.decay_mask())
    assert np.allclose(a.v, vm, rtol=0, atol=1e-15) and np.allclose(a.w, wm, rtol=0, atol=1e-15)
    # averaging identical replicas changes nothing, bitwise
    w0, v0 = a.w.copy(), a.v.copy()
    O.average_replicas(a, b)
    assert np.array_equal(a.w, w0) and np.array_equal(a.v, v0)


def test_conv1_block_against_autograd():
    s = synth.BASE_SEED + 1
    img, mean = synth.images(s, 0, 0, 2), synth.mean_image(s)
    cf = O.crop_flip(s, 0, 0, 2)
    w1 = synth.init_params(s)[:34848].reshape(96, 3, 11, 11).astype(np.float64)
    b1 = np.zeros(96)
    up = synth.normal(s, 0, (2, 96, 27, 27)).astype(np.float64)
    T = O.conv1_block(img, mean, cf, w1, b1, up)
    wt = torch.from_numpy(w1).requires_grad_(); bt = torch.from_numpy(b1).requires_grad_()
    y = F.max_pool2d(F.local_response_norm(F.relu(F.conv2d(torch.from_numpy(T["x0"]), wt, bt, stride=4)),
                                           5, alpha=5e-4, beta=0.75, k=2.0), 3, 2)
    (y * torch.from_numpy(up)).sum().backward()
    assert np.allclose(T["p1"], y.detach().numpy(), rtol=1e-12, atol=1e-12)
    assert np.linalg.norm(T["dW1"] - wt.grad.numpy()) < 1e-10 * np.linalg.norm(T["dW1"])
    assert np.linalg.norm(T["db1"] - bt.grad.numpy()) < 1e-10 * np.linalg.norm(T["db1"])


def test_topk_correct_against_sorting_and_ties():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((64, 1000))
    lab = rng.integers(0, 1000, 64)
    order = np.argsort(-z, axis=1, kind="stable")
    for k in (1, 5):
        want = np.array([int(lab[i] in order[i, :k]) for i in range(64)])
        assert np.array_equal(O.topk_correct(z, lab, k), want)
    # all-equal logits: exactly the classes 0..k-1 are "in the top k"
    z0 = np.zeros((6, 10))
    assert O.topk_correct(z0, np.array([0, 1, 4, 5, 9, 2]), 5).tolist() == [1, 1, 1, 0, 0, 1]
    assert O.topk_correct(z0, np.array([0, 1, 4, 5, 9, 2]), 1).tolist() == [1, 0, 0, 0, 0, 0]


def test_evaluation_pass_centre_crop_scaling_and_training_limit():
    """Evaluation = the training forward pass with the centre crop, no flip and the dropout masks replaced by their
    expectation: with p = 0 (no dropout) and the same crop the two passes must agree exactly."""
    seed, B = synth.BASE_SEED + 21, 2
    w = synth.init_params(seed, variance_preserving=True).astype(np.float64)
    img, lab, mean = synth.images(seed, 0, 0, B), synth.labels(seed, 0, 0, B), synth.mean_image(seed)
    net0 = O.OracleNet(O.OracleConfig(seed=seed, dropout_p=0.0), w)
    E0 = O.evaluate(net0, img, lab, mean)
    cf = np.tile(np.array([14, 14, 0], np.int32), (B, 1))
    T = net0.forward_backward(img, lab, mean, 0, cf=cf)
    assert np.allclose(E0["z"], T["z"], rtol=0, atol=1e-12) and abs(E0["loss"] - T["loss"]) < 1e-12
    # the crop is the centre window of the mean-subtracted image
    assert np.array_equal(E0["x0"][0, 1], img[0, 14:241, 14:241, 1].astype(np.float64) - mean[14:241, 14:241, 1])
    # p = 0.5 without rescaling at training time: evaluation halves the fc6 / fc7 outputs; inverted dropout does not
    Eh = O.evaluate(O.OracleNet(O.OracleConfig(seed=seed, dropout_p=0.5), w), img, lab, mean)
    Ei = O.evaluate(O.OracleNet(O.OracleConfig(seed=seed, dropout_p=0.5, inverted_dropout=True), w), img, lab, mean)
    assert np.allclose(Eh["f6"], 0.5 * E0["f6"]) and np.allclose(Ei["f6"], E0["f6"]) and np.allclose(Ei["z"], E0["z"])
    assert not np.allclose(Eh["z"], E0["z"])
    # mean over dropout masks of the training-time fc6 output (given identical inputs) approaches the halved output
    assert Eh["top1"].shape == (B,) and set(np.unique(Eh["top5"])) <= {0, 1}
