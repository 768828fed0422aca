"""Pins of the fp64 CPU oracle against things other than itself: published
hash vectors, closed forms, brute force on tiny shapes, central finite
differences, invariants and library special cases (PyTorch CPU fp64)."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import oracle as O
from paper_1412_2302_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(7)


def rel(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ------------------------------------------------------------------ hashing

def test_hash_matches_published_splitmix64_vectors():
    want = [int(l, 16) for l in open(os.path.join(GOLD, "splitmix64_seed0.txt")) if l.startswith("0x")]
    assert [O.draw(0, i) for i in range(3)] == want


def test_stream_key_composition():
    # key = finalise(seed ^ stream<<56 ^ replica<<48 ^ step); python big-int restatement of the finaliser
    def fin(z):
        M = 2**64 - 1
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M
        return z ^ (z >> 31)
    assert O.stream_key(14122302, 3, 1, 17) == fin(14122302 ^ (3 << 56) ^ (1 << 48) ^ 17)
    assert O.stream_key(5, 1, 0, 0) != O.stream_key(5, 2, 0, 0) != O.stream_key(5, 1, 1, 0)


def test_crop_flip_ranges_and_decode():
    cf = O.crop_flip(99, 1, 7, 4096)
    assert cf[:, 0].min() == 0 and cf[:, 0].max() == 29
    assert cf[:, 1].min() == 0 and cf[:, 1].max() == 29
    assert set(np.unique(cf[:, 2])) == {0, 1}
    assert abs(cf[:, 2].mean() - 0.5) < 0.03
    key = O.stream_key(99, 1, 1, 7)
    r = O.draw(key, 5)
    assert tuple(cf[5]) == ((r & 0xFFFF) % 30, ((r >> 16) & 0xFFFF) % 30, (r >> 32) & 1)
    # different step or replica -> different triples
    assert (O.crop_flip(99, 1, 8, 64) != cf[:64]).any()
    assert (O.crop_flip(99, 0, 7, 64) != cf[:64]).any()


def test_dropout_mask_statistics_and_reproducibility():
    m = O.dropout_mask(3, 2, 0, 11, 128, 4096, 0.5)
    assert abs(m.mean() - 0.5) < 0.003          # 524,288 draws
    assert (m == O.dropout_mask(3, 2, 0, 11, 128, 4096, 0.5)).all()
    assert (m != O.dropout_mask(3, 3, 0, 11, 128, 4096, 0.5)).any()
    assert O.dropout_mask(3, 2, 0, 11, 8, 4096, 0.0).all()
    assert abs(O.dropout_mask(3, 2, 0, 11, 64, 4096, 0.25).mean() - 0.75) < 0.01
    key = O.stream_key(3, 2, 0, 11)
    assert m[2, 5] == int((O.draw(key, 2 * 4096 + 5) >> 40) >= (1 << 23))
    # the first rows of a bigger batch are the same draws (idx = n*width + j)
    assert (O.dropout_mask(3, 2, 0, 11, 4, 4096, 0.5) == m[:4]).all()


# ------------------------------------------------------------ preprocessing

def test_preprocess_index_map():
    img = synth.images(1, 0, 0, 3)
    mean = synth.mean_image(1).astype(np.float64)
    # no crop offset, no flip, zero mean = top-left 227x227 block
    cf = np.zeros((3, 3), np.int32)
    X = O.preprocess(img, np.zeros_like(mean), cf)
    assert (X == img[:, :227, :227, :].transpose(0, 3, 1, 2)).all()
    # general: numpy slicing restatement, mean taken at the source pixel
    cf = np.array([[29, 0, 1], [3, 29, 0], [17, 5, 1]], np.int32)
    X = O.preprocess(img, mean, cf)
    for n, (ox, oy, fl) in enumerate(cf):
        blk = img[n, oy:oy + 227, ox:ox + 227, :].astype(np.float64) - mean[oy:oy + 227, ox:ox + 227, :]
        if fl:
            blk = blk[:, ::-1, :]
        assert (X[n] == blk.transpose(2, 0, 1)).all()
    # flip of flip is the identity
    cf0 = cf.copy(); cf0[:, 2] = 0
    cf1 = cf.copy(); cf1[:, 2] = 1
    assert (O.preprocess(img, mean, cf0) == O.preprocess(img, mean, cf1)[:, :, :, ::-1]).all()


# -------------------------------------------------------------- convolution

def brute_conv(x, w, b, s, p, g):
    N, Cin, H, W = x.shape
    Cout, cig, kh, kw = w.shape
    Ho, Wo = (H + 2 * p - kh) // s + 1, (W + 2 * p - kw) // s + 1
    y = np.zeros((N, Cout, Ho, Wo))
    for n in range(N):
        for co in range(Cout):
            grp = co // (Cout // g)
            for oy in range(Ho):
                for ox in range(Wo):
                    acc = b[co]
                    for ci in range(cig):
                        for ky in range(kh):
                            for kx in range(kw):
                                iy, ix = oy * s + ky - p, ox * s + kx - p
                                if 0 <= iy < H and 0 <= ix < W:
                                    acc += w[co, ci, ky, kx] * x[n, grp * cig + ci, iy, ix]
                    y[n, co, oy, ox] = acc
    return y


CASES = [  # N, Cin, H, W, Cout, k, s, p, g
    (2, 4, 7, 6, 4, 3, 1, 1, 1),
    (2, 4, 7, 7, 6, 3, 1, 1, 2),
    (1, 3, 15, 15, 4, 11, 4, 0, 1),
    (2, 4, 6, 5, 4, 5, 1, 2, 2),
    (1, 2, 5, 5, 2, 3, 2, 0, 1),
]


@pytest.mark.parametrize("case", CASES)
def test_conv_forward_brute_force_and_torch(case):
    N, Cin, H, W, Cout, k, s, p, g = case
    x = rng.standard_normal((N, Cin, H, W))
    w = rng.standard_normal((Cout, Cin // g, k, k))
    b = rng.standard_normal(Cout)
    y = O.conv_fwd(x, w, b, s, p, g)
    assert np.allclose(y, brute_conv(x, w, b, s, p, g), atol=1e-12)
    yt = F.conv2d(torch.from_numpy(x), torch.from_numpy(w), torch.from_numpy(b), stride=s, padding=p, groups=g)
    assert np.allclose(y, yt.numpy(), atol=1e-11)


@pytest.mark.parametrize("case", CASES)
def test_conv_backward_torch_autograd_and_finite_differences(case):
    N, Cin, H, W, Cout, k, s, p, g = case
    x = rng.standard_normal((N, Cin, H, W))
    w = rng.standard_normal((Cout, Cin // g, k, k))
    b = rng.standard_normal(Cout)
    y = O.conv_fwd(x, w, b, s, p, g)
    dy = rng.standard_normal(y.shape)
    dx = O.conv_bwd_data(dy, w, x.shape, s, p, g)
    dw, db = O.conv_bwd_weight(x, dy, w.shape, s, p, g)
    xt = torch.from_numpy(x).requires_grad_()
    wt = torch.from_numpy(w).requires_grad_()
    bt = torch.from_numpy(b).requires_grad_()
    (F.conv2d(xt, wt, bt, stride=s, padding=p, groups=g) * torch.from_numpy(dy)).sum().backward()
    assert np.allclose(dx, xt.grad.numpy(), atol=1e-11)
    assert np.allclose(dw, wt.grad.numpy(), atol=1e-11)
    assert np.allclose(db, bt.grad.numpy(), atol=1e-11)
    # central differences on a few coordinates, loss = sum(y * dy)
    h = 1e-5
    for _ in range(4):
        i = tuple(rng.integers(0, d) for d in x.shape)
        xp, xm = x.copy(), x.copy(); xp[i] += h; xm[i] -= h
        fd = ((O.conv_fwd(xp, w, b, s, p, g) - O.conv_fwd(xm, w, b, s, p, g)) * dy).sum() / (2 * h)
        assert abs(fd - dx[i]) < 1e-6 * max(1, abs(fd))
        j = tuple(rng.integers(0, d) for d in w.shape)
        wp, wm = w.copy(), w.copy(); wp[j] += h; wm[j] -= h
        fd = ((O.conv_fwd(x, wp, b, s, p, g) - O.conv_fwd(x, wm, b, s, p, g)) * dy).sum() / (2 * h)
        assert abs(fd - dw[j]) < 1e-6 * max(1, abs(fd))


def test_conv_closed_forms():
    # all ones: output = number of in-bounds taps * Cin/g
    x = np.ones((1, 4, 6, 6)); w = np.ones((2, 2, 3, 3))
    y = O.conv_fwd(x, w, None, 1, 1, 2)
    assert y[0, 0, 3, 3] == 18 and y[0, 1, 0, 0] == 8 and y[0, 0, 0, 2] == 12
    # centre delta kernel = identity (per channel)
    x = rng.standard_normal((2, 3, 5, 7)); w = np.zeros((3, 1, 3, 3)); w[:, 0, 1, 1] = 1
    assert (O.conv_fwd(x, w, None, 1, 1, 3) == x).all()
    # off-centre delta = shift; cross-correlation (no flip): y[oy,ox] = x[oy+ky-p, ox+kx-p]
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 2] = 1
    x = rng.standard_normal((1, 1, 5, 5))
    y = O.conv_fwd(x, w, None, 1, 1, 1)
    assert y[0, 0, 2, 2] == x[0, 0, 1, 3] and y[0, 0, 0, 0] == 0 and y[0, 0, 1, 4] == 0
    # 1x1 conv = matrix multiply over channels
    x = rng.standard_normal((2, 5, 4, 4)); w = rng.standard_normal((3, 5, 1, 1))
    assert np.allclose(O.conv_fwd(x, w, None, 1, 0, 1), np.einsum("oc,nchw->nohw", w[:, :, 0, 0], x))
    # kernel as large as the input = fully connected layer
    x = rng.standard_normal((3, 2, 4, 4)); w = rng.standard_normal((5, 2, 4, 4)); b = rng.standard_normal(5)
    assert np.allclose(O.conv_fwd(x, w, b, 1, 0, 1)[:, :, 0, 0], O.fc_fwd(x.reshape(3, -1), w.reshape(5, -1), b))


def test_conv_stride4_equals_space_to_depth_stride1():
    # 11x11/4 conv on 227 == 3x3/1 conv on the 4x4 space-to-depth of the (228-padded) input with a 12x12 zero-padded filter
    x = rng.standard_normal((1, 3, 27, 27)); w = rng.standard_normal((2, 3, 11, 11))
    y = O.conv_fwd(x, w, None, 4, 0, 1)          # 5x5
    xp = np.zeros((1, 3, 28, 28)); xp[:, :, :27, :27] = x
    wp = np.zeros((2, 3, 12, 12)); wp[:, :, :11, :11] = w
    xs = xp.reshape(1, 3, 7, 4, 7, 4).transpose(0, 3, 5, 1, 2, 4).reshape(1, 48, 7, 7)
    ws = wp.reshape(2, 3, 3, 4, 3, 4).transpose(0, 3, 5, 1, 2, 4).reshape(2, 48, 3, 3)
    assert np.allclose(O.conv_fwd(xs, ws, None, 1, 0, 1), y, atol=1e-12)


def test_group_symmetry_and_batch_equivariance():
    xh = rng.standard_normal((2, 2, 5, 5)); wh = rng.standard_normal((3, 2, 3, 3))
    y = O.conv_fwd(np.concatenate([xh, xh], 1), np.concatenate([wh, wh], 0), None, 1, 1, 2)
    assert (y[:, :3] == y[:, 3:]).all()
    x = rng.standard_normal((3, 4, 5, 5)); w = rng.standard_normal((4, 2, 3, 3))
    perm = [2, 0, 1]
    assert (O.conv_fwd(x[perm], w, None, 1, 1, 2) == O.conv_fwd(x, w, None, 1, 1, 2)[perm]).all()


# ---------------------------------------------------------------------- LRN

def test_lrn_hand_values():
    # one pixel; s_c = 2 + 1e-4 * (sum of squares over the clipped 5-window), by hand:
    a = np.array([10, 20, 30, 40, 50, 60], float).reshape(1, 6, 1, 1)
    s = [2 + 1e-4 * v for v in (100 + 400 + 900, 100 + 400 + 900 + 1600, 100 + 400 + 900 + 1600 + 2500,
                                400 + 900 + 1600 + 2500 + 3600, 900 + 1600 + 2500 + 3600, 1600 + 2500 + 3600)]
    assert np.allclose(s, [2.14, 2.30, 2.55, 2.90, 2.86, 2.77])
    assert np.allclose(O.lrn_scale(a).ravel(), s, rtol=1e-14)
    b = O.lrn_fwd(a).ravel()
    assert np.allclose(b, [v / sv ** 0.75 for v, sv in zip(a.ravel(), s)], rtol=1e-14)
    assert abs(b[0] - 5.651837543488) < 1e-11 and abs(b[5] - 27.944183440894) < 1e-11
    # constant 100 over 7 channels: window sizes 3,4,5,5,5,4,3 -> s = 5,6,7,7,7,6,5
    a = np.full((1, 7, 1, 1), 100.0)
    assert np.allclose(O.lrn_scale(a).ravel(), [5, 6, 7, 7, 7, 6, 5])
    assert abs(O.lrn_fwd(a).ravel()[3] - 100 * 7 ** -0.75) < 1e-12
    # all-ones interior channel: (2 + 5e-4)^-0.75
    assert abs(O.lrn_fwd(np.ones((1, 9, 1, 1))).ravel()[4] - 2.0005 ** -0.75) < 1e-15


def test_lrn_matches_torch_with_alpha_times_n():
    a = rng.standard_normal((2, 11, 3, 4)) * 30
    t = F.local_response_norm(torch.from_numpy(a), 5, alpha=5e-4, beta=0.75, k=2.0)  # torch divides alpha by n
    assert np.allclose(O.lrn_fwd(a), t.numpy(), rtol=1e-12)
    g = rng.standard_normal(a.shape)
    at = torch.from_numpy(a).requires_grad_()
    (F.local_response_norm(at, 5, alpha=5e-4, beta=0.75, k=2.0) * torch.from_numpy(g)).sum().backward()
    assert np.allclose(O.lrn_bwd(a, g), at.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_lrn_backward_finite_differences_and_hand_example():
    a = np.array([10, 20, 30, 40, 50, 60], float).reshape(1, 6, 1, 1)
    g = np.array([1, -1, 2, 0.5, -2, 1], float).reshape(1, 6, 1, 1)
    da = O.lrn_bwd(a, g).ravel()
    h = 1e-5
    for m in range(6):
        ap, am = a.copy(), a.copy(); ap[0, m] += h; am[0, m] -= h
        fd = ((O.lrn_fwd(ap) - O.lrn_fwd(am)) * g).sum() / (2 * h)
        assert abs(fd - da[m]) < 5e-9
    a = rng.standard_normal((2, 9, 2, 2)) * 50; g = rng.standard_normal(a.shape)
    da = O.lrn_bwd(a, g, alpha=1e-3)
    for _ in range(6):
        i = tuple(rng.integers(0, d) for d in a.shape)
        ap, am = a.copy(), a.copy(); ap[i] += h; am[i] -= h
        fd = ((O.lrn_fwd(ap, alpha=1e-3) - O.lrn_fwd(am, alpha=1e-3)) * g).sum() / (2 * h)
        assert abs(fd - da[i]) < 1e-7 * max(1, abs(fd))


# --------------------------------------------------------------------- pool

def test_pool_invariants_and_torch():
    x = rng.standard_normal((2, 3, 13, 13))
    y, arg = O.pool_fwd(x)
    assert y.shape == (2, 3, 6, 6)
    yt, it = F.max_pool2d(torch.from_numpy(x), 3, 2, return_indices=True)
    assert (y == yt.numpy()).all()
    oy, ox = np.meshgrid(np.arange(6), np.arange(6), indexing="ij")
    flat = (2 * oy + arg // 3) * 13 + 2 * ox + arg % 3
    assert (flat == it.numpy()).all()
    for n in range(2):
        for c in range(3):
            for i in range(6):
                for j in range(6):
                    win = x[n, c, 2 * i:2 * i + 3, 2 * j:2 * j + 3]
                    assert y[n, c, i, j] == win.max() == win[arg[n, c, i, j] // 3, arg[n, c, i, j] % 3]
    dy = rng.standard_normal(y.shape)
    dx = O.pool_bwd(dy, arg, x.shape)
    assert abs(dx.sum() - dy.sum()) < 1e-12
    xt = torch.from_numpy(x).requires_grad_()
    (F.max_pool2d(xt, 3, 2) * torch.from_numpy(dy)).sum().backward()
    assert np.allclose(dx, xt.grad.numpy(), atol=1e-14)


def test_pool_tie_break_is_first_in_row_major():
    x = np.zeros((1, 1, 5, 5))
    y, arg = O.pool_fwd(x)
    assert (arg == 0).all()
    x[0, 0, 1, 2] = 1.0; x[0, 0, 2, 1] = 1.0   # two equal maxima: row-major first is (1,2)
    y, arg = O.pool_fwd(x)
    assert arg[0, 0, 0, 0] == 1 * 3 + 2 and arg[0, 0, 0, 1] == 1 * 3 + 0


# ---------------------------------------------------------- FC, softmax, SGD

def test_fc_matches_einsum_and_autograd():
    x = rng.standard_normal((4, 7)); w = rng.standard_normal((5, 7)); b = rng.standard_normal(5); dy = rng.standard_normal((4, 5))
    assert np.allclose(O.fc_fwd(x, w, b), np.einsum("bk,nk->bn", x, w) + b)
    dx, dw, db = O.fc_bwd(x, w, dy)
    xt, wt, bt = (torch.from_numpy(t).requires_grad_() for t in (x, w, b))
    (F.linear(xt, wt, bt) * torch.from_numpy(dy)).sum().backward()
    assert np.allclose(dx, xt.grad.numpy()) and np.allclose(dw, wt.grad.numpy()) and np.allclose(db, bt.grad.numpy())


def test_softmax_xent_closed_forms():
    z = np.zeros((4, 1000)); lab = np.array([0, 5, 999, 17])
    p, L, dz = O.softmax_xent(z, lab)
    assert abs(L - math.log(1000)) < 1e-14 and abs(L - 6.907755278982137) < 1e-14
    z = rng.standard_normal((6, 1000)) * 10 + 500
    lab = rng.integers(0, 1000, 6)
    p, L, dz = O.softmax_xent(z, lab)
    assert np.allclose(p.sum(1), 1) and np.allclose(dz.sum(1), 0, atol=1e-15)
    zt = torch.from_numpy(z).requires_grad_()
    Lt = F.cross_entropy(zt, torch.from_numpy(lab)); Lt.backward()
    assert abs(L - Lt.item()) < 1e-12 and np.allclose(dz, zt.grad.numpy(), atol=1e-15)


def test_update_closed_form():
    mu, lr = 0.9, 0.01
    w0, v0 = rng.standard_normal(5), rng.standard_normal(5)
    w, v = w0.copy(), v0.copy()
    for t in range(1, 8):                       # g = 0, wd = 0: geometric series
        w, v = O.sgd_momentum(w, v, 0.0, lr, mu, 0.0, np.ones(5))
        assert np.allclose(v, mu ** t * v0) and np.allclose(w, w0 + v0 * mu * (1 - mu ** t) / (1 - mu))
    g = rng.standard_normal(5)                  # constant g from rest
    w, v = w0.copy(), np.zeros(5)
    for t in range(1, 6):
        w, v = O.sgd_momentum(w, v, g, lr, mu, 0.0, np.ones(5))
        assert np.allclose(v, -lr * g * (1 - mu ** t) / (1 - mu))
    # weight decay acts like an extra gradient wd*w, only where the mask is set
    w1, v1 = O.sgd_momentum(w0, v0, g, lr, mu, 5e-4, np.array([1, 1, 0, 0, 1.0]))
    assert np.allclose(v1, mu * v0 - lr * (g + 5e-4 * np.array([1, 1, 0, 0, 1.0]) * w0))
    m = O.decay_mask()
    off, tot = O.param_offsets()
    assert m.sum() == tot - 10568 and m[off["conv1.b"][0]] == 0 and m[off["fc8.W"][0]] == 1


def test_canonical_parameter_offsets():
    off, tot = O.param_offsets()
    assert tot == 60965224
    want = {"conv1.W": 0, "conv1.b": 34848, "conv2.W": 34944, "conv2.b": 342144, "conv3.W": 342400,
            "conv3.b": 1227136, "conv4.W": 1227520, "conv4.b": 1891072, "conv5.W": 1891456, "conv5.b": 2333824,
            "fc6.W": 2334080, "fc6.b": 40082816, "fc7.W": 40086912, "fc7.b": 56864128, "fc8.W": 56868224,
            "fc8.b": 60964224}
    assert {k: v[0] for k, v in off.items()} == want
    assert [n for n, _ in O.param_shapes()] == [n for n, _ in synth.PARAM_SHAPES]
    assert [s for _, s in O.param_shapes()] == [s for _, s in synth.PARAM_SHAPES]


def test_replica_average_algebra():
    a, b = rng.standard_normal(100), rng.standard_normal(100)
    ma, mb = O.replica_average(a, b)
    assert (ma == mb).all() and np.allclose(ma, 0.5 * (a + b))
    ia, ib = O.replica_average(a, a.copy())
    assert (ia == a).all() and (ib == a).all()          # identical replicas: bitwise identity
    # averaging params+momentum after separate updates == one update with the mean gradient
    w, v, ga, gb = (rng.standard_normal(50) for _ in range(4))
    mask = np.ones(50)
    wa, va = O.sgd_momentum(w, v, ga, 0.01, 0.9, 5e-4, mask)
    wb, vb = O.sgd_momentum(w, v, gb, 0.01, 0.9, 5e-4, mask)
    wm, vm = O.sgd_momentum(w, v, 0.5 * (ga + gb), 0.01, 0.9, 5e-4, mask)
    assert np.allclose(O.replica_average(wa, wb)[0], wm, atol=1e-15)
    assert np.allclose(O.replica_average(va, vb)[0], vm, atol=1e-15)


def test_round_bf16():
    x = np.array([1.0, 1.00390625, 1.005859375, -3.14159, 1e-3, 0.0])
    t = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert (O.round_bf16(x) == t).all()
    r = rng.standard_normal(1000) * 100
    assert (O.round_bf16(r) == torch.tensor(r, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()).all()


# ---------------------------------------------------------------- intensity augmentation (the one the paper skips)
def test_normal_draws_are_standard_normal_and_reproducible():
    z = O.normal_draws(7, 10, 0, 3, 60000)
    assert np.array_equal(z, O.normal_draws(7, 10, 0, 3, 60000))
    assert not np.array_equal(z[:100], O.normal_draws(7, 10, 1, 3, 100))            # another replica, other draws
    # moments of N(0,1) within sampling error (60000 draws: standard errors 0.004, 0.006, 0.01, 0.02)
    assert abs(z.mean()) < 0.02 and abs(z.var() - 1.0) < 0.03
    assert abs((z ** 3).mean()) < 0.05 and abs((z ** 4).mean() - 3.0) < 0.12
    # quantiles against the normal distribution function
    from math import erf, sqrt
    for x in (-2.0, -1.0, -0.25, 0.5, 1.5):
        assert abs((z < x).mean() - 0.5 * (1.0 + erf(x / sqrt(2.0)))) < 0.008
    # Box-Muller from the published hash: the first draw by hand
    r = O.draw(O.stream_key(7, 10, 0, 3), 0)
    u1, u2 = ((r >> 40) + 1) / 2.0 ** 24, ((r >> 16) & 0xFFFFFF) / 2.0 ** 24
    assert 0.0 < u1 <= 1.0 and 0.0 <= u2 < 1.0
    assert z[0] == np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def test_color_shift_special_cases():
    B = 64
    ident, ones = np.eye(3), np.ones(3)
    a = O.color_shift(5, 0, 2, B, ident, ones, 0.1)
    assert a.shape == (B, 3)
    # identity components, unit eigenvalues: the offsets are the draws themselves, image n using draws 3n..3n+2
    assert np.allclose(a, 0.1 * O.normal_draws(5, 10, 0, 2, 3 * B).reshape(B, 3), rtol=0, atol=1e-15)
    assert np.array_equal(O.color_shift(5, 0, 2, B, ident, ones, 0.0), np.zeros((B, 3)))
    # a rotation of the components preserves the length of every offset; eigenvalues scale the coordinates
    th = 0.7
    rot = np.array([[np.cos(th), -np.sin(th), 0.0], [np.sin(th), np.cos(th), 0.0], [0.0, 0.0, 1.0]])
    lam = np.array([3.0, 2.0, 0.5])
    b = O.color_shift(5, 0, 2, B, rot, lam, 0.1)
    assert np.allclose(np.linalg.norm(b, axis=1), np.linalg.norm(a * lam, axis=1), rtol=1e-12)
    # a single component along (1,1,1)/sqrt 3 shifts all three colours alike: a pure intensity change
    grey = np.zeros((3, 3)); grey[:, 0] = 1.0 / np.sqrt(3.0)
    c = O.color_shift(5, 0, 2, B, grey, np.array([4.0, 0.0, 0.0]), 0.1)
    assert np.allclose(c[:, 0], c[:, 1]) and np.allclose(c[:, 1], c[:, 2]) and np.abs(c).max() > 0
    # column i of eigvec is component i: with eigval e_1 only the second column matters
    only1 = O.color_shift(5, 0, 2, B, rot, np.array([0.0, 1.0, 0.0]), 0.1)
    assert np.allclose(only1, np.outer(a[:, 1], rot[:, 1]), atol=1e-15)


def test_preprocess_with_shift_is_a_per_image_colour_offset():
    rng = np.random.default_rng(4)
    img = rng.integers(0, 256, size=(3, 256, 256, 3), dtype=np.uint8)
    mean = rng.uniform(100, 140, size=(256, 256, 3))
    cf = O.crop_flip(9, 0, 0, 3)
    shift = rng.standard_normal((3, 3))
    x0, x1 = O.preprocess(img, mean, cf), O.preprocess(img, mean, cf, shift)
    d = x1 - x0
    for n in range(3):
        for c in range(3):
            assert np.allclose(d[n, c], shift[n, c], rtol=0, atol=1e-12)
