"""TEST INFRASTRUCTURE ONLY -- fp64 CPU oracle of one AlexNet SGD training step.

This module is what the CUDA path is checked against.  It is a plain, slow,
obviously-correct implementation: the C file beside it holds the naive loops
(convolution, LRN, max-pool, preprocessing, the counter hash), the rest is a
few lines of numpy in fp64.  It shares nothing with the CUDA path and must not
be imported by the product package; only tests, the smoke check and the
bench's cpu-baseline leg may use it.

What it follows
  * topology -- the paper's Methods section: 5 convolution layers, 3 of them
    followed by max-pooling, 2 fully connected layers and a softmax layer; the
    layer constants are those of Krizhevsky et al. 2012, which the paper cites.
  * preprocessing -- footnote of the "Parallel Data Loading" subsection: subtract
    the mean image, random crop, random flip.
  * two replicas, exchange and average of weights, biases and momentum -- the
    "Data parallelism" subsection and its figure.

Readings taken where the paper is silent are listed with the design notes of
this repository; the ones that matter here: conv -> +bias -> ReLU -> LRN ->
pool order; LRN alpha is not divided by the window size; cross-correlation;
momentum update v <- mu v - lr wd w - lr g, w <- w + v with decay on weights
only; dropout without rescaling; pool ties go to the first element in
row-major order; loss is the mean over the batch.

Parity status: all functions are pinned by tests/test_oracle_*.py.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "alexnet_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile the C part with gcc (OpenMP) if missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_mix64.restype = ctypes.c_uint64
        _lib.orc_mix64.argtypes = [ctypes.c_uint64]
        _lib.orc_key.restype = ctypes.c_uint64
        _lib.orc_key.argtypes = [ctypes.c_uint64] * 4
        _lib.orc_draw.restype = ctypes.c_uint64
        _lib.orc_draw.argtypes = [ctypes.c_uint64] * 2
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


I = ctypes.c_int
D = ctypes.c_double
U64 = ctypes.c_uint64

# ----------------------------------------------------------------- hashing


def mix64(z: int) -> int:
    return int(lib().orc_mix64(U64(z & (2**64 - 1))))


def stream_key(seed, stream, replica, step) -> int:
    return int(lib().orc_key(U64(seed), U64(stream), U64(replica), U64(step)))


def draw(key, idx) -> int:
    return int(lib().orc_draw(U64(key), U64(idx)))


def crop_flip(seed, replica, step, B) -> np.ndarray:
    """(B,3) int32: ox, oy in [0,29], flip in {0,1} -- one draw per image."""
    out = np.zeros((B, 3), np.int32)
    lib().orc_crop_flip(U64(seed), U64(replica), U64(step), I(B), _p(out))
    return out


def dropout_mask(seed, layer_stream, replica, step, B, width, p) -> np.ndarray:
    """(B,width) uint8 keep mask; layer_stream 2 = fc6, 3 = fc7."""
    out = np.zeros((B, width), np.uint8)
    lib().orc_dropout_mask(U64(seed), U64(layer_stream), U64(replica), U64(step), I(B), I(width), D(p), _p(out))
    return out


# ----------------------------------------------------------- layer functions


def preprocess(img_u8, mean, cf, shift=None) -> np.ndarray:
    """img_u8 (B,256,256,3) uint8, mean (256,256,3), cf (B,3) -> X (B,3,227,227) fp64.
    shift (B,3), optional: one RGB offset per image, added to every pixel (color_shift below)."""
    img_u8 = np.ascontiguousarray(img_u8, np.uint8)
    B = img_u8.shape[0]
    X = np.empty((B, 3, 227, 227), np.float64)
    cf = np.ascontiguousarray(cf, np.int32)
    lib().orc_preprocess(_p(img_u8), _p(_f64(mean)), _p(cf), I(B), _p(X))
    if shift is not None:
        X += np.asarray(shift, np.float64)[:, :, None, None]
    return X


def normal_draws(seed, stream, replica, step, count) -> np.ndarray:
    """count standard-normal draws from the counter hash: draw r(idx) gives u1 = (top 24 bits + 1) / 2^24 in (0, 1] and
    u2 = (bits 16..39) / 2^24 in [0, 1); z = sqrt(-2 ln u1) cos(2 pi u2) (Box-Muller, first variate)."""
    key = stream_key(seed, stream, replica, step)
    z = np.empty(count, np.float64)
    for i in range(count):
        r = draw(key, i)
        u1 = ((r >> 40) + 1) / 16777216.0
        u2 = ((r >> 16) & 0xFFFFFF) / 16777216.0
        z[i] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return z


def color_shift(seed, replica, step, B, eigvec, eigval, sigma) -> np.ndarray:
    """The intensity augmentation of Krizhevsky et al. 2012 (section 4.1), which the paper's experiments leave out
    ("Experiments", the sentence on the reported error rates): to every pixel of image n add
    eigvec @ (alpha_n * eigval), where eigvec (3,3: columns are the principal components of the RGB pixel values of
    the training set) and eigval (3,) are dataset constants and alpha_n (3,) ~ N(0, sigma^2) is drawn once per image
    (hash stream 10, index 3 n + i).  Returns (B,3) offsets; sigma = 0 gives zeros."""
    alpha = sigma * normal_draws(seed, 10, replica, step, 3 * B).reshape(B, 3)
    return (alpha * np.asarray(eigval, np.float64)[None, :]) @ np.asarray(eigvec, np.float64).T


def conv_fwd(x, w, b, stride, pad, groups):
    x, w = _f64(x), _f64(w)
    b = _f64(b) if b is not None else None
    N, Cin, H, W = x.shape
    Cout, _, kh, kw = w.shape
    Ho = (H + 2 * pad - kh) // stride + 1
    Wo = (W + 2 * pad - kw) // stride + 1
    y = np.empty((N, Cout, Ho, Wo), np.float64)
    lib().orc_conv_fwd(_p(x), _p(w), _p(b), _p(y), I(N), I(Cin), I(H), I(W), I(Cout), I(kh), I(kw), I(stride), I(pad), I(groups))
    return y


def conv_bwd_data(dy, w, x_shape, stride, pad, groups):
    dy, w = _f64(dy), _f64(w)
    N, Cin, H, W = x_shape
    Cout, _, kh, kw = w.shape
    dx = np.empty((N, Cin, H, W), np.float64)
    lib().orc_conv_bwd_data(_p(dy), _p(w), _p(dx), I(N), I(Cin), I(H), I(W), I(Cout), I(kh), I(kw), I(stride), I(pad), I(groups))
    return dx


def conv_bwd_weight(x, dy, w_shape, stride, pad, groups):
    x, dy = _f64(x), _f64(dy)
    N, Cin, H, W = x.shape
    Cout, cig, kh, kw = w_shape
    dw = np.empty(w_shape, np.float64)
    db = np.empty((Cout,), np.float64)
    lib().orc_conv_bwd_weight(_p(x), _p(dy), _p(dw), _p(db), I(N), I(Cin), I(H), I(W), I(Cout), I(kh), I(kw), I(stride), I(pad), I(groups))
    return dw, db


def lrn_fwd(a, size=5, alpha=1e-4, beta=0.75, k=2.0):
    a = _f64(a)
    N, C, H, W = a.shape
    b = np.empty_like(a)
    lib().orc_lrn_fwd(_p(a), _p(b), None, I(N), I(C), I(H * W), I(size), D(alpha), D(beta), D(k))
    return b


def lrn_scale(a, size=5, alpha=1e-4, beta=0.75, k=2.0):
    a = _f64(a)
    N, C, H, W = a.shape
    b = np.empty_like(a)
    s = np.empty_like(a)
    lib().orc_lrn_fwd(_p(a), _p(b), _p(s), I(N), I(C), I(H * W), I(size), D(alpha), D(beta), D(k))
    return s


def lrn_bwd(a, g, size=5, alpha=1e-4, beta=0.75, k=2.0):
    a, g = _f64(a), _f64(g)
    N, C, H, W = a.shape
    da = np.empty_like(a)
    lib().orc_lrn_bwd(_p(a), _p(g), _p(da), I(N), I(C), I(H * W), I(size), D(alpha), D(beta), D(k))
    return da


def pool_fwd(x, k=3, s=2):
    x = _f64(x)
    N, C, H, W = x.shape
    Ho, Wo = (H - k) // s + 1, (W - k) // s + 1
    y = np.empty((N, C, Ho, Wo), np.float64)
    arg = np.empty((N, C, Ho, Wo), np.uint8)
    lib().orc_pool_fwd(_p(x), _p(y), _p(arg), I(N), I(C), I(H), I(W), I(k), I(s))
    return y, arg


def pool_bwd(dy, arg, x_shape, k=3, s=2):
    dy = _f64(dy)
    arg = np.ascontiguousarray(arg, np.uint8)
    N, C, H, W = x_shape
    dx = np.empty(x_shape, np.float64)
    lib().orc_pool_bwd(_p(dy), _p(arg), _p(dx), I(N), I(C), I(H), I(W), I(k), I(s))
    return dx


def fc_fwd(x, w, b):
    """y = x W^T + b ; x (B,K), w (N,K)."""
    return _f64(x) @ _f64(w).T + _f64(b)


def fc_bwd(x, w, dy):
    """dx = dy W, dW = dy^T x, db = sum_n dy."""
    x, w, dy = _f64(x), _f64(w), _f64(dy)
    return dy @ w, dy.T @ x, dy.sum(axis=0)


def softmax_xent(z, labels):
    """p = softmax(z) (max-subtracted); L = -mean log p[label]; dz = (p - onehot)/B."""
    z = _f64(z)
    B = z.shape[0]
    zs = z - z.max(axis=1, keepdims=True)
    e = np.exp(zs)
    p = e / e.sum(axis=1, keepdims=True)
    logp = zs - np.log(e.sum(axis=1, keepdims=True))
    loss = -logp[np.arange(B), labels].mean()
    dz = p.copy()
    dz[np.arange(B), labels] -= 1.0
    dz /= B
    return p, float(loss), dz


def sgd_momentum(w, v, g, lr, mu, wd, decay_mask):
    """v <- mu v - lr wd w (where decay applies) - lr g ; w <- w + v (Krizhevsky et al. 2012, Sec. 5)."""
    v_new = mu * v - lr * wd * decay_mask * w - lr * g
    return w + v_new, v_new


def replica_average(a, b):
    """Step 3 of the paper's data-parallel figure: both replicas take the mean."""
    m = (a + b) / 2.0
    return m, m.copy()


def round_bf16(x):
    """Round-to-nearest-even to bfloat16, returned as fp64 (for the bf16-aware diagnostic mode)."""
    f = np.ascontiguousarray(x, np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    return r.view(np.float32).astype(np.float64).reshape(np.shape(x))


# ------------------------------------------------------- canonical parameters

# name, kind, (cin, cout, k, stride, pad, groups) or (K, N)
CONV = {
    "conv1": dict(cin=3, cout=96, k=11, s=4, p=0, g=1),
    "conv2": dict(cin=96, cout=256, k=5, s=1, p=2, g=2),
    "conv3": dict(cin=256, cout=384, k=3, s=1, p=1, g=1),
    "conv4": dict(cin=384, cout=384, k=3, s=1, p=1, g=2),
    "conv5": dict(cin=384, cout=256, k=3, s=1, p=1, g=2),
}
FC = {"fc6": (9216, 4096), "fc7": (4096, 4096), "fc8": (4096, 1000)}


def param_shapes():
    """Canonical order: conv1.W, conv1.b, ..., fc8.W, fc8.b; conv W is [Cout][Cin/g][kh][kw], FC W is [N][K]."""
    out = []
    for name, c in CONV.items():
        out.append((name + ".W", (c["cout"], c["cin"] // c["g"], c["k"], c["k"])))
        out.append((name + ".b", (c["cout"],)))
    for name, (K, N) in FC.items():
        out.append((name + ".W", (N, K)))
        out.append((name + ".b", (N,)))
    return out


def param_offsets():
    off, o = {}, 0
    for name, shp in param_shapes():
        n = int(np.prod(shp))
        off[name] = (o, n, shp)
        o += n
    return off, o


PARAM_COUNT = param_offsets()[1]  # 60,965,224


def unpack(flat):
    off, _ = param_offsets()
    return {k: flat[o:o + n].reshape(shp) for k, (o, n, shp) in off.items()}


def decay_mask(wd_on_biases=False):
    off, tot = param_offsets()
    m = np.zeros(tot, np.float64)
    for k, (o, n, _) in off.items():
        if k.endswith(".W") or wd_on_biases:
            m[o:o + n] = 1.0
    return m


@dataclass
class OracleConfig:
    seed: int = 14122302
    lr: float = 0.01
    momentum: float = 0.9
    weight_decay: float = 5e-4
    lrn_size: int = 5
    lrn_alpha: float = 1e-4
    lrn_beta: float = 0.75
    lrn_k: float = 2.0
    dropout_p: float = 0.5
    lrn_alpha_div_n: bool = False
    wd_on_biases: bool = False
    inverted_dropout: bool = False
    bf16_aware: bool = False  # diagnostic: round where the GPU stores bf16
    color: tuple = None       # (eigvec (3,3), eigval (3,), sigma): intensity augmentation in training passes; None = off


@dataclass
class OracleNet:
    cfg: OracleConfig
    w: np.ndarray  # canonical flat fp64
    v: np.ndarray = field(default=None)
    replica: int = 0

    def __post_init__(self):
        self.w = np.array(self.w, np.float64)
        self.v = np.zeros_like(self.w) if self.v is None else np.array(self.v, np.float64)

    # -- helpers
    def _q(self, x):
        return round_bf16(x) if self.cfg.bf16_aware else x

    def _lrn_args(self):
        c = self.cfg
        a = c.lrn_alpha / c.lrn_size if c.lrn_alpha_div_n else c.lrn_alpha
        return dict(size=c.lrn_size, alpha=a, beta=c.lrn_beta, k=c.lrn_k)

    def forward_backward(self, img_u8, labels, mean, step, cf=None, m6=None, m7=None, mean_over=None,
                         gates=None, args=None):
        """One forward + backward pass.  Returns a dict with every intermediate
        (canonical NCHW fp64), the flat canonical gradient 'g' and 'loss'.
        cf / m6 / m7 override the hashed crop-flip triples and dropout masks and
        mean_over the batch size of the loss mean, so that a few images of a
        larger batch can be evaluated on their own.

        gates / args: the discrete decisions of the backward pass (which units
        pass gradient through ReLU and dropout; which window element receives a
        pool gradient) are by default the oracle's own, taken in fp64.  A caller
        comparing against an implementation that stores bf16 activations passes
        that implementation's decisions here (dicts keyed a1..a5, f6, f7 and
        arg1, arg2, arg5) after checking them valid, so that both sides take
        each decision in the same precision; the forward pass is unaffected."""
        c = self.cfg
        q = self._q
        P = unpack(self.w)
        Pq = {k: q(a) if k.endswith(".W") else a for k, a in P.items()}
        B = img_u8.shape[0]
        T = {}
        T["cf"] = crop_flip(c.seed, self.replica, step, B) if cf is None else np.asarray(cf, np.int32)
        shift = color_shift(c.seed, self.replica, step, B, *c.color) if c.color else None
        T["x0"] = q(preprocess(img_u8, mean, T["cf"], shift))
        la = self._lrn_args()

        def conv_block(name, x):
            cc = CONV[name]
            z = conv_fwd(x, Pq[name + ".W"], P[name + ".b"], cc["s"], cc["p"], cc["g"])
            T["pre_a" + name[-1]] = z
            return q(np.maximum(z, 0.0))

        def gate(k):
            return np.asarray(gates[k], bool) if gates is not None else (T[k] > 0)

        def arg(k):
            return np.asarray(args[k], np.uint8) if args is not None else T[k]

        T["a1"] = conv_block("conv1", T["x0"])
        T["n1"] = q(lrn_fwd(T["a1"], **la))
        T["p1"], T["arg1"] = pool_fwd(T["n1"])
        T["a2"] = conv_block("conv2", T["p1"])
        T["n2"] = q(lrn_fwd(T["a2"], **la))
        T["p2"], T["arg2"] = pool_fwd(T["n2"])
        T["a3"] = conv_block("conv3", T["p2"])
        T["a4"] = conv_block("conv4", T["a3"])
        T["a5"] = conv_block("conv5", T["a4"])
        T["p5"], T["arg5"] = pool_fwd(T["a5"])
        flat = T["p5"].reshape(B, 9216)  # C,H,W order
        scale = 1.0 / (1.0 - c.dropout_p) if (c.inverted_dropout and c.dropout_p > 0) else 1.0
        if m6 is not None:
            T["m6"], T["m7"] = np.asarray(m6, np.uint8), np.asarray(m7, np.uint8)
        elif c.dropout_p > 0:
            T["m6"] = dropout_mask(c.seed, 2, self.replica, step, B, 4096, c.dropout_p)
            T["m7"] = dropout_mask(c.seed, 3, self.replica, step, B, 4096, c.dropout_p)
        else:
            T["m6"] = np.ones((B, 4096), np.uint8)
            T["m7"] = np.ones((B, 4096), np.uint8)
        T["pre_f6"] = fc_fwd(flat, Pq["fc6.W"], P["fc6.b"])
        T["f6"] = q(np.maximum(T["pre_f6"], 0.0) * T["m6"] * scale)
        T["pre_f7"] = fc_fwd(T["f6"], Pq["fc7.W"], P["fc7.b"])
        T["f7"] = q(np.maximum(T["pre_f7"], 0.0) * T["m7"] * scale)
        T["z"] = fc_fwd(T["f7"], Pq["fc8.W"], P["fc8.b"])
        T["prob"], T["loss"], dz = softmax_xent(T["z"], labels)
        if mean_over is not None:
            dz = dz * (B / float(mean_over))
        T["dz"] = q(dz)

        # ---- backward
        G = {}
        d7, G["fc8.W"], G["fc8.b"] = fc_bwd(T["f7"], Pq["fc8.W"], T["dz"])
        d7 = q(d7 * gate("f7") * scale)          # dropout mask and ReLU: f7 > 0 iff kept and positive
        T["df7"] = d7
        d6, G["fc7.W"], G["fc7.b"] = fc_bwd(T["f6"], Pq["fc7.W"], d7)
        d6 = q(d6 * gate("f6") * scale)
        T["df6"] = d6
        dp5, G["fc6.W"], G["fc6.b"] = fc_bwd(flat, Pq["fc6.W"], d6)
        T["dp5"] = q(dp5).reshape(T["p5"].shape)
        da5 = pool_bwd(T["dp5"], arg("arg5"), T["a5"].shape) * gate("a5")
        T["da5"] = q(da5)

        def conv_back(name, x, dy, need_dx=True):
            cc = CONV[name]
            dw, db = conv_bwd_weight(x, dy, P[name + ".W"].shape, cc["s"], cc["p"], cc["g"])
            G[name + ".W"], G[name + ".b"] = dw, db
            if not need_dx:
                return None
            return conv_bwd_data(dy, Pq[name + ".W"], x.shape, cc["s"], cc["p"], cc["g"])

        T["da4"] = q(conv_back("conv5", T["a4"], T["da5"]) * gate("a4"))
        T["da3"] = q(conv_back("conv4", T["a3"], T["da4"]) * gate("a3"))
        T["dp2"] = q(conv_back("conv3", T["p2"], T["da3"]))
        T["dn2"] = pool_bwd(T["dp2"], arg("arg2"), T["n2"].shape)
        T["da2"] = q(lrn_bwd(T["a2"], T["dn2"], **la) * gate("a2"))
        T["dp1"] = q(conv_back("conv2", T["p1"], T["da2"]))
        T["dn1"] = pool_bwd(T["dp1"], arg("arg1"), T["n1"].shape)
        T["da1"] = q(lrn_bwd(T["a1"], T["dn1"], **la) * gate("a1"))
        conv_back("conv1", T["x0"], T["da1"], need_dx=False)

        off, tot = param_offsets()
        g = np.empty(tot, np.float64)
        for k, (o, n, _) in off.items():
            g[o:o + n] = G[k].reshape(-1)
        T["g"] = g
        return T

    def train_step(self, img_u8, labels, mean, step, **kw):
        c = self.cfg
        T = self.forward_backward(img_u8, labels, mean, step, **kw)
        self.w, self.v = sgd_momentum(self.w, self.v, T["g"], c.lr, c.momentum, c.weight_decay,
                                      decay_mask(c.wd_on_biases))
        return T


def loader_order(n_images, batch, seed, shuffle, n_batches):
    """Dataset indices of the first n_batches minibatches of the loading process: sample j of the stream is entry
    perm_e[j mod n_epoch] of the dataset, e = j // n_epoch, n_epoch = (n_images // batch) * batch; perm_e is the
    identity or, with shuffle, the Fisher-Yates shuffle driven by the counter hash (stream 9, keyed by the epoch):
    for i = n_epoch-1 .. 1: swap entries i and draw(key_e, i) mod (i+1)."""
    n_epoch = (n_images // batch) * batch
    out, perms = [], {}
    for b in range(n_batches):
        idx = []
        for i in range(batch):
            j = b * batch + i
            e, pos = divmod(j, n_epoch)
            if e not in perms:
                perm = list(range(n_epoch))
                if shuffle:
                    key = mix64((seed ^ (9 << 56) ^ e) & (2**64 - 1))
                    for t in range(n_epoch - 1, 0, -1):
                        r = draw(key, t) % (t + 1)
                        perm[t], perm[r] = perm[r], perm[t]
                perms[e] = perm
            idx.append(perms[e][pos])
        out.append(np.array(idx, np.int64))
    return out


EVAL_CROP = 14      # (256 - 227) // 2: the centre 227 x 227 window starts at row/column 14


def topk_correct(z, labels, k):
    """Per sample 1 if the label is among the k largest logits, else 0.  Rank of the label = number of logits
    strictly greater than it plus the number of equal logits with a smaller class index (so ties are broken
    towards the smaller index and every sample has exactly k classes in its top k)."""
    z = _f64(z)
    labels = np.asarray(labels, np.int64)
    zl = z[np.arange(z.shape[0]), labels][:, None]
    idx = np.arange(z.shape[1])[None, :]
    rank = (z > zl).sum(axis=1) + ((z == zl) & (idx < labels[:, None])).sum(axis=1)
    return (rank < k).astype(np.int32)


def evaluate(net: OracleNet, img_u8, labels, mean):
    """Evaluation forward pass (the accuracy measurements of the paper's Experiments section are top-1 / top-5
    errors): centre crop, no flip, no dropout mask; with the non-inverted dropout of training the outputs of
    fc6 and fc7 are multiplied by (1 - p) instead (Krizhevsky et al. 2012, Sec. 4.2).  Returns logits, mean
    loss, and the per-sample top-1 / top-5 indicator vectors."""
    c = net.cfg
    P = unpack(net.w)
    B = img_u8.shape[0]
    cf = np.tile(np.array([EVAL_CROP, EVAL_CROP, 0], np.int32), (B, 1))
    x = preprocess(img_u8, mean, cf)
    la = net._lrn_args()

    def conv_block(name, x):
        cc = CONV[name]
        return np.maximum(conv_fwd(x, P[name + ".W"], P[name + ".b"], cc["s"], cc["p"], cc["g"]), 0.0)

    a = conv_block("conv1", x)
    a, _ = pool_fwd(lrn_fwd(a, **la))
    a = conv_block("conv2", a)
    a, _ = pool_fwd(lrn_fwd(a, **la))
    a = conv_block("conv5", conv_block("conv4", conv_block("conv3", a)))
    a, _ = pool_fwd(a)
    scale = 1.0 if (c.inverted_dropout or c.dropout_p == 0) else 1.0 - c.dropout_p
    f6 = np.maximum(fc_fwd(a.reshape(B, 9216), P["fc6.W"], P["fc6.b"]), 0.0) * scale
    f7 = np.maximum(fc_fwd(f6, P["fc7.W"], P["fc7.b"]), 0.0) * scale
    z = fc_fwd(f7, P["fc8.W"], P["fc8.b"])
    _, loss, _ = softmax_xent(z, labels)
    return dict(x0=x, f6=f6, f7=f7, z=z, loss=loss, top1=topk_correct(z, labels, 1), top5=topk_correct(z, labels, 5))


def average_replicas(a: OracleNet, b: OracleNet):
    """Exchange and average weights, biases and momentum of two replicas."""
    a.w, b.w = replica_average(a.w, b.w)
    a.v, b.v = replica_average(a.v, b.v)


def conv1_block(img_u8, mean, cf, w1, b1, upstream, cfg: OracleConfig = None, gates=None, args=None):
    """The conv1 block alone: preprocess -> conv1 -> ReLU -> LRN -> pool, with
    loss = sum(pooled * upstream); returns intermediates and dW1, db1.
    gates / args as in OracleNet.forward_backward."""
    cfg = cfg or OracleConfig()
    la = dict(size=cfg.lrn_size, alpha=cfg.lrn_alpha, beta=cfg.lrn_beta, k=cfg.lrn_k)
    T = {}
    T["x0"] = preprocess(img_u8, mean, cf)
    cc = CONV["conv1"]
    T["pre_a1"] = conv_fwd(T["x0"], w1, b1, cc["s"], cc["p"], cc["g"])
    T["a1"] = np.maximum(T["pre_a1"], 0.0)
    T["n1"] = lrn_fwd(T["a1"], **la)
    T["p1"], T["arg1"] = pool_fwd(T["n1"])
    T["loss"] = float((T["p1"] * upstream).sum())
    T["dn1"] = pool_bwd(_f64(upstream), T["arg1"] if args is None else np.asarray(args["arg1"], np.uint8), T["n1"].shape)
    T["da1"] = lrn_bwd(T["a1"], T["dn1"], **la) * ((T["a1"] > 0) if gates is None else np.asarray(gates["a1"], bool))
    T["dW1"], T["db1"] = conv_bwd_weight(T["x0"], T["da1"], w1.shape, cc["s"], cc["p"], cc["g"])
    return T
