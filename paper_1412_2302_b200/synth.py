"""Seeded synthetic inputs, shared by the tests, the bench and the CPU checker.

Only data generation lives here -- no layer arithmetic, no hashing of the
method.  The images stand in for ILSVRC-2012 as the paper's pipeline sees it:
256x256 RGB uint8 pictures with one of 1000 labels.  Pixel statistics do not
matter for dense convolutions, so bytes are iid uniform.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 14122302

# canonical parameter tensors in order; conv W is [Cout][Cin/groups][k][k], FC W is [N][K]
PARAM_SHAPES = [
    ("conv1.W", (96, 3, 11, 11)), ("conv1.b", (96,)),
    ("conv2.W", (256, 48, 5, 5)), ("conv2.b", (256,)),
    ("conv3.W", (384, 256, 3, 3)), ("conv3.b", (384,)),
    ("conv4.W", (384, 192, 3, 3)), ("conv4.b", (384,)),
    ("conv5.W", (256, 192, 3, 3)), ("conv5.b", (256,)),
    ("fc6.W", (4096, 9216)), ("fc6.b", (4096,)),
    ("fc7.W", (4096, 4096)), ("fc7.b", (4096,)),
    ("fc8.W", (1000, 4096)), ("fc8.b", (1000,)),
]


def _rng(seed, *tags):
    return np.random.default_rng([int(seed)] + [int(t) for t in tags])


def images(seed, replica, step, batch):
    """uint8 (batch, 256, 256, 3), iid uniform bytes."""
    return _rng(seed, 4, replica, step).integers(0, 256, size=(batch, 256, 256, 3), dtype=np.uint8)


def labels(seed, replica, step, batch):
    """int32 (batch,), uniform in [0, 1000)."""
    return _rng(seed, 5, replica, step).integers(0, 1000, size=(batch,), dtype=np.int32)


def mean_image(seed):
    """float32 (256, 256, 3), uniform in [100, 140): not constant, so that a
    wrong source coordinate in the mean subtraction is visible."""
    return _rng(seed, 7).uniform(100.0, 140.0, size=(256, 256, 3)).astype(np.float32)


def init_params(seed, std=0.01, variance_preserving=False, bias=0.0, input_std=74.0):
    """Flat canonical float32 parameter vector.  Weights N(0, std^2), or
    N(0, 2/fan_in) when variance_preserving (keeps deep-layer signals alive in
    parity tests; conv1 is further divided by input_std, the spread of the
    mean-subtracted uniform bytes, so activations stay O(1)); biases constant."""
    rng = _rng(seed, 6)
    parts = []
    for name, shp in PARAM_SHAPES:
        n = int(np.prod(shp))
        if name.endswith(".W"):
            s = np.sqrt(2.0 / np.prod(shp[1:])) if variance_preserving else std
            if variance_preserving and name == "conv1.W":
                s /= input_std
            parts.append((rng.standard_normal(n) * s).astype(np.float32))
        else:
            parts.append(np.full(n, bias, np.float32))
    return np.concatenate(parts)


def normal(seed, tag, shape, std=1.0):
    """float32 N(0, std^2) tensor, e.g. the upstream gradient of the conv1-block case."""
    return (_rng(seed, 8, tag).standard_normal(shape) * std).astype(np.float32)


def bf16_grid(seed, tag, shape, lo=-1.0, hi=1.0):
    """float32 values exactly representable in bfloat16 (multiples of 1/64 in
    [lo, hi]), for kernel-level tests where both sides must see identical inputs."""
    k = _rng(seed, 9, tag).integers(int(lo * 64), int(hi * 64) + 1, size=shape)
    return (k / 64.0).astype(np.float32)
