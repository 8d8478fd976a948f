"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path's tests and benchmark.

Holds no arithmetic of the method: only random draws.  CIFAR-10/100 are not available offline, so images are
iid N(0,1) tensors of CIFAR shape (NCHW, 3x32x32) and labels are uniform over the classes; a fresh batch is
drawn for every iteration so that delayed samples are distinguishable.
"""
import numpy as np

from . import nets

WEIGHT_SEED = 20180427


def batch(t, batch_size, in_shape, num_classes):
    """Inputs of iteration t: x ~ N(0,1) float32 [B, C, H, W], labels int32 uniform in [0, classes)."""
    x = np.random.default_rng(1000 + t).standard_normal((batch_size,) + tuple(in_shape), dtype=np.float32)
    y = np.random.default_rng(2000 + t).integers(0, num_classes, size=batch_size).astype(np.int32)
    return x, y


def init_weights(layers, seed=WEIGHT_SEED, perturb_affine=0.0):
    """He-normal N(0, 2/fan_in) conv/FC weights, zero biases, BN gamma=1 and beta=0, as float32 in the
    canonical flat order.  `perturb_affine` > 0 adds N(0, perturb_affine^2) noise to biases, gamma and beta so
    that tests exercise non-trivial values of them."""
    rng = np.random.default_rng(seed)
    w = np.zeros(nets.param_count(layers), dtype=np.float32)
    for _, name, off, shape, fan_in in nets.param_segments(layers):
        n = int(np.prod(shape))
        if fan_in is not None:
            w[off:off + n] = rng.standard_normal(n) * np.sqrt(2.0 / fan_in)
        else:
            base = 1.0 if name.endswith("gamma") else 0.0
            noise = rng.standard_normal(n) * perturb_affine if perturb_affine > 0 else 0.0
            w[off:off + n] = base + noise
    return w
