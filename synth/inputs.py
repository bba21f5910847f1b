"""Seeded synthetic tensors standing in for the paper's image workloads.

The paper measures on ImageNetV2 / CIFAR-10 activations and pretrained weights;
none of that data is used here.  Activations are ReLU'd standard normals,
weights are He-normal N(0, 2/(9*C)) (fan-in 9*C), or plain N(0,1) for the
smallest case.  Values are generated in float64 by numpy's Philox counter-based
generator from a fixed seed and rounded once to the storage dtype; the same
bytes go to the oracle and to the GPU.
"""
from dataclasses import dataclass
import numpy as np


@dataclass(frozen=True)
class ConvCase:
    name: str
    m: int
    N: int
    H: int
    W: int
    C: int
    K: int
    dtype: str          # "fp32" or "fp16"
    relu_inputs: bool
    he_weights: bool
    seed: int
    point_kinds: tuple  # keys into synth.points.POINT_SETS for this tile


CONFIGS = {
    "cfg1": ConvCase("cfg1", 2, 1, 16, 16, 8, 8, "fp32", False, False, 1001, ("std",)),
    "cfg2": ConvCase("cfg2", 4, 8, 56, 56, 64, 64, "fp16", True, True, 1002, ("std", "nova", "dyadic")),
    "cfg3": ConvCase("cfg3", 6, 32, 56, 56, 256, 256, "fp16", True, True, 1003, ("half", "nova", "std")),
    "cfg4": ConvCase("cfg4", 8, 32, 28, 28, 512, 512, "fp16", True, True, 1004, ("std", "nova")),
}


def _rng(seed, stream):
    return np.random.Generator(np.random.Philox(key=seed, counter=[0, 0, 0, stream]))


def make_conv_inputs(N, H, W, C, K, dtype="fp16", relu_inputs=True, he_weights=True,
                     seed=0, c_valid=None, r=3):
    """x [N,H,W,C] and g [K,r,r,C] in the storage dtype (numpy arrays).

    c_valid < C zero-fills channels c_valid..C-1 of both tensors (used when a
    3-channel image is padded to 8 channels); the He fan-in is then 9*c_valid.
    """
    cv = C if c_valid is None else c_valid
    x = _rng(seed, 1).standard_normal((N, H, W, C))
    if relu_inputs:
        x = np.maximum(x, 0.0)
    g = _rng(seed, 2).standard_normal((K, r, r, C))
    if he_weights:
        g *= np.sqrt(2.0 / (float(r * r) * cv))
    if cv < C:
        x[..., cv:] = 0.0
        g[..., cv:] = 0.0
    np_dtype = {"fp16": np.float16, "fp32": np.float32}[dtype]
    return x.astype(np_dtype), g.astype(np_dtype)


# (C_in, C_out, pool_after) for the 13 conv layers of VGG-16; input 224x224x3.
VGG16_LAYERS = (
    (3, 64, False), (64, 64, True),
    (64, 128, False), (128, 128, True),
    (128, 256, False), (256, 256, False), (256, 256, True),
    (256, 512, False), (512, 512, False), (512, 512, True),
    (512, 512, False), (512, 512, False), (512, 512, True),
)


def make_vgg_inputs(N, HW=224, dtype="fp16", seed=1005):
    """Image batch [N,HW,HW,8] (channels 3..7 zero) and the 13 weight tensors.

    Layer 0's weights are [64,3,3,8] with channels 3..7 zero and fan-in 27.
    """
    np_dtype = {"fp16": np.float16, "fp32": np.float32}[dtype]
    x = np.maximum(_rng(seed, 1).standard_normal((N, HW, HW, 8)), 0.0)
    x[..., 3:] = 0.0
    weights = []
    for li, (ci, co, _) in enumerate(VGG16_LAYERS):
        cpad = max(ci, 8)
        g = _rng(seed, 10 + li).standard_normal((co, 3, 3, cpad)) * np.sqrt(2.0 / (9.0 * ci))
        if ci < cpad:
            g[..., ci:] = 0.0
        weights.append(g.astype(np_dtype))
    return x.astype(np_dtype), weights
