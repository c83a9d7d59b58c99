"""Layer shapes and seeded synthetic inputs for the XNOR-Net forward block.

This module holds NO arithmetic of the method: only shape tables and
random-number generation.  It is the one module both the CUDA tests/benchmark
and the CPU oracle's callers may share, so that both sides see identical bits.

The shapes are those of the networks the paper evaluates (AlexNet and
ResNet-18, Section 4.2) and of its efficiency study (Section 4.1, Fig. 4b-c:
one layer, 14x14 input, channels and filter size varied).  No dataset is
used: activations stand in for post-BatchNorm feature maps (standard normal)
and weights are Gaussian.
"""
from collections import namedtuple

import numpy as np

ConvShape = namedtuple("ConvShape", "name N C_in H W C_out k stride pad w_std")


def _s(name, N, C_in, HW, k, stride, pad, C_out, w_std=1.0):
    return ConvShape(name, N, C_in, HW, HW, C_out, k, stride, pad, w_std)


def out_hw(s):
    return ((s.H + 2 * s.pad - s.k) // s.stride + 1,
            (s.W + 2 * s.pad - s.k) // s.stride + 1)


def macs(s):
    """Nominal 1-bit multiply-accumulates of one layer (all taps counted)."""
    ho, wo = out_hw(s)
    return s.N * ho * wo * s.C_out * s.C_in * s.k * s.k


SINGLE = [_s("single_64x14", 1, 64, 14, 3, 1, 1, 64)]

ALEXNET = [
    _s("alexnet_conv2", 256, 96, 27, 5, 1, 2, 256, 0.01),
    _s("alexnet_conv3", 256, 256, 13, 3, 1, 1, 384, 0.01),
    _s("alexnet_conv4", 256, 384, 13, 3, 1, 1, 384, 0.01),
    _s("alexnet_conv5", 256, 384, 13, 3, 1, 1, 256, 0.01),
]

RESNET18 = [
    _s("resnet_64_56", 256, 64, 56, 3, 1, 1, 64),
    _s("resnet_64_128_s2", 256, 64, 56, 3, 2, 1, 128),
    _s("resnet_128_28", 256, 128, 28, 3, 1, 1, 128),
    _s("resnet_256_14", 256, 256, 14, 3, 1, 1, 256),
    _s("resnet_512_7", 256, 512, 7, 3, 1, 1, 512),
]

SWEEP = [
    _s("sweep_c%d_k%d" % (c, k), 64, c, 14, k, 1, (k - 1) // 2, 256)
    for c in (32, 64, 128, 256, 512, 1024) for k in (1, 3, 5, 7)
]

# The 16 binary 3x3 layers of ResNet-18 after its first (full-precision)
# convolution and max-pool: (C_in, C_out, input H=W, stride).
CHAIN_LAYERS = ([(64, 64, 56, 1)] * 4 + [(64, 128, 56, 2)] + [(128, 128, 28, 1)] * 3 +
                [(128, 256, 28, 2)] + [(256, 256, 14, 1)] * 3 +
                [(256, 512, 14, 2)] + [(512, 512, 7, 1)] * 3)


def chain_shapes(N=256):
    return [_s("chain_%02d" % i, N, ci, hw, 3, st, 1, co, 0.05)
            for i, (ci, co, hw, st) in enumerate(CHAIN_LAYERS)]


CONFIGS = {"single": SINGLE, "alexnet": ALEXNET, "resnet18": RESNET18, "sweep": SWEEP}
CONFIG_INDEX = {"single": 1, "alexnet": 2, "resnet18": 3, "sweep": 4, "chain": 5}


def layer_seed(config, layer_index):
    return 1000 * CONFIG_INDEX[config] + layer_index


def normal(shape, seed, std=1.0):
    """Counter-based (Philox) standard normals scaled by std, as fp32."""
    g = np.random.Generator(np.random.Philox(int(seed)))
    a = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


def make_input(s, seed, n_images=None):
    n = s.N if n_images is None else n_images
    return normal((n, s.C_in, s.H, s.W), seed)


def make_weights(s, seed):
    return normal((s.C_out, s.C_in, s.k, s.k), seed + 500, s.w_std)


def scaled(s, N):
    """Same layer with another batch size."""
    return s._replace(N=N)
