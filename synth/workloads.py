"""Synthetic workloads shaped like the paper's MNIST / CIFAR10 / ImageNet runs.

All tensors come from ``numpy.random.Generator(PCG64(seed))``.  Draw order inside one
config: input, labels, then the weights layer by layer.  The real datasets are not used
anywhere; uniform int8 tensors of the same shapes stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

GEMM_SWEEP_DIMS = (256, 1024, 4096, 8192)


def uniform_int8(rng: np.random.Generator, shape) -> np.ndarray:
    """int8 uniform over [-127, 127] (the value -128 never appears)."""
    return rng.integers(-127, 128, size=shape, dtype=np.int8)


def gaussian_like_int8(rng: np.random.Generator, shape) -> np.ndarray:
    """Bell-shaped int8 with sigma ~ 32.7, clipped to [-127, 127]; integer-only recipe:
    the sum of 8 uniform bytes (mean 1020, sigma ~ 209) is centred and scaled by 5/32."""
    s = rng.integers(0, 256, size=(8,) + tuple(shape), dtype=np.int64).sum(axis=0)
    v = ((s - 1020) * 5) >> 5
    return np.clip(v, -127, 127).astype(np.int8)


def he_like_exponent(fan_in: int) -> int:
    """Static weight exponent: -(5 + ceil(log2(fan_in) / 2)); gives -10 at fan-in 784."""
    return -(5 + math.ceil(math.log2(fan_in) / 2))


@dataclass
class Net:
    """A feed-forward net: 3x3 stride-1 pad-1 convolutions, 2x2 max-pools, fully connected
    layers.  ``layers`` entries are dicts with key ``op`` in {"conv", "pool", "fc"}."""

    name: str
    batch: int
    in_shape: tuple  # (H, W, C) for conv nets, (K,) for MLPs
    n_classes: int
    s_in: int
    seed: int
    layers: list = field(default_factory=list)
    m_u: int = 5

    def n_weights(self) -> int:
        t = 0
        for L in self.layers:
            if L["op"] == "conv":
                t += L["cout"] * 9 * L["cin"]
            elif L["op"] == "fc":
                t += L["n"] * L["k"]
        return t

    def macs_per_pass(self) -> int:
        """Multiply-accumulates of one forward pass."""
        t = 0
        if len(self.in_shape) == 3:
            h, w, _ = self.in_shape
        for L in self.layers:
            if L["op"] == "conv":
                t += self.batch * h * w * L["cout"] * 9 * L["cin"]
            elif L["op"] == "pool":
                h, w = h // 2, w // 2
            else:
                t += self.batch * L["n"] * L["k"]
        return t

    def int8_ops_per_step(self) -> int:
        """2 * MACs of forward + wgrad for every layer + dgrad for all but the first."""
        t = 0
        first = True
        if len(self.in_shape) == 3:
            h, w, _ = self.in_shape
        for L in self.layers:
            if L["op"] == "conv":
                m = self.batch * h * w * L["cout"] * 9 * L["cin"]
            elif L["op"] == "pool":
                h, w = h // 2, w // 2
                continue
            else:
                m = self.batch * L["n"] * L["k"]
            t += 2 * m * (2 if first else 3)
            first = False
        return t


def _conv_stack(h, w, cin, widths, pools_after, weight_exp=None):
    layers = []
    for i, co in enumerate(widths, start=1):
        s_w = weight_exp if weight_exp is not None else he_like_exponent(9 * cin)
        layers.append({"op": "conv", "cin": cin, "cout": co, "relu": True, "s_w": s_w})
        cin = co
        if i in pools_after:
            layers.append({"op": "pool"})
            h, w = h // 2, w // 2
    return layers, h, w, cin


def _fc(k, n, relu, s_w=None):
    return {"op": "fc", "k": k, "n": n, "relu": relu,
            "s_w": s_w if s_w is not None else he_like_exponent(k)}


def config_net(idx: int, batch: int | None = None, scale: int = 1) -> Net:
    """The five benchmark configurations (index 1 is the GEMM sweep and has no net).

    ``batch`` overrides the batch size; ``scale`` > 1 divides the image side (conv nets)
    so that the oracle can run a shrunken copy of the same architecture."""
    if idx == 0:
        net = Net("mlp_784_256_256_10", batch or 64, (784,), 10, -7, 0)
        net.layers = [_fc(784, 256, True, -10), _fc(256, 256, True, -10), _fc(256, 10, False, -10)]
        return net
    if idx == 2:
        side = 28 // scale
        net = Net("mnist_cnn", batch or 256, (side, side, 1), 10, -7, 2)
        convs, h, w, c = _conv_stack(side, side, 1, [32, 64], {2})
        net.layers = convs + [_fc(h * w * c, 128, True), _fc(128, 10, False)]
        return net
    if idx == 3:
        side = 32 // scale
        net = Net("cifar_vgg11", batch or 256, (side, side, 3), 10, -7, 3)
        convs, h, w, c = _conv_stack(side, side, 3, [64, 128, 256, 256, 512, 512, 512, 512],
                                     {1, 2, 4, 6, 8})
        net.layers = convs + [_fc(h * w * c, 10, False)]
        return net
    if idx == 4:
        side = 224 // scale
        net = Net("imagenet_vgg16", batch or 64, (side, side, 3), 1000, -7, 4)
        convs, h, w, c = _conv_stack(
            side, side, 3, [64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512],
            {2, 4, 7, 10, 13})
        net.layers = convs + [_fc(h * w * c, 4096, True), _fc(4096, 4096, True),
                              _fc(4096, 1000, False)]
        return net
    raise ValueError("config %d has no network" % idx)


def make_net_inputs(net: Net):
    """Returns (x int8, labels int32, [weights int8 ...]) for ``net`` from its seed."""
    rng = np.random.Generator(np.random.PCG64(net.seed))
    x = uniform_int8(rng, (net.batch,) + tuple(net.in_shape))
    labels = rng.integers(0, net.n_classes, size=(net.batch,), dtype=np.int32)
    weights = []
    for L in net.layers:
        if L["op"] == "conv":
            weights.append(uniform_int8(rng, (L["cout"], 3, 3, L["cin"])))
        elif L["op"] == "fc":
            weights.append(uniform_int8(rng, (L["n"], L["k"])))
    return x, labels, weights


def make_step_batch(net: Net, step: int):
    """The mini-batch of training step ``step`` (x int8, labels int32).  Step 0 is the batch of
    ``make_net_inputs``; every later step draws a fresh batch from ``PCG64([seed, step])``."""
    if step == 0:
        rng = np.random.Generator(np.random.PCG64(net.seed))
    else:
        rng = np.random.Generator(np.random.PCG64([net.seed, step]))
    x = uniform_int8(rng, (net.batch,) + tuple(net.in_shape))
    labels = rng.integers(0, net.n_classes, size=(net.batch,), dtype=np.int32)
    return x, labels


def gemm_operands(M: int, N: int, K: int, dist: str = "uniform", seed: int = 1):
    """Operands of the fused-GEMM sweep: a[M,K] and w[N,K] (both K-contiguous)."""
    rng = np.random.Generator(np.random.PCG64([seed, M, N, K, 0 if dist == "uniform" else 1]))
    gen = uniform_int8 if dist == "uniform" else gaussian_like_int8
    return gen(rng, (M, K)), gen(rng, (N, K))


def gemm_grad_operands(M: int, N: int, K: int, dist: str = "uniform", seed: int = 1):
    """Operands of the sweep's gradient variant: e[K,M] and a[K,N]; the product
    g[M,N] = sum_k e[k,m] a[k,n] contracts over the rows of both (a weight-gradient multiply)."""
    rng = np.random.Generator(np.random.PCG64([seed, M, N, K, 2 if dist == "uniform" else 3]))
    gen = uniform_int8 if dist == "uniform" else gaussian_like_int8
    return gen(rng, (K, M)), gen(rng, (K, N))
