"""Seeded synthetic inputs and workload shapes.

This module serves both the CPU oracle's tests and the CUDA path's tests / benchmark.  It holds
none of the method's arithmetic: only shapes, random draws and the value structure of the
paper's workloads (post-ReLU activations, Kaiming-normal weights, small output gradients, rare
outliers).  Every tensor is a pure function of (seed, tensor name, shape); draws come from
numpy's counter-based Philox generator.

Stand-ins: the paper trains ResNets / YOLO models on image datasets and a latent-replay buffer;
none of that data is used here.  The layer shapes follow those workloads and the values follow
the distributions named in each workload below.
"""
from __future__ import annotations

from collections import namedtuple

import numpy as np

ConvDesc = namedtuple("ConvDesc", "N C_in H W C_out Kh Kw stride_h stride_w pad_h pad_w")

# element formats / roles: plain integers shared by name with both sides' own enums
E4M3, E5M2, E2M1, E3M2, E2M3 = 0, 1, 2, 3, 4
ROLE_X, ROLE_W, ROLE_DY = 0, 1, 2

_TENSOR_IDS = {"x": 1, "w": 2, "dy": 3, "outlier": 4}


def conv_desc(N, C_in, H, W, C_out, K, stride=1, pad=None):
    if pad is None:
        pad = K // 2
    return ConvDesc(N, C_in, H, W, C_out, K, K, stride, stride, pad, pad)


def out_hw(d):
    d = ConvDesc(*d)
    return ((d.H + 2 * d.pad_h - d.Kh) // d.stride_h + 1, (d.W + 2 * d.pad_w - d.Kw) // d.stride_w + 1)


def _rng(seed, name, part=0):
    return np.random.Generator(np.random.Philox(key=[int(seed), _TENSOR_IDS[name] + 16 * int(part)]))


_BIG = 1 << 26   # tensors of this many elements or more are drawn slice by slice along their first axis, in parallel


def _draw(seed, name, shape, fn):
    """`fn(generator, shape)` over the whole tensor from one stream, or - for big tensors - over each slice of the
    first axis from a stream of its own (key: seed, tensor name, slice index), drawn by a thread pool.  Either way
    the tensor is a pure function of (seed, name, shape)."""
    n = int(np.prod(shape))
    if n < _BIG or shape[0] < 2:
        return fn(_rng(seed, name), shape)
    from concurrent.futures import ThreadPoolExecutor
    import os

    out = np.empty(shape, dtype=np.float32)

    def one(i):
        out[i] = fn(_rng(seed, name, i + 1), shape[1:])

    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
        list(ex.map(one, range(shape[0])))
    return out


def make_x(d, seed, kind="relu"):
    """Activations, fp32 NCHW.  kind: 'relu' = max(N(0,1),0); 'relu_outliers' = the same with each
    element independently multiplied by 50 with probability 0.01; 'gauss' = N(0,1);
    'uniform' = U[0,1); 'silu' = z*sigmoid(z) with z ~ N(0,1); 'smallint' = integers in {-2..2}."""
    d = ConvDesc(*d)
    shape = (d.N, d.C_in, d.H, d.W)
    if kind == "uniform":
        return _draw(seed, "x", shape, lambda g, s: g.random(s, dtype=np.float32))
    if kind == "smallint":
        return _rng(seed, "x").integers(-2, 3, size=shape).astype(np.float32)
    x = _draw(seed, "x", shape, lambda g, s: g.standard_normal(s, dtype=np.float32))
    if kind == "gauss":
        return x
    if kind == "silu":
        # post-SiLU activations: z * sigmoid(z) of a standard normal pre-activation (small negatives down to -0.278)
        x64 = x.astype(np.float64)
        return (x64 / (1.0 + np.exp(-x64))).astype(np.float32)
    np.maximum(x, 0.0, out=x)
    if kind == "relu_outliers":
        mask = _draw(seed, "outlier", shape, lambda g, s: g.random(s, dtype=np.float32)) < 0.01
        x[mask] *= 50.0
    elif kind != "relu":
        raise ValueError(kind)
    return x


def make_w(d, seed, kind="kaiming"):
    """Weights, fp32 OIHW.  'kaiming' = N(0, 2/(C_in*Kh*Kw)); 'smallint' = integers in {-2..2}."""
    d = ConvDesc(*d)
    shape = (d.C_out, d.C_in, d.Kh, d.Kw)
    g = _rng(seed, "w")
    if kind == "smallint":
        return g.integers(-2, 3, size=shape).astype(np.float32)
    w = g.standard_normal(shape, dtype=np.float32)
    w *= np.float32(np.sqrt(2.0 / (d.C_in * d.Kh * d.Kw)))
    return w


def make_dy(d, seed, kind="small", sigma=1e-3):
    """Output gradient, fp32 [N, C_out, Ho, Wo].  'small' = N(0, sigma^2); 'gauss' = N(0,1);
    'smallint' = integers in {-2..2}."""
    d = ConvDesc(*d)
    ho, wo = out_hw(d)
    shape = (d.N, d.C_out, ho, wo)
    if kind == "smallint":
        return _rng(seed, "dy").integers(-2, 3, size=shape).astype(np.float32)
    y = _draw(seed, "dy", shape, lambda g, s: g.standard_normal(s, dtype=np.float32))
    if kind == "small":
        y *= np.float32(sigma)
    return y


# --------------------------------------------------------------------------------------------
# Workloads.  A workload is a list of layers; a layer names its shape, the element format of
# each tensor and the value distribution of each tensor.
Layer = namedtuple("Layer", "name desc fmt_x fmt_w fmt_dy x_kind w_kind dy_kind seed")


def config1():
    """Small single 3x3 conv: N=8, 32->64 channels, 32x32, MXFP8 (E4M3 X/W, E5M2 dY), seed 0."""
    return [Layer("cfg1_3x3", conv_desc(8, 32, 32, 32, 64, 3), E4M3, E4M3, E5M2, "relu", "kaiming", "small", 0)]


def config2():
    """Single 3x3 conv: N=32, 64->128 channels, 80x80, activations with 1% x50 outliers, MXFP4."""
    return [Layer("cfg2_3x3", conv_desc(32, 64, 80, 80, 128, 3), E2M1, E2M1, E2M1, "relu_outliers", "kaiming", "small", 1)]


def config3(batch=16, image=640):
    """Backbone-shaped conv stack (nano-width detector backbone: stride-2 3x3 convs widening
    16->32->64->128->256, each followed by a split/bottleneck/concat stage of 1x1 and 3x3
    stride-1 convs).  The 3->16 stem is not an MX layer; the 24 convs after it are.  Each layer
    is exercised with its own synthetic input of the right shape (post-SiLU activations: z*sigmoid(z) of a
    standard normal z, which keeps the small negatives down to -0.278); MXFP8 E4M3 forward tensors, E5M2 gradients."""
    layers = []
    res = image // 2  # after the stem
    seed = 200

    def add(name, cin, cout, k, s, r):
        nonlocal seed
        layers.append(Layer(name, conv_desc(batch, cin, r, r, cout, k, s), E4M3, E4M3, E5M2, "silu", "kaiming", "small", seed))
        seed += 1

    c = 16
    for stage, (cout, nb) in enumerate([(32, 1), (64, 2), (128, 2), (256, 1)]):
        add(f"s{stage}_down", c, cout, 3, 2, res)
        res //= 2
        c = cout
        add(f"s{stage}_cv1", c, c, 1, 1, res)
        for b in range(nb):
            add(f"s{stage}_b{b}_a", c // 2, c // 2, 3, 1, res)
            add(f"s{stage}_b{b}_b", c // 2, c // 2, 3, 1, res)
        add(f"s{stage}_cv2", (2 + nb) * c // 2, c, 1, 1, res)
    return layers


def config4():
    """Latent-replay backward workload: stored activations N=256, C=512, 14x14 (max(N(0,1),0)),
    kept only as MXFP4; 3x3 (pad 1) and 1x1 convs 512->512."""
    return [
        Layer("cfg4_3x3", conv_desc(256, 512, 14, 14, 512, 3), E2M1, E2M1, E2M1, "relu", "kaiming", "small", 3),
        Layer("cfg4_1x1", conv_desc(256, 512, 14, 14, 512, 1), E2M1, E2M1, E2M1, "relu", "kaiming", "small", 3),
    ]


def config5(channels=(64, 128, 256, 512), sizes=(14, 28, 56), N=256):
    """Throughput sweep: 3x3 and 1x1, stride 1 and 2, C_in = C_out, Gaussian tensors, MXFP8 E4M3
    and MXFP4 E2M1."""
    layers = []
    for fmt, fname in ((E4M3, "e4m3"), (E2M1, "e2m1")):
        for k in (3, 1):
            for s in (1, 2):
                for c in channels:
                    for hw in sizes:
                        seed = 5000 + fmt * 1000 + k * 100 + s * 50 + (c // 64) * 4 + hw // 14
                        layers.append(Layer(f"cfg5_{fname}_k{k}s{s}_c{c}_hw{hw}", conv_desc(N, c, hw, hw, c, k, s),
                                            fmt, fmt, fmt, "gauss", "kaiming", "gauss", seed))
    return layers


def fp6_layers(N=256):
    """Two mid-size 3x3 layers in the 6-bit element formats: E3M2 activations with E4M3 weights and E5M2 gradients
    (the MicroQonv+ mix), and E2M3 everywhere (the "-6" variant); Gaussian tensors as in the sweep."""
    return [
        Layer("fp6_e3m2act_k3s1_c256_hw28", conv_desc(N, 256, 28, 28, 256, 3), E3M2, E4M3, E5M2, "gauss", "kaiming", "gauss", 6001),
        Layer("fp6_e2m3_k3s1_c256_hw28", conv_desc(N, 256, 28, 28, 256, 3), E2M3, E2M3, E2M3, "gauss", "kaiming", "gauss", 6002),
    ]


CONFIGS = {"config1": config1, "config2": config2, "config3": config3, "config4": config4, "config5": config5}


def layer_tensors(layer):
    """(X, W, dY) fp32 numpy arrays for a layer."""
    return (make_x(layer.desc, layer.seed, layer.x_kind), make_w(layer.desc, layer.seed, layer.w_kind),
            make_dy(layer.desc, layer.seed, layer.dy_kind))
