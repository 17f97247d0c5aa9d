"""Random parameter sets shaped like the two evaluated networks (data generation only).

Names are plain dictionary keys; the topology code that consumes them lives with each
consumer.  All arrays are float32 holding bfloat16-representable values.

GoogLeNet (branch-slimmed form): per inception module ``m`` with Inception-v1 channels
(Cin; c1, c3r, c3, c5r, c5, pp) the parameters are the 3x3 path ``m.3x3r`` (1x1, Cin->c3r)
and ``m.3x3`` (3x3, c3r->c3), and the three branches that the merged 5x5 convolution
replaces, each acting directly on the module input: ``m.b1`` (1x1, Cin->c1), ``m.b5``
(5x5, Cin->c5) and ``m.bp`` (3x3, Cin->pp).  He-normal with the fan-in of each filter's own
size; biases N(0, 0.01).

ResNet-50 (bottleneck v1): every convolution has no bias and is followed by BatchNorm
(mean N(0,0.1), variance U(0.5,1.5), scale factor m = 1) and Scale (gamma U(0.5,1.5),
beta N(0,0.1)).
"""
from __future__ import annotations

import numpy as np

from . import ALEXNET_CONVS, INCEPTION_V1, RESNET50_STAGES, he_normal, normal, uniform


def conv_params(seed, name, cout, k, cin, bias=True):
    p = {f"{name}.w": he_normal(seed, f"{name}.w", cout, k, cin)}
    if bias:
        p[f"{name}.b"] = normal(seed, f"{name}.b", (cout,), std=0.01)
    return p


def bn_params(seed, name, c):
    return {
        f"{name}.mean": normal(seed, f"{name}.mean", (c,), std=0.1),
        f"{name}.var": uniform(seed, f"{name}.var", (c,), 0.5, 1.5),
        f"{name}.gamma": uniform(seed, f"{name}.gamma", (c,), 0.5, 1.5),
        f"{name}.beta": normal(seed, f"{name}.beta", (c,), std=0.1),
    }


def inception_params(seed, m, table=None):
    cin, c1, c3r, c3, _c5r, c5, pp = (table or INCEPTION_V1)[m]
    p = {}
    p.update(conv_params(seed, f"{m}.3x3r", c3r, 1, cin))
    p.update(conv_params(seed, f"{m}.3x3", c3, 3, c3r))
    p.update(conv_params(seed, f"{m}.b1", c1, 1, cin))
    p.update(conv_params(seed, f"{m}.b5", c5, 5, cin))
    p.update(conv_params(seed, f"{m}.bp", pp, 3, cin))
    return p


def googlenet_params(seed=0):
    p = {}
    p.update(conv_params(seed, "conv1", 64, 7, 3))
    p.update(conv_params(seed, "conv2r", 64, 1, 64))
    p.update(conv_params(seed, "conv2", 192, 3, 64))
    for m in INCEPTION_V1:
        p.update(inception_params(seed, m))
    p.update(conv_params(seed, "fc", 1000, 1, 1024))
    return p


def googlenet_paper_params(seed=0):
    """GoogLeNet slimmed the paper's way: per module 1x1 (Cin -> c3r/2), 3x3 (-> c3+c1), 1x1 (Cin -> c5r),
    5x5 (-> c5+pp); stem and classifier as in googlenet_params."""
    p = {}
    p.update(conv_params(seed, "conv1", 64, 7, 3))
    p.update(conv_params(seed, "conv2r", 64, 1, 64))
    p.update(conv_params(seed, "conv2", 192, 3, 64))
    for m, (cin, c1, c3r, c3, c5r, c5, pp) in INCEPTION_V1.items():
        p.update(conv_params(seed, f"{m}.p3r", c3r // 2, 1, cin))
        p.update(conv_params(seed, f"{m}.p3", c3 + c1, 3, c3r // 2))
        p.update(conv_params(seed, f"{m}.p5r", c5r, 1, cin))
        p.update(conv_params(seed, f"{m}.p5", c5 + pp, 5, c5r))
    p.update(conv_params(seed, "fc", 1000, 1, 1024))
    return p


def resnet50_conv_names():
    """(name, Cout, k, Cin) of every convolution, in execution order."""
    out = [("conv1", 64, 7, 3)]
    cin = 64
    for si, (w, n) in enumerate(RESNET50_STAGES):
        for b in range(n):
            blk = f"res{si + 2}{chr(97 + b)}"
            if b == 0:
                out.append((f"{blk}.br1", 4 * w, 1, cin))
            out.append((f"{blk}.2a", w, 1, cin))
            out.append((f"{blk}.2b", w, 3, w))
            out.append((f"{blk}.2c", 4 * w, 1, w))
            cin = 4 * w
    return out


def resnet50_params(seed=0):
    p = {}
    for name, cout, k, cin in resnet50_conv_names():
        p.update(conv_params(seed, name, cout, k, cin, bias=False))
        p.update(bn_params(seed, f"{name}.bn", cout))
    p.update(conv_params(seed, "fc", 1000, 1, 2048))
    return p


def alexnet_params(seed=0):
    """AlexNet: grouped filters are stored per group, [Cout][k][k][Cin / groups]; He-normal on that fan-in."""
    p = {}
    for name, cout, k, _s, _p, groups, cin in ALEXNET_CONVS:
        p.update(conv_params(seed, name, cout, k, cin // groups))
    return p


def images(seed, batch, h=224, w=224, c=3, name="x"):
    """N(0,1) input images [B,H,W,C]; entry n depends only on (seed, n)."""
    return np.stack([normal(seed, f"{name}[{n}]", (h, w, c)) for n in range(batch)])
