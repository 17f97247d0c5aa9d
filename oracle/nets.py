"""CPU checker, network level (test infrastructure only).

The evaluated networks written as the UNFUSED, UNMERGED layer sequence (Eq. f_map,
Section 3.1; Eq. LR, Section 3.2): every convolution is followed by separate
BatchNorm / Scale / ReLU / LRN / pooling passes, and an inception module is its separate
branch convolutions concatenated.  Each network is a list of ``Step``s at the granularity
at which the slim path stores a tensor, so a test can run it free (each step fed the
checker's own previous outputs) or teacher-forced (each step fed the tensors the GPU
stored).  A step's function never rounds; ``run`` rounds a step's output to bfloat16
exactly where the slim path stores one.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Sequence

import numpy as np

import oracle as O

# Inception-v1 channel table (Cin; c1, c3r, c3, c5r, c5, pp); 3a's 96/128/32/64 -> 256
# are the numbers Section 3.2 prints.  The slim form built here does not use c5r.
_INCEPTION = {
    "3a": (192, 64, 96, 128, 16, 32, 32), "3b": (256, 128, 128, 192, 32, 96, 64),
    "4a": (480, 192, 96, 208, 16, 48, 64), "4b": (512, 160, 112, 224, 24, 64, 64),
    "4c": (512, 128, 128, 256, 24, 64, 64), "4d": (512, 112, 144, 288, 32, 64, 64),
    "4e": (528, 256, 160, 320, 32, 128, 128), "5a": (832, 256, 160, 320, 32, 128, 128),
    "5b": (832, 384, 192, 384, 48, 128, 128),
}
_LRN = dict(size=5, alpha=1e-4, beta=0.75, k=1.0)


@dataclass
class Step:
    name: str                      # tensor this step produces
    src: Sequence[str]             # tensors it reads ("x" = network input)
    fn: Callable[..., np.ndarray]  # unrounded float64 result
    stored_bf16: bool = True       # the slim path stores this tensor in bfloat16
    virtual: bool = False          # pure re-arrangement (concat): no arithmetic of its own


def _p(params, key):
    v = params.get(key)
    return None if v is None else np.asarray(v, np.float64)


def _conv(params, name, x, stride=1, pad=0):
    return O.conv2d(x, _p(params, name + ".w"), _p(params, name + ".b"), stride, pad)


def _conv_bn_scale(params, name, x, stride, pad, eps):
    """conv -> BatchNorm -> Scale as three passes (Eq. Y_batch_scala_conv, read bottom-up)."""
    y = _conv(params, name, x, stride, pad)
    y = O.batchnorm(y, _p(params, name + ".bn.mean"), _p(params, name + ".bn.var"), 1.0, eps)
    return O.scale(y, _p(params, name + ".bn.gamma"), _p(params, name + ".bn.beta"))


def stem_steps(params):
    """Stem slim layer: conv 7x7/2 pad 3 -> ReLU -> max-pool 3x3/2 pad 1 -> LRN."""
    def conv1(x):
        y = O.relu(_conv(params, "conv1", x, 2, 3))
        y, _ = O.maxpool(y, 3, 2, 1)
        return O.lrn(y, **_LRN)
    return [Step("conv1", ["x"], conv1)]


def inception_steps(params, m, src, table=None):
    """Branch-slimmed module: 3x3 path, and the three branches the merged 5x5 replaces.

    Output channel order: [3x3 path | 1x1 branch | 5x5 branch | 3x3 'pool' branch].
    """
    def reduce_(x):
        return O.relu(_conv(params, f"{m}.3x3r", x, 1, 0))

    def three(x):
        return O.relu(_conv(params, f"{m}.3x3", x, 1, 1))

    def merged(x):
        b1 = O.relu(_conv(params, f"{m}.b1", x, 1, 0))
        b5 = O.relu(_conv(params, f"{m}.b5", x, 1, 2))
        bp = O.relu(_conv(params, f"{m}.bp", x, 1, 1))
        return O.concat([b1, b5, bp])

    return [
        Step(f"{m}.3x3r", [src], reduce_),
        Step(f"{m}.3x3", [f"{m}.3x3r"], three),
        Step(f"{m}.m5", [src], merged),
        Step(m, [f"{m}.3x3", f"{m}.m5"], lambda a, b: O.concat([a, b]), virtual=True),
    ]


def googlenet_steps(params, streamline=False):
    """streamline: the stem in the approximate form of Section 3.1 (Method): each pooling layer is removed and its
    stride multiplied into the convolution below it (conv1 7x7/4, conv2 3x3/2), each LRN layer is pruned; the ReLU
    stays.  The inception stages are unchanged."""
    def conv2r(x):
        return O.relu(_conv(params, "conv2r", x, 1, 0))

    def conv2(x):  # conv2/3x3 -> ReLU -> LRN -> pool: the order Section 3.1's example gives
        y = O.lrn(O.relu(_conv(params, "conv2", x, 1, 1)), **_LRN)
        return O.maxpool(y, 3, 2, 1)[0]

    if streamline:
        steps = [Step("conv1", ["x"], lambda x: O.relu(_conv(params, "conv1", x, 4, 3))), Step("conv2r", ["conv1"], conv2r),
                 Step("conv2", ["conv2r"], lambda x: O.relu(_conv(params, "conv2", x, 2, 1)))]
    else:
        steps = stem_steps(params) + [Step("conv2r", ["conv1"], conv2r), Step("conv2", ["conv2r"], conv2)]
    src = "conv2"
    for m in _INCEPTION:
        steps += inception_steps(params, m, src)
        src = m
        if m in ("3b", "4e"):
            name = "pool3" if m == "3b" else "pool4"
            steps.append(Step(name, [src], lambda x: O.maxpool(x, 3, 2, 1)[0]))
            src = name
    steps.append(Step("avgpool", [src], O.avgpool_global))
    steps.append(Step("fc", ["avgpool"], lambda x: _conv(params, "fc", x, 1, 0), stored_bf16=False))
    return steps


def googlenet_streamline_steps(params):
    return googlenet_steps(params, streamline=True)


def googlenet_paper_steps(params):
    """GoogLeNet with the paper's own branch slimming (Section 3.2, Method / Branch Reducing / Tensor-Branch
    Slimming): per module a 1x1 reducer with half the original width feeding a 3x3 convolution of c3 + c1
    outputs, and the original 5x5 reducer feeding a 5x5 convolution of c5 + pp outputs; the two branch
    outputs are concatenated.  Each convolution is followed by its own ReLU pass."""
    def conv2r(x):
        return O.relu(_conv(params, "conv2r", x, 1, 0))

    def conv2(x):
        y = O.lrn(O.relu(_conv(params, "conv2", x, 1, 1)), **_LRN)
        return O.maxpool(y, 3, 2, 1)[0]

    steps = stem_steps(params) + [Step("conv2r", ["conv1"], conv2r), Step("conv2", ["conv2r"], conv2)]
    src = "conv2"
    for m in _INCEPTION:
        steps += [
            Step(f"{m}.p3r", [src], lambda x, m=m: O.relu(_conv(params, f"{m}.p3r", x, 1, 0))),
            Step(f"{m}.p3", [f"{m}.p3r"], lambda x, m=m: O.relu(_conv(params, f"{m}.p3", x, 1, 1))),
            Step(f"{m}.p5r", [src], lambda x, m=m: O.relu(_conv(params, f"{m}.p5r", x, 1, 0))),
            Step(f"{m}.p5", [f"{m}.p5r"], lambda x, m=m: O.relu(_conv(params, f"{m}.p5", x, 1, 2))),
            Step(m, [f"{m}.p3", f"{m}.p5"], lambda a, b: O.concat([a, b]), virtual=True),
        ]
        src = m
        if m in ("3b", "4e"):
            name = "pool3" if m == "3b" else "pool4"
            steps.append(Step(name, [src], lambda x: O.maxpool(x, 3, 2, 1)[0]))
            src = name
    steps.append(Step("avgpool", [src], O.avgpool_global))
    steps.append(Step("fc", ["avgpool"], lambda x: _conv(params, "fc", x, 1, 0), stored_bf16=False))
    return steps


def resnet50_steps(params, eps=1e-5):
    def conv1(x):
        y = O.relu(_conv_bn_scale(params, "conv1", x, 2, 3, eps))
        return O.maxpool(y, 3, 2, 1)[0]

    steps = [Step("conv1", ["x"], conv1)]
    src = "conv1"
    for si, (w, n) in enumerate(((64, 3), (128, 4), (256, 6), (512, 3))):
        for b in range(n):
            blk = f"res{si + 2}{chr(97 + b)}"
            s = 2 if (b == 0 and si > 0) else 1   # stride sits on the first 1x1 and on the projection
            res = src
            if b == 0:
                steps.append(Step(f"{blk}.br1", [src],
                                  lambda x, blk=blk, s=s: _conv_bn_scale(params, f"{blk}.br1", x, s, 0, eps)))
                res = f"{blk}.br1"
            steps.append(Step(f"{blk}.2a", [src],
                              lambda x, blk=blk, s=s: O.relu(_conv_bn_scale(params, f"{blk}.2a", x, s, 0, eps))))
            steps.append(Step(f"{blk}.2b", [f"{blk}.2a"],
                              lambda x, blk=blk: O.relu(_conv_bn_scale(params, f"{blk}.2b", x, 1, 1, eps))))
            steps.append(Step(f"{blk}.2c", [f"{blk}.2b", res],
                              lambda x, r, blk=blk: O.relu(O.add(_conv_bn_scale(params, f"{blk}.2c", x, 1, 0, eps), r))))
            src = f"{blk}.2c"
    steps.append(Step("avgpool", [src], O.avgpool_global))
    steps.append(Step("fc", ["avgpool"], lambda x: _conv(params, "fc", x, 1, 0), stored_bf16=False))
    return steps


# AlexNet, two-tower (grouped) form: (name, stride, pad, groups); LRN after conv1 and conv2, 3x3/2 pooling without
# padding after norm1, norm2 and conv5; fc6 is a 6x6 convolution over the 6x6 plane; dropout is the identity at
# inference; no softmax (logits).
_ALEXNET = (("conv1", 4, 0, 1), ("conv2", 1, 2, 2), ("conv3", 1, 1, 1), ("conv4", 1, 1, 2), ("conv5", 1, 1, 2),
            ("fc6", 1, 0, 1), ("fc7", 1, 0, 1), ("fc8", 1, 0, 1))


def alexnet_steps(params):
    """AlexNet as the unfused layer sequence conv -> ReLU -> LRN -> pool (Section 4.3 slims "the first two
    convolution layers followed by LRN layers": the slim layers are conv1 = conv + ReLU + LRN and conv2 = grouped
    conv + ReLU + LRN).  Pooling: 3x3, stride 2, no padding (227 -> 55 -> 27 -> 13 -> 6)."""
    def gconv(name, stride, pad, groups):
        return lambda x: O.conv2d_grouped(x, _p(params, name + ".w"), _p(params, name + ".b"), stride, pad, groups)

    cfg = {n: (s, p, g) for n, s, p, g in _ALEXNET}
    pool = lambda x: O.maxpool(x, 3, 2, 0)[0]
    steps = [
        Step("conv1", ["x"], lambda x: O.lrn(O.relu(gconv("conv1", *cfg["conv1"])(x)), **_LRN)),
        Step("pool1", ["conv1"], pool),
        Step("conv2", ["pool1"], lambda x: O.lrn(O.relu(gconv("conv2", *cfg["conv2"])(x)), **_LRN)),
        Step("pool2", ["conv2"], pool),
        Step("conv3", ["pool2"], lambda x: O.relu(gconv("conv3", *cfg["conv3"])(x))),
        Step("conv4", ["conv3"], lambda x: O.relu(gconv("conv4", *cfg["conv4"])(x))),
        Step("conv5", ["conv4"], lambda x: O.relu(gconv("conv5", *cfg["conv5"])(x))),
        Step("pool5", ["conv5"], pool),
        Step("fc6", ["pool5"], lambda x: O.relu(gconv("fc6", *cfg["fc6"])(x))),
        Step("fc7", ["fc6"], lambda x: O.relu(gconv("fc7", *cfg["fc7"])(x))),
        Step("fc8", ["fc7"], gconv("fc8", *cfg["fc8"]), stored_bf16=False),
    ]
    return steps


def run(steps, x, given=None, rounding=True):
    """Run a step list.

    Free-running when ``given`` is None: each step reads the checker's own (bfloat16-rounded)
    outputs.  Teacher-forced otherwise: each step reads ``given[name]`` (the tensors another
    implementation stored) for every source it has.  ``rounding=False`` keeps every tensor in
    float64 (used only to pin the composition against an independent float64 library).
    Returns {name: float64 array}.
    """
    out = {"x": np.asarray(x, np.float64)}
    for st in steps:
        ins = [np.asarray(given[s], np.float64) if (given is not None and s in given) else out[s]
               for s in st.src]
        y = st.fn(*ins)
        out[st.name] = O.round_bf16(y) if (rounding and st.stored_bf16 and not st.virtual) else y
    return out
