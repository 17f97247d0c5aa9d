"""CPU checker (test infrastructure only): one step of the layer-wise regression that re-learns a slim layer.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; the CUDA library never
does.  Everything is float64 numpy; tensors are NHWC, filters ``[Cout][k][k][Cin]``.

What it follows (Section 3.1, "Theoretical analysis"): the slim layer f~(W, b; X) is a single convolution (with
the ReLU the method keeps) that has to reproduce the feature map Y_CNN the original layer group made from the same
input X, and Eq. (w_b) / Lemma 1 fit it by stochastic gradient descent on

    sum_i || Y_CNN^i - f~(W, b; X^i) ||_F^2 .

Readings the paper leaves open, taken here:
  * the constant in front of the sum: 1 / (2 B) for a mini-batch of B images (the Euclidean loss of the framework
    the paper uses); the minimiser does not depend on it;
  * "SGD": v <- momentum * v + lr * (grad + decay * W);  W <- W - v  (the same framework's update; momentum = 0
    and decay = 0 give the plain rule); the bias takes no weight decay.
"""
from __future__ import annotations

import numpy as np

import oracle as O


def slim_forward(x, w, b, stride=1, pad=0, relu=True):
    """f~(W, b; X): the convolution of Eq. (y_i = Y_com), followed by the ReLU the method keeps."""
    z = O.conv2d(x, w, b, stride, pad)
    return np.maximum(z, 0.0) if relu else z


def regression_loss(y, yt, batch=None):
    """1/(2B) * sum_i ||Y_CNN^i - Y^i||_F^2 (Eq. (w_b) with the constant of the reading above).

    `batch`: the B of the constant when y holds only some of the mini-batch's samples (a shard of a data-parallel
    step): the objective is a sum over samples, so the shards' values add up to the mini-batch's."""
    d = np.asarray(y, np.float64) - np.asarray(yt, np.float64)
    return float(np.sum(d * d) / (2.0 * (batch or y.shape[0])))


def grad_preactivation(y, yt, relu=True, batch=None):
    """dL/dZ for Y = ReLU(Z): (Y - Y_CNN) / B where the unit is active (Y > 0), zero elsewhere (`batch` as above)."""
    y = np.asarray(y, np.float64)
    g = (y - np.asarray(yt, np.float64)) / (batch or y.shape[0])
    return np.where(y > 0.0, g, 0.0) if relu else g


def shard_gradients(x, yt, w, b, batch, stride=1, pad=0, relu=True):
    """What one rank of a data-parallel step contributes from its shard (x, yt) of a mini-batch of `batch` samples:
    (dW, db, loss), each a sum over the shard's samples with the mini-batch's constant.  Eq. (w_b) sums over samples, so
    adding these over a partition of the mini-batch gives the gradient and loss of the whole of it."""
    y = slim_forward(x, w, b, stride, pad, relu)
    dz = grad_preactivation(y, yt, relu, batch)
    return conv2d_wgrad(x, dz, w.shape[1], stride, pad), bias_grad(dz), regression_loss(y, yt, batch)


def conv2d_wgrad(x, dz, k, stride=1, pad=0):
    """dL/dW[j, r, s, c] = sum over (n, ho, wo) of dZ[n, ho, wo, j] * x[n, ho*stride - pad + r, wo*stride - pad + s, c],
    the derivative of y = conv(x; W) with zero padding with respect to each filter tap."""
    x = np.asarray(x, np.float64)
    dz = np.asarray(dz, np.float64)
    B, H, W, C = x.shape
    _, Ho, Wo, Cout = dz.shape
    xp = np.zeros((B, H + 2 * pad, W + 2 * pad, C), np.float64)
    xp[:, pad:pad + H, pad:pad + W, :] = x
    dw = np.empty((Cout, k, k, C), np.float64)
    for r in range(k):
        for s in range(k):
            patch = xp[:, r:r + stride * (Ho - 1) + 1:stride, s:s + stride * (Wo - 1) + 1:stride, :]
            dw[:, r, s, :] = np.tensordot(dz, patch, axes=([0, 1, 2], [0, 1, 2]))
    return dw


def bias_grad(dz):
    """dL/db[j] = sum over (n, ho, wo) of dZ[n, ho, wo, j]."""
    return np.asarray(dz, np.float64).sum(axis=(0, 1, 2))


def sgd_update(w, v, g, lr, momentum=0.0, decay=0.0):
    """v <- momentum * v + lr * (g + decay * w);  w <- w - v.  Returns (w, v)."""
    v = momentum * np.asarray(v, np.float64) + lr * (np.asarray(g, np.float64) + decay * np.asarray(w, np.float64))
    return np.asarray(w, np.float64) - v, v


def regression_step(x, yt, w, b, vw, vb, lr, momentum=0.0, decay=0.0, stride=1, pad=0, relu=True):
    """One SGD step of Eq. (w_b) on a mini-batch (X, Y_CNN).  Returns (w, b, vw, vb, loss before the step, dW, db)."""
    k = w.shape[1]
    y = slim_forward(x, w, b, stride, pad, relu)
    loss = regression_loss(y, yt)
    dz = grad_preactivation(y, yt, relu)
    dw = conv2d_wgrad(x, dz, k, stride, pad)
    db = bias_grad(dz)
    w2, vw2 = sgd_update(w, vw, dw, lr, momentum, decay)
    b2, vb2 = sgd_update(b, vb, db, lr, momentum, 0.0)      # no weight decay on the bias
    return w2, b2, vw2, vb2, loss, dw, db
