"""Pins of the layer-wise regression oracle (Eq. (w_b), Lemma 1): finite differences, a library second opinion,
the linear least-squares closed form, the BatchNorm fold as a zero-loss point, and hand-worked update arithmetic."""
import numpy as np
import pytest

import oracle as O
import oracle.finetune as F


def rng(seed):
    return np.random.default_rng(seed)


def problem(seed, B=2, H=6, W=5, C=3, Cout=4, k=3, stride=1, pad=1):
    r = rng(seed)
    x = r.normal(size=(B, H, W, C))
    w = r.normal(size=(Cout, k, k, C)) * 0.4
    b = r.normal(size=Cout) * 0.1
    Ho, Wo = O.out_size(H, k, stride, pad), O.out_size(W, k, stride, pad)
    yt = np.abs(r.normal(size=(B, Ho, Wo, Cout)))
    return x, w, b, yt


@pytest.mark.parametrize("k,stride,pad,relu", [(3, 1, 1, True), (3, 2, 1, True), (5, 1, 2, False), (1, 1, 0, True), (2, 2, 0, True)])
def test_gradients_match_central_differences(k, stride, pad, relu):
    x, w, b, yt = problem(k * 10 + stride, k=k, stride=stride, pad=pad)
    loss = lambda w_, b_: F.regression_loss(F.slim_forward(x, w_, b_, stride, pad, relu), yt)
    y = F.slim_forward(x, w, b, stride, pad, relu)
    dz = F.grad_preactivation(y, yt, relu)
    dw, db = F.conv2d_wgrad(x, dz, k, stride, pad), F.bias_grad(dz)
    h = 1e-6
    r = rng(7)
    for _ in range(24):
        idx = tuple(int(r.integers(0, n)) for n in w.shape)
        e = np.zeros_like(w); e[idx] = h
        fd = (loss(w + e, b) - loss(w - e, b)) / (2 * h)
        assert abs(fd - dw[idx]) <= 1e-6 * max(1.0, abs(fd)), (idx, fd, dw[idx])
    for j in range(w.shape[0]):
        e = np.zeros_like(b); e[j] = h
        fd = (loss(w, b + e) - loss(w, b - e)) / (2 * h)
        assert abs(fd - db[j]) <= 1e-6 * max(1.0, abs(fd))


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (5, 1, 2), (7, 2, 3)])
def test_gradients_vs_torch_autograd(k, stride, pad):
    torch = pytest.importorskip("torch")
    x, w, b, yt = problem(100 + k, B=3, H=9, W=8, C=5, Cout=6, k=k, stride=stride, pad=pad)
    tw = torch.tensor(w.transpose(0, 3, 1, 2).copy(), dtype=torch.float64, requires_grad=True)
    tb = torch.tensor(b, dtype=torch.float64, requires_grad=True)
    tx = torch.tensor(x.transpose(0, 3, 1, 2).copy(), dtype=torch.float64)
    ty = torch.relu(torch.nn.functional.conv2d(tx, tw, tb, stride=stride, padding=pad))
    tl = ((ty - torch.tensor(yt.transpose(0, 3, 1, 2).copy())) ** 2).sum() / (2 * x.shape[0])
    tl.backward()
    y = F.slim_forward(x, w, b, stride, pad)
    assert abs(F.regression_loss(y, yt) - tl.item()) <= 1e-12 * abs(tl.item())
    dz = F.grad_preactivation(y, yt)
    np.testing.assert_allclose(F.conv2d_wgrad(x, dz, k, stride, pad), tw.grad.numpy().transpose(0, 2, 3, 1), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(F.bias_grad(dz), tb.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_linear_case_is_least_squares():
    """1x1 convolution without ReLU: Eq. (w_b) is linear least squares.  The gradient is X^T (X W - Y) / B and it
    vanishes at the solution of the normal equations."""
    r = rng(3)
    B, H, W, C, Cout = 2, 4, 4, 5, 3
    x = r.normal(size=(B, H, W, C))
    yt = r.normal(size=(B, H, W, Cout))
    X = np.concatenate([x.reshape(-1, C), np.ones((B * H * W, 1))], axis=1)          # bias as a constant column
    sol, *_ = np.linalg.lstsq(X, yt.reshape(-1, Cout), rcond=None)
    w_star, b_star = sol[:C].T.reshape(Cout, 1, 1, C), sol[C]
    y = F.slim_forward(x, w_star, b_star, relu=False)
    dz = F.grad_preactivation(y, yt, relu=False)
    assert np.abs(F.conv2d_wgrad(x, dz, 1)).max() < 1e-12 and np.abs(F.bias_grad(dz)).max() < 1e-12
    w = r.normal(size=(Cout, 1, 1, C)); b = r.normal(size=Cout)
    y = F.slim_forward(x, w, b, relu=False)
    dz = F.grad_preactivation(y, yt, relu=False)
    G = X.T @ (X @ np.concatenate([w.reshape(Cout, C).T, b[None]], axis=0) - yt.reshape(-1, Cout)) / B
    np.testing.assert_allclose(F.conv2d_wgrad(x, dz, 1).reshape(Cout, C), G[:C].T, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(F.bias_grad(dz), G[C], rtol=1e-12, atol=1e-13)
    assert F.regression_loss(F.slim_forward(x, w_star, b_star, relu=False), yt) <= F.regression_loss(y, yt)


def test_folded_batchnorm_is_a_zero_loss_point():
    """The feature map of conv -> BatchNorm -> Scale -> ReLU is reproduced exactly by the folded convolution (Lemma 2),
    so the regression of Eq. (w_b) has loss 0 and zero gradient there."""
    r = rng(5)
    x = r.normal(size=(2, 6, 6, 4))
    w = r.normal(size=(5, 3, 3, 4)) * 0.3
    b = r.normal(size=5) * 0.1
    mu, var = r.normal(size=5) * 0.1, r.uniform(0.5, 1.5, size=5)
    gamma, beta = r.uniform(0.5, 1.5, size=5), r.normal(size=5) * 0.1
    teacher = O.relu(O.scale(O.batchnorm(O.conv2d(x, w, b, 1, 1), mu, var, 1.0, 1e-5), gamma, beta))
    wf, bf = O.fold_bn(w, b, mu, var, 1.0, 1e-5, gamma, beta)
    y = F.slim_forward(x, wf, bf, 1, 1)
    assert F.regression_loss(y, teacher) < 1e-24
    dz = F.grad_preactivation(y, teacher)
    assert np.abs(F.conv2d_wgrad(x, dz, 3, 1, 1)).max() < 1e-12


def test_wgrad_special_cases():
    # all-ones input and gradient: every tap sums the number of output positions whose tap lands inside the image
    B, H, W, C, Cout, k, pad = 1, 5, 4, 2, 3, 3, 1
    dw = F.conv2d_wgrad(np.ones((B, H, W, C)), np.ones((B, H, W, Cout)), k, 1, pad)
    rows = [sum(0 <= ho - pad + r < H for ho in range(H)) for r in range(k)]
    cols = [sum(0 <= wo - pad + s < W for wo in range(W)) for s in range(k)]
    for r_ in range(k):
        for s_ in range(k):
            assert np.all(dw[:, r_, s_, :] == rows[r_] * cols[s_])
    # a single non-zero gradient element picks out the input patch under it
    x = rng(9).normal(size=(1, 5, 5, 2))
    dz = np.zeros((1, 3, 3, 1)); dz[0, 1, 2, 0] = 2.0
    dw = F.conv2d_wgrad(x, dz, 3, 2, 1)                  # stride 2, pad 1: output (1, 2) sees rows 1..3, cols 3..5
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    np.testing.assert_array_equal(dw[0], 2.0 * xp[0, 2:5, 4:7, :])


def test_relu_mask_and_scale():
    y = np.array([[[[0.0, 2.0, 1.0]]], [[[3.0, 0.0, 1.0]]]])
    yt = np.array([[[[1.0, 1.0, 1.0]]], [[[1.0, 5.0, 0.0]]]])
    g = F.grad_preactivation(y, yt)
    np.testing.assert_array_equal(g, np.array([[[[0.0, 0.5, 0.0]]], [[[1.0, 0.0, 0.5]]]]))
    assert F.regression_loss(y, yt) == (1 + 1 + 0 + 4 + 25 + 1) / 4.0
    np.testing.assert_array_equal(F.grad_preactivation(y, yt, relu=False)[0, 0, 0], [-0.5, 0.5, 0.0])


def test_sgd_update_by_hand():
    w, v = np.array([1.0, -2.0]), np.zeros(2)
    w, v = F.sgd_update(w, v, np.array([0.5, 1.0]), lr=0.1, momentum=0.9, decay=0.0)
    np.testing.assert_allclose(v, [0.05, 0.1]); np.testing.assert_allclose(w, [0.95, -2.1])
    w, v = F.sgd_update(w, v, np.array([1.0, 0.0]), lr=0.1, momentum=0.9, decay=0.0)
    np.testing.assert_allclose(v, [0.145, 0.09]); np.testing.assert_allclose(w, [0.805, -2.19])
    w, v = F.sgd_update(np.array([2.0]), np.array([0.0]), np.array([0.0]), lr=0.5, momentum=0.0, decay=0.1)
    np.testing.assert_allclose(w, [1.9])                 # decay alone: w - lr * decay * w


def test_steps_recover_a_realisable_teacher():
    """Lemma 1 in the small: a 1x1 teacher layer is re-learned from (X, Y) pairs by repeated steps."""
    r = rng(11)
    x = r.normal(size=(4, 5, 5, 3))
    wt, bt = r.normal(size=(2, 1, 1, 3)), np.array([0.3, -0.2])
    yt = F.slim_forward(x, wt, bt, relu=False)
    w, b = np.zeros_like(wt), np.zeros(2)
    vw, vb = np.zeros_like(w), np.zeros(2)
    losses = []
    for _ in range(600):
        w, b, vw, vb, loss, _, _ = F.regression_step(x, yt, w, b, vw, vb, lr=0.05, momentum=0.0, relu=False)
        losses.append(loss)
    assert losses[-1] < 1e-10 * losses[0] and all(b_ <= a_ for a_, b_ in zip(losses[5:], losses[6:]) if a_ > 1e-20 * losses[0])
    np.testing.assert_allclose(w, wt, atol=1e-5); np.testing.assert_allclose(b, bt, atol=1e-5)


def test_shard_gradients_add_up_to_the_mini_batch_gradient():
    """Eq. (w_b) is a sum over samples: gradients and loss of any partition of the mini-batch, each taken with the
    mini-batch's 1/B, add up to the whole step's (uneven shards, stride 2, ReLU)."""
    rng = np.random.default_rng(11)
    B, H, Cin, Cout, k, s, p = 5, 7, 3, 4, 3, 2, 1
    x = rng.normal(size=(B, H, H, Cin)); w = rng.normal(size=(Cout, k, k, Cin)) * 0.3; b = rng.normal(size=Cout) * 0.1
    Ho = (H + 2 * p - k) // s + 1
    yt = np.abs(rng.normal(size=(B, Ho, Ho, Cout)))
    _, _, _, _, loss, dw, db = F.regression_step(x, yt, w, b, np.zeros_like(w), np.zeros_like(b), 0.1, 0.0, 0.0, s, p)
    parts = [F.shard_gradients(x[a:e], yt[a:e], w, b, B, s, p) for a, e in ((0, 2), (2, 3), (3, 5))]
    assert np.allclose(sum(q[0] for q in parts), dw, rtol=0, atol=1e-12)
    assert np.allclose(sum(q[1] for q in parts), db, rtol=0, atol=1e-12)
    assert abs(sum(q[2] for q in parts) - loss) < 1e-12
    # a shard taken as a mini-batch of its own differs by the ratio of the batch sizes
    own = F.regression_step(x[:2], yt[:2], w, b, np.zeros_like(w), np.zeros_like(b), 0.1, 0.0, 0.0, s, p)
    assert np.allclose(parts[0][0] * (B / 2), own[5], atol=1e-12)
