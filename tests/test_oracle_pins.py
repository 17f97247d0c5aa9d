"""Pins of the CPU checker against what the paper and the mathematics fix.

Nothing here touches the CUDA library.  Each group is chosen so that a plausible mistake
in the checker (a dropped term, a wrong sign or index, a transposed operand, a wrong
window alignment) fails at least one assertion.
"""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle as O
import oracle.nets as N
import dr_synth as S
import dr_synth.params as P

rng = np.random.default_rng(1234)


def nhwc_to_torch(x):
    return torch.from_numpy(np.ascontiguousarray(np.transpose(x, (0, 3, 1, 2))))


def torch_to_nhwc(t):
    return np.transpose(t.numpy(), (0, 2, 3, 1))


def w_to_torch(w):  # [Cout][k][k][Cin] -> [Cout][Cin][k][k]
    return torch.from_numpy(np.ascontiguousarray(np.transpose(w, (0, 3, 1, 2))))


# ----------------------------------------------------------------------------- conv
@pytest.mark.parametrize("n,k,s,p", [(224, 7, 2, 3), (112, 3, 2, 1), (56, 3, 2, 1), (28, 5, 1, 2),
                                     (28, 3, 2, 1), (14, 3, 2, 1), (56, 1, 2, 0), (64, 7, 2, 3)])
def test_out_size_formula(n, k, s, p):
    assert O.out_size(n, k, s, p) == (n + 2 * p - k) // s + 1


def test_out_size_chain_of_the_networks():
    # 224 -> 112 (7x7/2 pad 3) -> 56 -> 28 -> 14 -> 7 (3x3/2 pad 1 pools), and 64 -> 32 -> 16
    n = O.out_size(224, 7, 2, 3)
    chain = [n]
    for _ in range(4):
        n = O.out_size(n, 3, 2, 1)
        chain.append(n)
    assert chain == [112, 56, 28, 14, 7]
    assert O.out_size(O.out_size(64, 7, 2, 3), 3, 2, 1) == 16


def test_conv_identity_1x1():
    x = rng.standard_normal((2, 5, 4, 6))
    w = np.eye(6).reshape(6, 1, 1, 6)
    assert np.array_equal(O.conv2d(x, w), x)


@pytest.mark.parametrize("k,s,p", [(7, 2, 3), (5, 1, 2), (3, 1, 1), (3, 2, 1), (1, 1, 0)])
def test_conv_all_ones_counts_in_bounds_taps(k, s, p):
    H, W, Cin = 13, 11, 3
    y = O.conv2d(np.ones((1, H, W, Cin)), np.ones((2, k, k, Cin)), None, s, p)
    Ho, Wo = y.shape[1:3]
    for ho, wo in itertools.product(range(Ho), range(Wo)):
        nh = sum(0 <= ho * s - p + r < H for r in range(k))
        nw = sum(0 <= wo * s - p + t < W for t in range(k))
        assert y[0, ho, wo, 0] == nh * nw * Cin
    if (k, s, p) == (7, 2, 3):
        assert y[0, 0, 0, 0] == 16 * Cin      # corner of 7x7 pad 3: 4x4 taps in bounds
    if (k, s, p) == (5, 1, 2):
        assert y[0, 0, 0, 0] == 9 * Cin       # corner of 5x5 pad 2: 3x3 taps in bounds


def test_conv_single_tap_picks_the_right_neighbour():
    # A filter that is 1 at tap (r,s) and channel c only shifts the input: catches swapped
    # r/s, a wrong pad sign and transposed filter indices.
    H, W, Cin = 6, 7, 3
    x = rng.standard_normal((1, H, W, Cin))
    for r, s, c in [(0, 2, 1), (2, 0, 0), (1, 1, 2), (0, 0, 0), (2, 1, 1)]:
        w = np.zeros((1, 3, 3, Cin)); w[0, r, s, c] = 1.0
        y = O.conv2d(x, w, None, 1, 1)
        for ho, wo in itertools.product(range(H), range(W)):
            hi, wi = ho - 1 + r, wo - 1 + s
            exp = x[0, hi, wi, c] if (0 <= hi < H and 0 <= wi < W) else 0.0
            assert y[0, ho, wo, 0] == exp


def test_conv_linearity_and_bias():
    x1, x2 = rng.standard_normal((2, 1, 6, 6, 4))
    w = rng.standard_normal((5, 3, 3, 4)); b = rng.standard_normal(5)
    y = O.conv2d(2.0 * x1 - 3.0 * x2, w, None, 1, 1)
    np.testing.assert_allclose(y, 2 * O.conv2d(x1, w, None, 1, 1) - 3 * O.conv2d(x2, w, None, 1, 1), atol=1e-12)
    np.testing.assert_allclose(O.conv2d(x1, w, b, 1, 1) - O.conv2d(x1, w, None, 1, 1),
                               np.broadcast_to(b, (1, 6, 6, 5)), atol=1e-13)


def brute_conv(x, w, b, s, p):
    B, H, W, Cin = x.shape; Cout, k = w.shape[0], w.shape[1]
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    xp = np.zeros((B, H + 2 * p, W + 2 * p, Cin)); xp[:, p:p + H, p:p + W] = x
    y = np.zeros((B, Ho, Wo, Cout))
    for n, ho, wo, j in itertools.product(range(B), range(Ho), range(Wo), range(Cout)):
        y[n, ho, wo, j] = (xp[n, ho * s:ho * s + k, wo * s:wo * s + k, :] * w[j]).sum() + (b[j] if b is not None else 0)
    return y


@pytest.mark.parametrize("k,s,p,H,W", [(7, 2, 3, 9, 10), (5, 1, 2, 6, 5), (3, 1, 1, 5, 7), (1, 2, 0, 7, 6), (3, 2, 1, 8, 8)])
def test_conv_vs_brute_force_and_torch(k, s, p, H, W):
    x = rng.standard_normal((2, H, W, 3)); w = rng.standard_normal((4, k, k, 3)); b = rng.standard_normal(4)
    y = O.conv2d(x, w, b, s, p)
    np.testing.assert_allclose(y, brute_conv(x, w, b, s, p), atol=1e-12)
    t = F.conv2d(nhwc_to_torch(x), w_to_torch(w), torch.from_numpy(b), stride=s, padding=p)
    np.testing.assert_allclose(y, torch_to_nhwc(t), atol=1e-12)


# ----------------------------------------------------------------------------- BN fold (Lemma 2)
def _bn_set(C):
    return dict(mu=rng.standard_normal(C) * 0.3, var=rng.uniform(0.5, 1.5, C),
                gamma=rng.uniform(0.5, 1.5, C), beta=rng.standard_normal(C) * 0.1)


@pytest.mark.parametrize("m,eps", [(1.0, 0.0), (7.5, 0.0), (1.0, 1e-5), (999.98, 1e-3)])
def test_fold_equals_conv_bn_scale(m, eps):
    x = rng.standard_normal((2, 6, 5, 4)); w = rng.standard_normal((5, 3, 3, 4)); b = rng.standard_normal(5)
    s = _bn_set(5)
    mu, var = s["mu"] * m, s["var"] * m          # stored blobs are the statistics times m
    ref = O.scale(O.batchnorm(O.conv2d(x, w, b, 1, 1), mu, var, m, eps), s["gamma"], s["beta"])
    wf, bf = O.fold_bn(w, b, mu, var, m, eps, s["gamma"], s["beta"])
    got = O.conv2d(x, wf, bf, 1, 1)
    assert np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()
    # no-bias form
    ref0 = O.scale(O.batchnorm(O.conv2d(x, w, None, 1, 1), mu, var, m, eps), s["gamma"], s["beta"])
    wf0, bf0 = O.fold_bn(w, None, mu, var, m, eps, s["gamma"], s["beta"])
    assert np.abs(O.conv2d(x, wf0, bf0, 1, 1) - ref0).max() <= 1e-12 * np.abs(ref0).max()


def test_fold_closed_form_values():
    # eta = gamma / sqrt(var/m);  W~ = eta W;  B~ = eta B + beta - eta mu / m, typed out for one channel
    w = np.array([[[[2.0]]]]); b = np.array([0.5])
    wf, bf = O.fold_bn(w, b, np.array([3.0]), np.array([8.0]), 2.0, 0.0, np.array([4.0]), np.array([-1.0]))
    eta = 4.0 / np.sqrt(8.0 / 2.0)                 # = 2
    assert wf[0, 0, 0, 0] == eta * 2.0 == 4.0
    assert bf[0] == eta * 0.5 + (-1.0) - eta * 3.0 / 2.0 == -3.0


def test_fold_special_cases():
    w = rng.standard_normal((3, 1, 1, 2)); b = rng.standard_normal(3)
    one, zero = np.ones(3), np.zeros(3)
    wf, bf = O.fold_bn(w, b, zero, one * 5.0, 5.0, 0.0, one, zero)   # identity BN and Scale
    assert np.array_equal(wf, w) and np.array_equal(bf, b)
    s = _bn_set(3)
    a = O.fold_bn(w, b, s["mu"], s["var"], 1.0, 0.0, s["gamma"], s["beta"])
    c = O.fold_bn(w, b, 4 * s["mu"], 4 * s["var"], 4.0, 0.0, s["gamma"], s["beta"])  # (mu,var,m) -> c(mu,var,m)
    np.testing.assert_allclose(a[0], c[0], rtol=1e-14); np.testing.assert_allclose(a[1], c[1], rtol=1e-13)


def test_bn_scale_vs_torch_batch_norm():
    x = rng.standard_normal((2, 4, 3, 6)); s = _bn_set(6)
    ref = F.batch_norm(nhwc_to_torch(x), torch.from_numpy(s["mu"]), torch.from_numpy(s["var"]),
                       torch.from_numpy(s["gamma"]), torch.from_numpy(s["beta"]), False, 0.0, 1e-5)
    got = O.scale(O.batchnorm(x, s["mu"], s["var"], 1.0, 1e-5), s["gamma"], s["beta"])
    np.testing.assert_allclose(got, torch_to_nhwc(ref), atol=1e-12)


# ----------------------------------------------------------------------------- branch merge (Section 3.2)
def test_equal_kernel_branches_concatenate_exactly():
    x = rng.standard_normal((1, 6, 6, 5))
    wl, wr = rng.standard_normal((3, 3, 3, 5)), rng.standard_normal((4, 3, 3, 5))
    bl, br = rng.standard_normal(3), rng.standard_normal(4)
    merged = O.conv2d(x, np.concatenate([wl, wr]), np.concatenate([bl, br]), 1, 1)
    separate = O.concat([O.conv2d(x, wl, bl, 1, 1), O.conv2d(x, wr, br, 1, 1)])
    assert np.array_equal(merged, separate)


def test_zero_embedded_merge_equals_separate_branches():
    Cin = 6
    x = rng.standard_normal((2, 7, 6, Cin))
    w1, w5, w3 = rng.standard_normal((3, 1, 1, Cin)), rng.standard_normal((2, 5, 5, Cin)), rng.standard_normal((4, 3, 3, Cin))
    b = rng.standard_normal(9)
    wm = np.full((9, 5, 5, Cin), np.nan)          # every filter must be overwritten
    O.embed_filter(w1, 5, wm, 0); O.embed_filter(w5, 5, wm, 3); O.embed_filter(w3, 5, wm, 5)
    assert np.count_nonzero(wm[0]) == Cin and wm[0, 2, 2, 0] == w1[0, 0, 0, 0]
    assert np.array_equal(wm[5, 1:4, 1:4], w3[0]) and np.count_nonzero(wm[5]) == 9 * Cin
    merged = O.conv2d(x, wm, b, 1, 2)
    separate = O.concat([O.conv2d(x, w1, b[0:3], 1, 0), O.conv2d(x, w5, b[3:5], 1, 2), O.conv2d(x, w3, b[5:9], 1, 1)])
    assert np.array_equal(merged, separate)


def test_golden_inception_3a_channels():
    path = os.path.join(os.path.dirname(__file__), "golden", "inception_3a_channels.txt")
    g = {k: int(v) for k, v in (l.split() for l in open(path) if l.strip() and not l.startswith("#"))}
    for table in (N._INCEPTION, S.INCEPTION_V1):
        cin, c1, c3r, c3, c5r, c5, pp = table["3a"]
        assert (c3r, c3, c5, c5 + pp, c1 + c3 + c5 + pp) == (g["c3r"], g["c3"], g["c5"], g["c5_plus_pool"], g["out"])
    # every module's output width feeds the next module's input
    names = list(N._INCEPTION)
    for a, b in zip(names, names[1:]):
        _, c1, _, c3, _, c5, pp = N._INCEPTION[a]
        assert c1 + c3 + c5 + pp == N._INCEPTION[b][0]
    assert sum(N._INCEPTION["5b"][i] for i in (1, 3, 5, 6)) == 1024
    assert N._INCEPTION == S.INCEPTION_V1


# ----------------------------------------------------------------------------- max-pool
def brute_pool(x, k, s, p):
    B, H, W, C = x.shape
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    y = np.zeros((B, Ho, Wo, C)); am = np.zeros((B, Ho, Wo, C), np.int32)
    for n, ho, wo, c in itertools.product(range(B), range(Ho), range(Wo), range(C)):
        cand = [(x[n, h, w, c], h * W + w) for h in range(ho * s - p, ho * s - p + k) for w in range(wo * s - p, wo * s - p + k)
                if 0 <= h < H and 0 <= w < W]
        best = max(v for v, _ in cand)
        y[n, ho, wo, c] = best
        am[n, ho, wo, c] = min(i for v, i in cand if v == best)
    return y, am


@pytest.mark.parametrize("H,W", [(7, 7), (8, 6), (5, 9), (2, 2), (1, 1)])
def test_maxpool_vs_brute_force_and_torch(H, W):
    x = rng.standard_normal((2, H, W, 3))
    y, am = O.maxpool(x, 3, 2, 1)
    yb, ab = brute_pool(x, 3, 2, 1)
    assert np.array_equal(y, yb) and np.array_equal(am, ab)
    ty, ti = F.max_pool2d(nhwc_to_torch(x), 3, 2, 1, return_indices=True)
    assert np.array_equal(y, torch_to_nhwc(ty)) and np.array_equal(am, torch_to_nhwc(ti))


def test_maxpool_negative_input_padding_never_wins_and_ties_take_first():
    x = np.full((1, 6, 6, 2), -5.0)
    y, am = O.maxpool(x, 3, 2, 1)
    assert np.all(y == -5.0)                      # zero padding would have produced 0
    # all-equal window -> first in-bounds position in row-major order
    assert am[0, 0, 0, 0] == 0 and am[0, 1, 1, 0] == 1 * 6 + 1 and am[0, 2, 0, 1] == 3 * 6 + 0
    ramp = np.arange(36, dtype=np.float64).reshape(1, 6, 6, 1)
    y, am = O.maxpool(ramp, 3, 2, 1)
    assert np.array_equal(am[0, :, :, 0], np.array([[7, 9, 11], [19, 21, 23], [31, 33, 35]]))
    assert np.array_equal(y[0, :, :, 0], am[0, :, :, 0].astype(np.float64))


# ----------------------------------------------------------------------------- LRN
def test_lrn_closed_forms():
    v, C = 3.0, 8
    a, b, k = 1e-4, 0.75, 1.0
    y = O.lrn(np.full((1, 2, 2, C), v), 5, a, b, k)
    inner = v * (k + a * v * v) ** (-b)                 # 5 of 5 in range: (alpha/5)*5 v^2
    e1 = v * (k + 0.8 * a * v * v) ** (-b)              # channel 1 and C-2: 4 in range
    e0 = v * (k + 0.6 * a * v * v) ** (-b)              # channel 0 and C-1: 3 in range
    np.testing.assert_allclose(y[0, 0, 0], [e0, e1, inner, inner, inner, inner, e1, e0], rtol=1e-14)
    # large alpha so that a dropped 1/size or a wrong window width is far outside tolerance
    y2 = O.lrn(np.full((1, 1, 1, C), 2.0), 5, 2.0, 0.75, 1.0)
    np.testing.assert_allclose(y2[0, 0, 0, 3], 2.0 * (1.0 + 2.0 * 4.0) ** -0.75, rtol=1e-14)
    x = rng.standard_normal((1, 2, 3, 7))
    np.testing.assert_allclose(O.lrn(x, 5, 0.0, 0.75, 2.0), x * 2.0 ** -0.75, rtol=1e-14)   # alpha = 0
    np.testing.assert_allclose(O.lrn(x, 1, 0.5, 0.75, 1.0), x * (1 + 0.5 * x * x) ** -0.75, rtol=1e-14)  # n = 1


@pytest.mark.parametrize("C,size", [(7, 5), (64, 5), (3, 5), (9, 3)])
def test_lrn_vs_torch(C, size):
    x = rng.standard_normal((2, 3, 2, C)) * 4
    ref = F.local_response_norm(nhwc_to_torch(x), size, alpha=0.3, beta=0.75, k=1.5)
    np.testing.assert_allclose(O.lrn(x, size, 0.3, 0.75, 1.5), torch_to_nhwc(ref), rtol=1e-12)


# ----------------------------------------------------------------------------- small definitions
def test_relu_add_concat_avgpool():
    a, b = rng.standard_normal((2, 2, 3, 3, 4))
    assert np.array_equal(O.relu(a), np.maximum(a, 0))
    assert np.array_equal(O.add(a, b), a + b)
    c = rng.standard_normal((2, 3, 3, 2))
    assert np.array_equal(O.concat([a, c, b]), np.concatenate([a, c, b], axis=-1))
    np.testing.assert_allclose(O.avgpool_global(a)[:, 0, 0, :], a.mean(axis=(1, 2)), rtol=1e-14)


def test_round_bf16_matches_torch_and_ties_to_even():
    a = (rng.standard_normal(20000) * np.exp(rng.uniform(-20, 20, 20000))).astype(np.float32)
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(a.astype(np.float64)), ref)
    assert np.array_equal(S.round_bf16(a).astype(np.float64), ref)
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: ties go to the even mantissa (1.0);
    # 1 + 3*2^-8 lies halfway between 1+2^-7 and 1+2^-6: goes up to 1 + 2^-6
    assert O.round_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert O.round_bf16(np.array([1 + 3 * 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    assert O.round_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -30]))[0] == 1 + 2.0 ** -7   # double is not pre-rounded to float


# ----------------------------------------------------------------------------- composition vs an independent float64 library
def _t_conv(p, name, t, s, pad):
    b = p.get(name + ".b")
    return F.conv2d(t, w_to_torch(p[name + ".w"].astype(np.float64)), None if b is None else torch.from_numpy(b.astype(np.float64)),
                    stride=s, padding=pad)


def _t_bn(p, name, t, eps=1e-5):
    g = lambda k: torch.from_numpy(p[f"{name}.bn.{k}"].astype(np.float64))
    return F.batch_norm(t, g("mean"), g("var"), g("gamma"), g("beta"), False, 0.0, eps)


def test_stem_and_inception_composition_vs_torch():
    p = {}
    p.update(P.conv_params(0, "conv1", 64, 7, 3))
    table = {"t": (16, 8, 12, 16, 4, 8, 8)}
    p.update(P.inception_params(0, "t", table))
    x = P.images(0, 2, 20, 18)
    out = N.run(N.stem_steps(p), x, rounding=False)
    t = F.local_response_norm(F.max_pool2d(F.relu(_t_conv(p, "conv1", nhwc_to_torch(x.astype(np.float64)), 2, 3)), 3, 2, 1),
                              5, alpha=1e-4, beta=0.75, k=1.0)
    np.testing.assert_allclose(out["conv1"], torch_to_nhwc(t), atol=1e-11)

    xi = rng.standard_normal((1, 6, 5, 16))
    out = N.run(N.inception_steps(p, "t", "x", table), xi, rounding=False)
    ti = nhwc_to_torch(xi)
    three = F.relu(_t_conv(p, "t.3x3", F.relu(_t_conv(p, "t.3x3r", ti, 1, 0)), 1, 1))
    ref = torch.cat([three, F.relu(_t_conv(p, "t.b1", ti, 1, 0)), F.relu(_t_conv(p, "t.b5", ti, 1, 2)),
                     F.relu(_t_conv(p, "t.bp", ti, 1, 1))], dim=1)
    np.testing.assert_allclose(out["t"], torch_to_nhwc(ref), atol=1e-11)
    assert out["t"].shape[-1] == 16 + 8 + 8 + 8


def test_googlenet_composition_vs_torch_one_image():
    p = P.googlenet_params(0)
    x = P.images(0, 1)
    out = N.run(N.googlenet_steps(p), x, rounding=False)
    lrn = lambda t: F.local_response_norm(t, 5, alpha=1e-4, beta=0.75, k=1.0)
    pool = lambda t: F.max_pool2d(t, 3, 2, 1)
    t = nhwc_to_torch(x.astype(np.float64))
    t = lrn(pool(F.relu(_t_conv(p, "conv1", t, 2, 3))))
    t = F.relu(_t_conv(p, "conv2r", t, 1, 0))
    t = pool(lrn(F.relu(_t_conv(p, "conv2", t, 1, 1))))
    for m in S.INCEPTION_V1:
        three = F.relu(_t_conv(p, f"{m}.3x3", F.relu(_t_conv(p, f"{m}.3x3r", t, 1, 0)), 1, 1))
        t = torch.cat([three, F.relu(_t_conv(p, f"{m}.b1", t, 1, 0)), F.relu(_t_conv(p, f"{m}.b5", t, 1, 2)),
                       F.relu(_t_conv(p, f"{m}.bp", t, 1, 1))], dim=1)
        if m in ("3b", "4e"):
            t = pool(t)
    assert t.shape[1:] == (1024, 7, 7)
    t = _t_conv(p, "fc", t.mean(dim=(2, 3), keepdim=True), 1, 0)
    ref = torch_to_nhwc(t)
    assert out["fc"].shape == (1, 1, 1, 1000)
    assert np.abs(out["fc"] - ref).max() <= 1e-10 * np.abs(ref).max()


def test_googlenet_paper_form_composition_vs_torch():
    p = P.googlenet_paper_params(0)
    x = P.images(0, 1, 96, 96)
    out = N.run(N.googlenet_paper_steps(p), x, rounding=False)
    lrn = lambda t: F.local_response_norm(t, 5, alpha=1e-4, beta=0.75, k=1.0)
    pool = lambda t: F.max_pool2d(t, 3, 2, 1)
    t = nhwc_to_torch(x.astype(np.float64))
    t = lrn(pool(F.relu(_t_conv(p, "conv1", t, 2, 3))))
    t = F.relu(_t_conv(p, "conv2r", t, 1, 0))
    t = pool(lrn(F.relu(_t_conv(p, "conv2", t, 1, 1))))
    for m in S.INCEPTION_V1:
        a = F.relu(_t_conv(p, f"{m}.p3", F.relu(_t_conv(p, f"{m}.p3r", t, 1, 0)), 1, 1))
        b = F.relu(_t_conv(p, f"{m}.p5", F.relu(_t_conv(p, f"{m}.p5r", t, 1, 0)), 1, 2))
        t = torch.cat([a, b], dim=1)
        if m in ("3b", "4e"):
            t = pool(t)
    ref = torch_to_nhwc(_t_conv(p, "fc", t.mean(dim=(2, 3), keepdim=True), 1, 0))
    assert np.abs(out["fc"] - ref).max() <= 1e-10 * np.abs(ref).max()
    # Section 3.2's numbers for 3a: 3x3 reducer 96 -> 48, 3x3 conv 128 -> 192 (printed "196"), 5x5 conv 32 -> 64
    assert p["3a.p3r.w"].shape[0] == 48 and p["3a.p3.w"].shape[0] == 192 and p["3a.p5.w"].shape[0] == 64


def test_googlenet_streamline_composition_vs_torch():
    """Stem of Section 3.1 (Method): conv stride = conv stride x pool stride, no pool, no LRN, ReLU kept."""
    p = P.googlenet_params(0)
    x = P.images(0, 1, 96, 96)
    out = N.run(N.googlenet_streamline_steps(p), x, rounding=False)
    pool = lambda t: F.max_pool2d(t, 3, 2, 1)
    t = nhwc_to_torch(x.astype(np.float64))
    t = F.relu(_t_conv(p, "conv1", t, 4, 3))
    assert tuple(out["conv1"].shape) == (1, 24, 24, 64) and np.abs(out["conv1"] - torch_to_nhwc(t)).max() <= 1e-10 * float(t.abs().max())
    t = F.relu(_t_conv(p, "conv2", F.relu(_t_conv(p, "conv2r", t, 1, 0)), 2, 1))
    assert tuple(out["conv2"].shape) == (1, 12, 12, 192)
    for m in S.INCEPTION_V1:
        three = F.relu(_t_conv(p, f"{m}.3x3", F.relu(_t_conv(p, f"{m}.3x3r", t, 1, 0)), 1, 1))
        t = torch.cat([three, F.relu(_t_conv(p, f"{m}.b1", t, 1, 0)), F.relu(_t_conv(p, f"{m}.b5", t, 1, 2)),
                       F.relu(_t_conv(p, f"{m}.bp", t, 1, 1))], dim=1)
        if m in ("3b", "4e"):
            t = pool(t)
    ref = torch_to_nhwc(_t_conv(p, "fc", t.mean(dim=(2, 3), keepdim=True), 1, 0))
    assert np.abs(out["fc"] - ref).max() <= 1e-10 * np.abs(ref).max()
    # the exact stem and the approximate one give different functions (the paper re-trains): same shapes only
    exact = N.run(N.googlenet_steps(p), x, rounding=False)
    assert exact["conv2"].shape == out["conv2"].shape and np.abs(exact["conv2"] - out["conv2"]).max() > 1e-3


def test_resnet50_composition_vs_torch_small_image():
    p = P.resnet50_params(0)
    x = P.images(0, 1, 64, 64)
    steps = N.resnet50_steps(p, eps=1e-5)
    assert sum(1 for s in steps if not s.virtual) == 1 + 16 * 3 + 4 + 2   # 53 convs incl. fc, + avg-pool
    out = N.run(steps, x, rounding=False)
    t = nhwc_to_torch(x.astype(np.float64))
    t = F.max_pool2d(F.relu(_t_bn(p, "conv1", _t_conv(p, "conv1", t, 2, 3))), 3, 2, 1)
    for si, (w, n) in enumerate(S.RESNET50_STAGES):
        for b in range(n):
            blk = f"res{si + 2}{chr(97 + b)}"
            s = 2 if (b == 0 and si > 0) else 1
            r = _t_bn(p, f"{blk}.br1", _t_conv(p, f"{blk}.br1", t, s, 0)) if b == 0 else t
            u = F.relu(_t_bn(p, f"{blk}.2a", _t_conv(p, f"{blk}.2a", t, s, 0)))
            u = F.relu(_t_bn(p, f"{blk}.2b", _t_conv(p, f"{blk}.2b", u, 1, 1)))
            t = F.relu(_t_bn(p, f"{blk}.2c", _t_conv(p, f"{blk}.2c", u, 1, 0)) + r)
    assert t.shape[1:] == (2048, 2, 2)
    ref = torch_to_nhwc(_t_conv(p, "fc", t.mean(dim=(2, 3), keepdim=True), 1, 0))
    assert np.abs(out["fc"] - ref).max() <= 1e-10 * np.abs(ref).max()


def test_teacher_forcing_uses_given_tensors():
    p = P.conv_params(0, "conv1", 64, 7, 3)
    x = P.images(0, 1, 16, 16)
    free = N.run(N.stem_steps(p), x)
    forced = N.run(N.stem_steps(p), x * 0, given={"x": x})
    assert np.array_equal(free["conv1"], forced["conv1"])
    assert np.array_equal(free["conv1"], O.round_bf16(free["conv1"]))


# ---- grouped convolution and AlexNet (Section 4.3: conv1 + norm1, conv2 + norm2 slimmed) ------------------
def test_grouped_conv_vs_torch_and_block_diagonal_dense():
    """Grouped convolution against the library routine, and against the dense convolution whose filters are the
    grouped ones placed block-diagonally (zeros across groups): the identity the GPU path relies on."""
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 9, 7, 12))
    w = rng.standard_normal((10, 3, 3, 6))           # groups = 2: Cin_g = 6, Cout_g = 5
    b = rng.standard_normal(10)
    y = O.conv2d_grouped(x, w, b, 1, 1, 2)
    ref = F.conv2d(nhwc_to_torch(x), w_to_torch(w), torch.from_numpy(b), stride=1, padding=1, groups=2)
    assert np.abs(y - torch_to_nhwc(ref)).max() <= 1e-12 * float(ref.abs().max())
    dense = np.zeros((10, 3, 3, 12))
    dense[:5, :, :, :6] = w[:5]
    dense[5:, :, :, 6:] = w[5:]
    assert np.array_equal(O.conv2d(x, dense, b, 1, 1), y) or np.abs(O.conv2d(x, dense, b, 1, 1) - y).max() <= 1e-13 * np.abs(y).max()
    # a wrong group assignment is caught: swapping the input halves changes the result
    assert np.abs(O.conv2d_grouped(x[..., ::-1].copy(), w, b, 1, 1, 2) - y).max() > 1e-3
    # groups = 1 is the plain convolution
    w1 = rng.standard_normal((4, 3, 3, 12))
    assert np.array_equal(O.conv2d_grouped(x, w1, None, 2, 0, 1), O.conv2d(x, w1, None, 2, 0))


def test_alexnet_composition_vs_torch():
    """Whole AlexNet (227x227, two-tower groups, LRN after conv1/conv2, unpadded 3x3/2 pools) vs PyTorch float64."""
    p = P.alexnet_params(0)
    assert p["conv2.w"].shape == (256, 5, 5, 48) and p["conv4.w"].shape == (384, 3, 3, 192) and p["fc6.w"].shape == (4096, 6, 6, 256)
    x = P.images(0, 1, 227, 227)
    steps = N.alexnet_steps(p)
    out = N.run(steps, x, rounding=False)
    assert [out[n].shape[1] for n in ("conv1", "pool1", "conv2", "pool2", "conv5", "pool5", "fc6")] == [55, 27, 27, 13, 13, 6, 1]

    def tc(name, t, s, pad, groups=1):
        return F.conv2d(t, w_to_torch(p[name + ".w"].astype(np.float64)), torch.from_numpy(p[name + ".b"].astype(np.float64)),
                        stride=s, padding=pad, groups=groups)
    lrn = lambda t: F.local_response_norm(t, 5, alpha=1e-4, beta=0.75, k=1.0)
    pool = lambda t: F.max_pool2d(t, 3, 2, 0)
    t = nhwc_to_torch(x.astype(np.float64))
    t = pool(lrn(F.relu(tc("conv1", t, 4, 0))))
    assert np.abs(out["pool1"] - torch_to_nhwc(t)).max() <= 1e-10 * float(t.abs().max())
    t = pool(lrn(F.relu(tc("conv2", t, 1, 2, 2))))
    assert np.abs(out["pool2"] - torch_to_nhwc(t)).max() <= 1e-10 * float(t.abs().max())
    t = F.relu(tc("conv3", t, 1, 1))
    t = F.relu(tc("conv4", t, 1, 1, 2))
    t = pool(F.relu(tc("conv5", t, 1, 1, 2)))
    t = F.relu(tc("fc6", t, 1, 0))
    t = F.relu(tc("fc7", t, 1, 0))
    ref = torch_to_nhwc(tc("fc8", t, 1, 0))
    assert out["fc8"].shape == (1, 1, 1, 1000) and np.abs(out["fc8"] - ref).max() <= 1e-10 * np.abs(ref).max()


def _np_space_to_depth(x, k, s, pad, Cp):
    """y[n][R][S][(ah*s + aw)*C + c] = x[n][R*s + ah - pad][S*s + aw - pad][c], zero elsewhere (written out for the pin)."""
    B, H, W, C = x.shape
    kp = -(-k // s)
    Hs, Ws = (H + 2 * pad - k) // s + kp, (W + 2 * pad - k) // s + kp
    y = np.zeros((B, Hs, Ws, Cp), x.dtype)
    for R in range(Hs):
        for S_ in range(Ws):
            for ah in range(s):
                for aw in range(s):
                    h, w = R * s + ah - pad, S_ * s + aw - pad
                    if 0 <= h < H and 0 <= w < W:
                        y[:, R, S_, (ah * s + aw) * C:(ah * s + aw + 1) * C] = x[:, h, w, :]
    return y


def _np_s2d_filter(w, s, Cp):
    Cout, k, _, C = w.shape
    kp = -(-k // s)
    o = np.zeros((Cout, kp, kp, Cp), w.dtype)
    for r in range(k):
        for q in range(k):
            o[:, r // s, q // s, ((r % s) * s + q % s) * C:((r % s) * s + q % s + 1) * C] = w[:, r, q, :]
    return o


@pytest.mark.parametrize("H,W,k,s,pad", [(35, 31, 11, 4, 0), (32, 40, 7, 4, 3), (17, 18, 5, 2, 2), (20, 20, 3, 3, 1)])
def test_space_to_depth_identity(H, W, k, s, pad):
    """A strided convolution over a few channels equals the stride-1 convolution of the space-to-depth image with
    the re-laid filters (the form the tensor-core kernels run AlexNet's conv1 and the stride-product stem in)."""
    rng = np.random.default_rng(7)
    x = rng.standard_normal((2, H, W, 3)); w = rng.standard_normal((5, k, k, 3)); b = rng.standard_normal(5)
    ref = O.conv2d(x, w, b, s, pad)
    got = O.conv2d(_np_space_to_depth(x, k, s, pad, 64), _np_s2d_filter(w, s, 64), b, 1, 0)
    assert got.shape == ref.shape and np.abs(got - ref).max() <= 1e-12 * np.abs(ref).max()
