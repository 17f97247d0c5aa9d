"""GPU parity of the stand-alone non-tensor kernels and the parameter kernels against the CPU checker."""
import numpy as np
import pytest

import dr_synth as S
from util import assert_layer_close, to_dev_bf16, to_dev_f32, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dr():
    import paper_1708_04728_b200 as dr
    return dr


@pytest.fixture(scope="module")
def O():
    import oracle
    return oracle


def _empty_like_bf16(shape):
    import torch
    return torch.empty(shape, dtype=torch.bfloat16, device="cuda")


SHAPES = [(2, 7, 9, 64), (1, 5, 6, 24), (3, 4, 4, 200), (1, 3, 5, 7), (1, 14, 14, 832)]


@pytest.mark.parametrize("shape", SHAPES + [(1, 1, 1, 3)])
def test_relu_and_add_exact(dr, O, shape):
    a, b = S.normal(1, "a", shape), S.normal(1, "b", shape)
    ta, tb = to_dev_bf16(a), to_dev_bf16(b)
    y = _empty_like_bf16(shape)
    dr.dr_relu(a.size, ta, y)
    assert np.array_equal(to_host(y), O.relu(a))          # exact: max with zero
    dr.dr_add(a.size, ta, tb, y)
    assert np.array_equal(to_host(y), O.round_bf16(O.add(a, b)))   # one rounding of an exact fp32 sum


def test_empty_inputs_are_accepted(dr):
    y = _empty_like_bf16((8,))
    dr.dr_relu(0, y, y)
    dr.dr_add(0, y, y, y)
    dr.dr_maxpool(0, 4, 4, 8, 3, 2, 1, y, y)
    dr.dr_lrn(0, 4, 4, 8, 5, 1e-4, 0.75, 1.0, y, y)
    assert dr.dr_device_status()[0] == 0


@pytest.mark.parametrize("shape", SHAPES + [(2, 112, 112, 64), (1, 2, 2, 8), (1, 1, 1, 16)])
def test_maxpool_bit_exact_with_argmax(dr, O, shape):
    import torch
    B, H, W, Cc = shape
    x = S.normal(2, "x", shape)
    # plant exact ties: duplicate the maximum inside some windows
    x[:, 0:2, 0:2, :] = x[:, 0:1, 0:1, :]
    ref, ref_arg = O.maxpool(x, 3, 2, 1)
    y = _empty_like_bf16(ref.shape)
    arg = torch.empty(ref.shape, dtype=torch.int32, device="cuda")
    dr.dr_maxpool(B, H, W, Cc, 3, 2, 1, to_dev_bf16(x), y, arg)
    assert np.array_equal(to_host(y), ref)
    assert np.array_equal(arg.cpu().numpy(), ref_arg)
    y2 = _empty_like_bf16(ref.shape)
    dr.dr_maxpool(B, H, W, Cc, 3, 2, 1, to_dev_bf16(x), y2, None)     # the path without argmax (packed maxima)
    assert np.array_equal(to_host(y2), ref)


def test_maxpool_other_geometry(dr, O):
    x = S.normal(3, "x", (2, 9, 8, 16))
    for k, s, p in [(2, 2, 0), (3, 1, 1), (3, 2, 0)]:
        ref, ref_arg = O.maxpool(x, k, s, p)
        import torch
        y = _empty_like_bf16(ref.shape); arg = torch.empty(ref.shape, dtype=torch.int32, device="cuda")
        dr.dr_maxpool(2, 9, 8, 16, k, s, p, to_dev_bf16(x), y, arg)
        assert np.array_equal(to_host(y), ref) and np.array_equal(arg.cpu().numpy(), ref_arg)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("size,alpha,beta,k", [(5, 1e-4, 0.75, 1.0), (5, 0.5, 0.75, 2.0), (3, 1.0, 0.5, 1.0), (9, 0.3, 0.75, 1.0)])
def test_lrn(dr, O, shape, size, alpha, beta, k):
    B, H, W, Cc = shape
    x = S.normal(4, "x", shape, std=3.0)
    y = _empty_like_bf16(shape)
    dr.dr_lrn(B, H, W, Cc, size, alpha, beta, k, to_dev_bf16(x), y)
    assert_layer_close(to_host(y), O.round_bf16(O.lrn(x, size, alpha, beta, k)), "lrn")


@pytest.mark.parametrize("shape", SHAPES)
def test_bn_and_scale(dr, O, shape):
    B, H, W, Cc = shape
    x = S.normal(5, "x", shape)
    mean, var = S.normal(5, "m", (Cc,), 0.1), S.uniform(5, "v", (Cc,), 0.5, 1.5)
    gamma, beta = S.uniform(5, "g", (Cc,), 0.5, 1.5), S.normal(5, "b", (Cc,), 0.1)
    dm, dv, dg, db = map(to_dev_f32, (mean * 3.0, var * 3.0, gamma, beta))
    y = _empty_like_bf16(shape)
    dr.dr_bn(B, H, W, Cc, to_dev_bf16(x), dm, dv, 3.0, 1e-5, None, None, y)        # BatchNorm layer alone, m = 3
    ref_bn = O.batchnorm(x, mean.astype(np.float64) * 3.0, var.astype(np.float64) * 3.0, 3.0, 1e-5)
    assert_layer_close(to_host(y), O.round_bf16(ref_bn), "bn")
    dr.dr_bn(B, H, W, Cc, to_dev_bf16(x), dm, dv, 3.0, 1e-5, dg, db, y)            # BatchNorm + Scale
    assert_layer_close(to_host(y), O.round_bf16(O.scale(ref_bn, gamma, beta)), "bn+scale")
    dr.dr_scale(B, H, W, Cc, to_dev_bf16(x), dg, db, y)                            # Scale layer alone
    assert_layer_close(to_host(y), O.round_bf16(O.scale(x, gamma, beta)), "scale")


def test_concat_and_avgpool(dr, O):
    parts = [S.normal(6, f"p{i}", (2, 5, 5, c)) for i, c in enumerate((16, 8, 24))]
    y = _empty_like_bf16((2, 5, 5, 48))
    off = 0
    for p in parts:
        dr.dr_concat(2 * 5 * 5, p.shape[-1], to_dev_bf16(p), 48, off, y)
        off += p.shape[-1]
    assert np.array_equal(to_host(y), O.concat(parts))
    for shape in [(3, 7, 7, 1024), (2, 2, 2, 2048), (1, 5, 3, 70)]:
        x = S.normal(6, "x", shape)
        ya = _empty_like_bf16((shape[0], 1, 1, shape[3]))
        dr.dr_avgpool_global(*shape, to_dev_bf16(x), ya)
        assert_layer_close(to_host(ya), O.round_bf16(O.avgpool_global(x)), "avgpool")


@pytest.mark.parametrize("Cout,k,Cin,bias", [(64, 7, 3, False), (96, 1, 192, True), (256, 3, 64, False)])
def test_fold_bn_matches_closed_form(dr, O, Cout, k, Cin, bias):
    import torch
    w = S.he_normal(7, "w", Cout, k, Cin)
    b = S.normal(7, "b", (Cout,), 0.1) if bias else None
    mean, var = S.normal(7, "m", (Cout,), 0.1), S.uniform(7, "v", (Cout,), 0.5, 1.5)
    gamma, beta = S.uniform(7, "g", (Cout,), 0.5, 1.5), S.normal(7, "be", (Cout,), 0.1)
    wo = _empty_like_bf16(w.shape); bo = torch.empty(Cout, dtype=torch.float32, device="cuda")
    dr.dr_fold_bn(Cout, k * k * Cin, to_dev_bf16(w), None if b is None else to_dev_f32(b), to_dev_f32(mean * 2), to_dev_f32(var * 2),
                  2.0, 1e-5, to_dev_f32(gamma), to_dev_f32(beta), wo, bo)
    wr, br = O.fold_bn(w, b, mean.astype(np.float64) * 2, var.astype(np.float64) * 2, 2.0, 1e-5, gamma, beta)
    got_w = to_host(wo)
    # folded weights are bfloat16: within one rounding step (2^-8 relative) of the float64 closed form
    assert np.all(np.abs(got_w - wr) <= 2.0 ** -8 * np.abs(wr) + 1e-30)
    assert np.abs(bo.cpu().numpy().astype(np.float64) - br).max() <= 1e-6 * max(1.0, np.abs(br).max())


def test_embed_filter_exact(dr, O):
    Cin = 24
    w1, w5, w3 = S.he_normal(8, "w1", 8, 1, Cin), S.he_normal(8, "w5", 4, 5, Cin), S.he_normal(8, "w3", 12, 3, Cin)
    big = _empty_like_bf16((24, 5, 5, Cin))
    dr.dr_embed_filter(8, Cin, 1, 5, to_dev_bf16(w1), 0, big)
    dr.dr_embed_filter(4, Cin, 5, 5, to_dev_bf16(w5), 8, big)
    dr.dr_embed_filter(12, Cin, 3, 5, to_dev_bf16(w3), 12, big)
    ref = np.zeros((24, 5, 5, Cin))
    O.embed_filter(w1, 5, ref, 0); O.embed_filter(w5, 5, ref, 8); O.embed_filter(w3, 5, ref, 12)
    assert np.array_equal(to_host(big), ref)


@pytest.mark.parametrize("B,H,W,k,s,pad,Cout", [(2, 227, 227, 11, 4, 0, 96), (1, 224, 224, 7, 4, 3, 64), (3, 37, 29, 5, 2, 2, 32)])
def test_space_to_depth_conv(dr, O, B, H, W, k, s, pad, Cout):
    """dr_space_to_depth / dr_s2d_filter: the re-laid tensors are bit-exact copies (against a restatement of the index
    map), and the stride-1 convolution over them matches the checker's strided convolution of the original."""
    import torch
    from test_oracle_pins import _np_s2d_filter, _np_space_to_depth
    x = S.normal(40, "x", (B, H, W, 3)); w = S.he_normal(40, "w", Cout, k, 3); b = S.normal(40, "b", (Cout,), 0.1)
    kp = -(-k // s)
    Ho, Wo = (H + 2 * pad - k) // s + 1, (W + 2 * pad - k) // s + 1
    y = torch.full((B, Ho + kp - 1, Wo + kp - 1, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    wr = torch.full((Cout, kp, kp, 64), 7.0, dtype=torch.bfloat16, device="cuda")
    dr.dr_space_to_depth(B, H, W, 3, k, s, pad, 64, to_dev_bf16(x), y)
    dr.dr_s2d_filter(Cout, k, 3, s, 64, to_dev_bf16(w), wr)
    assert np.array_equal(to_host(y), _np_space_to_depth(x.astype(np.float64), k, s, pad, 64))
    assert np.array_equal(to_host(wr), _np_s2d_filter(w.astype(np.float64), s, 64))
    d = dr.dr_conv_desc(k=kp, stride=1, pad=0, Cin=64, Cout=Cout, flags=dr.DR_BIAS | dr.DR_RELU)
    out = torch.empty((B, Ho, Wo, Cout), dtype=torch.bfloat16, device="cuda")
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    dr.dr_conv_slim(d, B, Ho + kp - 1, Wo + kp - 1, y, wr, to_dev_f32(b), None, out)
    assert dr.dr_device_status()[0] == 0 and dr.dr_last_conv_path() == dr.DR_PATH_UMMA_TMA
    assert_layer_close(to_host(out), O.round_bf16(O.relu(O.conv2d(x, w, b, s, pad))), "space-to-depth conv")
