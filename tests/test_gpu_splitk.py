"""GPU parity of the split-K convolution kernel (dr_conv_slim_ws) against the unfused CPU checker.

The kernel takes layers with few output pixels and a long reduction — single-image inference,
the regime of the paper's timings (Section 4.1).  Cases: the merged 5x5 convolutions of the
14x14 and 7x7 inception stages at batch 1, a 3x3 layer, tiles that span two images, the FC layer
with float32 output and a channel count that is not a multiple of 16, a residual epilogue, and a
store into a channel slice.  Integer-free arithmetic: the bar is the per-layer tolerance.
"""
import numpy as np
import pytest

import dr_synth as S
from util import assert_layer_close, to_dev_bf16, to_dev_f32, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dr():
    import paper_1708_04728_b200 as dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)
    yield dr
    dr.dr_set_conv_path(dr.DR_PATH_AUTO)


@pytest.fixture(scope="module")
def O():
    import oracle
    return oracle


def run_ws(dr, x, w, b, k, s, p, flags, residual=None, ldc=0, coff=0, ws=None, expect_splitk=True):
    import torch
    B, H, W, Cin = x.shape
    Cout = w.shape[0]
    d = dr.dr_conv_desc(k=k, stride=s, pad=p, Cin=Cin, Cout=Cout, flags=flags, pool_k=3, pool_stride=2, pool_pad=1,
                        lrn_size=5, lrn_alpha=1e-4, lrn_beta=0.75, lrn_k=1.0, y_ldc=ldc, y_coff=coff)
    Ho, Wo = (H + 2 * p - k) // s + 1, (W + 2 * p - k) // s + 1
    L = ldc or Cout
    dt = torch.float32 if flags & dr.DR_OUT_F32 else torch.bfloat16
    y = torch.full((B, Ho, Wo, L), 768.0, dtype=dt, device="cuda")
    need = dr.dr_conv_workspace_bytes(d, B, H, W)
    if expect_splitk:
        assert need > dr.DR_CONV_WS_COUNTER_BYTES, "the layer was expected to want split-K scratch"
    if ws is None:
        ws = torch.empty(max(need, 4096) + 256, dtype=torch.uint8, device="cuda")
        ws = ws[(-ws.data_ptr()) % 256:]
        ws[:dr.DR_CONV_WS_COUNTER_BYTES].zero_()
        ws[dr.DR_CONV_WS_COUNTER_BYTES:].fill_(0xFF)          # NaN bit patterns: stale scratch must never reach the output
    dr.dr_conv_slim_ws(d, B, H, W, to_dev_bf16(x), to_dev_bf16(w), None if b is None else to_dev_f32(b),
                       None if residual is None else to_dev_bf16(residual), y, None, ws, ws.numel())
    st, info = dr.dr_device_status()
    assert st == 0, f"device status {st} {info}"
    if expect_splitk:
        assert dr.dr_last_conv_path() == dr.DR_PATH_UMMA_SPLITK
        assert int(ws[:dr.DR_CONV_WS_COUNTER_BYTES].view(torch.int32).abs().sum()) == 0, "tile counters not left at zero"
    yh = to_host(y)
    if L != Cout:
        mask = np.ones(L, bool); mask[coff:coff + Cout] = False
        assert np.all(yh[..., mask] == 768.0), "wrote outside its channel slice"
    return yh[..., coff:coff + Cout], ws, y


# (B,H,W,Cin,Cout,k,s,p)
SHAPES = [
    (1, 14, 14, 480, 304, 5, 1, 2),    # 4a merged 5x5: two m-tiles (196 pixels), 32-channel K tail
    (1, 7, 7, 832, 640, 5, 1, 2),      # 5b merged 5x5: 49 pixels, K = 20800
    (1, 14, 14, 528, 512, 5, 1, 2),    # 4e merged 5x5: 16-channel K tail
    (1, 28, 28, 192, 128, 5, 1, 2),    # 3a merged 5x5: seven m-tiles
    (1, 14, 14, 96, 208, 3, 1, 1),     # 4a 3x3
    (2, 7, 7, 160, 320, 3, 1, 1),      # 98 pixels: the tile spans two images
    (1, 7, 7, 1024, 256, 1, 1, 0),     # 1x1 with K = 1024, plain 2-D loads
    (3, 9, 5, 72, 24, 3, 2, 1),        # stride 2, 8-channel K tail, Cout = 24 (16-column tail, not a multiple of 16)
]


@pytest.mark.parametrize("shape", SHAPES)
def test_splitk_bias_relu(dr, O, shape):
    B, H, W, Cin, Cout, k, s, p = shape
    x = S.normal(30, "x", (B, H, W, Cin)); w = S.he_normal(30, "w", Cout, k, Cin); b = S.normal(30, "b", (Cout,), 0.1)
    got, ws, _ = run_ws(dr, x, w, b, k, s, p, dr.DR_BIAS | dr.DR_RELU)
    ref = O.relu(O.conv2d(x, w, b, s, p))
    assert_layer_close(got, O.round_bf16(ref), f"split-K {shape}")
    # a second call on the same workspace (counters re-armed by the first) gives bit-identical output
    got2, _, _ = run_ws(dr, x, w, b, k, s, p, dr.DR_BIAS | dr.DR_RELU, ws=ws)
    assert np.array_equal(got, got2)


def test_splitk_fc_f32_and_slice(dr, O):
    x = S.normal(31, "x", (1, 1, 1, 1024)); w = S.he_normal(31, "w", 1000, 1, 1024); b = S.normal(31, "b", (1000,), 0.1)
    got, _, _ = run_ws(dr, x, w, b, 1, 1, 0, dr.DR_BIAS | dr.DR_OUT_F32)
    ref = O.conv2d(x, w, b, 1, 0)
    assert np.abs(got - ref).max() <= 2e-3 * np.abs(ref).max()
    x = S.normal(32, "x", (1, 14, 14, 480)); w = S.he_normal(32, "w", 304, 5, 480)
    got, _, _ = run_ws(dr, x, w, None, 5, 1, 2, 0, ldc=512, coff=208)       # raw conv into channels [208, 512)
    assert_layer_close(got, O.round_bf16(O.conv2d(x, w, None, 1, 2)), "slice")


def test_splitk_residual_relu(dr, O):
    B, H, W, Cin, Cout = 1, 7, 7, 1024, 2048
    x = S.normal(33, "x", (B, H, W, Cin)); w = S.he_normal(33, "w", Cout, 1, Cin); b = S.normal(33, "b", (Cout,), 0.1)
    r = S.normal(33, "r", (B, H, W, Cout))
    flags = dr.DR_BIAS | dr.DR_RESIDUAL | dr.DR_RELU_AFTER_RESIDUAL
    got, _, _ = run_ws(dr, x, w, b, 1, 1, 0, flags, residual=r)
    ref = O.relu(O.add(O.conv2d(x, w, b, 1, 0), r))
    assert_layer_close(got, O.round_bf16(ref), "residual")


def test_large_layers_and_missing_workspace_take_the_persistent_kernel(dr, O):
    x = S.normal(34, "x", (1, 14, 14, 480)); w = S.he_normal(34, "w", 304, 5, 480); b = S.normal(34, "b", (304,), 0.1)
    import torch
    d = dr.dr_conv_desc(k=5, stride=1, pad=2, Cin=480, Cout=304, flags=dr.DR_BIAS | dr.DR_RELU)
    assert dr.dr_conv_workspace_bytes(d, 256, 14, 14) == 0          # enough tiles for the persistent kernel
    y = torch.empty((1, 14, 14, 304), dtype=torch.bfloat16, device="cuda")
    dr.dr_conv_slim_ws(d, 1, 14, 14, to_dev_bf16(x), to_dev_bf16(w), to_dev_f32(b), None, y, None, None, 0)
    assert dr.dr_device_status()[0] == 0 and dr.dr_last_conv_path() == dr.DR_PATH_UMMA_TMA
    small = torch.zeros(4096, dtype=torch.uint8, device="cuda")     # too small for the partial tiles: not an error
    y2 = torch.empty_like(y)
    dr.dr_conv_slim_ws(d, 1, 14, 14, to_dev_bf16(x), to_dev_bf16(w), to_dev_f32(b), None, y2, None, small, small.numel())
    assert dr.dr_device_status()[0] == 0 and dr.dr_last_conv_path() == dr.DR_PATH_UMMA_TMA
    ref = O.round_bf16(O.relu(O.conv2d(x, w, b, 1, 2)))
    assert_layer_close(to_host(y), ref, "no workspace")
    assert np.array_equal(to_host(y), to_host(y2))
